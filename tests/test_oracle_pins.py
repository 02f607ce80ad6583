"""Pins for the CPU oracle: it is checked here against things other than itself — library
routines (scipy log_softmax, numpy stable argsort / argmax), brute-force enumeration of all
nodes and of all prefix-closed trees, closed forms, a hand-worked example, and the invariants
the paper proves (Lemma 1, Theorem 1, Corollaries 1-2).  No GPU involved."""
import itertools
import math
import os

import numpy as np
import pytest
import torch
from scipy.special import log_softmax

from oracle import cadd_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def f64(t):
    return t.to(torch.float64).numpy()


def quad_coef(batch, t_draft, a, b, c):
    return torch.tensor([[t_draft, a, b, c]] * batch, dtype=torch.float64)


def rand_logits(seed, batch, L, V, dtype=torch.float32, scale=2.0, quant=None):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(batch, L, V, generator=g) * scale
    if quant:
        x = torch.round(x * quant) / quant      # force exact ties
    return x.to(dtype)


# ---------------------------------------------------------------- O1 / O2: softmax + top-K
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V,K", [(7, 3), (1000, 8), (4099, 32)])
def test_softmax_topk_matches_library(dtype, V, K):
    g = torch.Generator().manual_seed(V + K)
    for trial in range(4):
        row = (torch.randn(V, generator=g) * (1 + trial)).to(dtype)
        m, lz, tok, a, lp, ke, nf, pinf = O.row_softmax_topk(row, K)
        x = f64(row)
        ref_lp = log_softmax(x)
        order = np.argsort(-x, kind="stable")[:K]          # (value desc, id asc)
        assert ke == min(K, V) and nf == 0 and pinf == 0
        assert tok.numpy().tolist() == order.tolist()
        np.testing.assert_allclose(lp.numpy(), ref_lp[order], rtol=0, atol=1e-12)
        assert m == x.max()
        np.testing.assert_allclose(a.numpy(), x[order] - x.max(), rtol=0, atol=0)
        np.testing.assert_allclose(lz, np.log(np.exp(x - x.max()).sum()), rtol=1e-13)


def test_softmax_topk_closed_forms():
    V, K = 513, 5
    row = torch.full((V,), 1.25, dtype=torch.bfloat16)      # uniform: lp = -ln V, ids 0..K-1
    m, lz, tok, a, lp, ke, *_ = O.row_softmax_topk(row, K)
    assert tok.tolist() == list(range(K))
    np.testing.assert_allclose(lp.numpy(), -math.log(V), rtol=1e-14)
    assert lz == pytest.approx(math.log(V), rel=1e-15)
    # one token at c, the rest at 0: p = e^c / (e^c + V - 1)
    c = 3.0
    row = torch.zeros(V, dtype=torch.float32)
    row[100] = c
    m, lz, tok, a, lp, ke, *_ = O.row_softmax_topk(row, K)
    assert tok.tolist() == [100, 0, 1, 2, 3]
    assert math.exp(lp[0]) == pytest.approx(math.exp(c) / (math.exp(c) + V - 1), rel=1e-13)
    assert math.exp(lp[1]) == pytest.approx(1.0 / (math.exp(c) + V - 1), rel=1e-13)


def test_softmax_topk_nonfinite():
    row = torch.tensor([0.0, float("nan"), -float("inf"), 1.0, 1.0], dtype=torch.float32)
    m, lz, tok, a, lp, ke, nf, pinf = O.row_softmax_topk(row, 4)
    assert ke == 3 and nf == 1 and pinf == 0
    assert tok.tolist() == [3, 4, 0, -1]
    assert lz == pytest.approx(math.log(2 + math.exp(-1.0)), rel=1e-15)
    row[2] = float("inf")
    *_, nf, pinf = O.row_softmax_topk(row, 4)
    assert nf == 1 and pinf == 1


def test_softmax_topk_lists_of_a_row_with_positive_infinity():
    """+Inf is invalid input: it is flagged and carries no mass, and the lists reported for the row are those of
    its finite logits alone — the library log-softmax of the finite sub-row, with the original token ids."""
    for dtype in (torch.float32, torch.bfloat16):
        row = torch.tensor([0.0, float("nan"), float("inf"), 1.0, 1.0, -float("inf"), 0.5, float("inf"), -2.0], dtype=dtype)
        m, lz, tok, a, lp, ke, nf, pinf = O.row_softmax_topk(row, 4)
        keep = np.array([0, 3, 4, 6, 8])                       # ids of the finite logits
        x = f64(row)[keep]
        order = np.argsort(-x, kind="stable")[:4]
        assert nf == 1 and pinf == 1 and ke == 4
        assert tok.tolist() == keep[order].tolist() == [3, 4, 6, 0]
        assert m == 1.0
        np.testing.assert_allclose(lp.numpy(), log_softmax(x)[order], rtol=0, atol=1e-15)
        np.testing.assert_allclose(a.numpy(), x[order] - 1.0, rtol=0, atol=0)
        assert lz == pytest.approx(math.log(2 + math.exp(-0.5) + math.exp(-1.0) + math.exp(-3.0)), rel=1e-15)
    # a request with such a row returns the empty tree, flagged, and still reports those lists
    x = torch.zeros(1, 2, 9)
    x[0, 0] = row.float()
    t = O.build_tree(x, K=4, B_max=8, cost_coef=quad_coef(1, 1.0, 1.0, 0.01, 0.0))
    assert int(t.n_nodes[0]) == 0 and int(t.status[0]) & O.ST_NONFINITE
    assert t.topk_token[0, 0].tolist() == [3, 4, 6, 0]
    assert t.topk_token[0, 1].tolist() == [0, 1, 2, 3]


# ---------------------------------------------------------------- hand-worked example
def _golden():
    d = {}
    for line in open(os.path.join(GOLDEN, "two_position_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        d[k] = [float(t) for t in v]
    return d


def test_hand_worked_example():
    g = _golden()
    logits = torch.tensor(np.log(np.array([[g["q1"], g["q2"]]])), dtype=torch.float32)
    coef = torch.tensor([g["cost"]], dtype=torch.float64)
    t = O.build_tree(logits, K=3, B_max=12, cost_coef=coef)
    n = int(g["n_star"][0])
    assert int(t.n_nodes[0]) == n
    assert t.token_ids[0, 1:n + 1].tolist() == [int(v) for v in g["tokens"]]
    assert t.parent_idx[0, 1:n + 1].tolist() == [int(v) for v in g["parents"]]
    assert t.depth[0, 1:n + 1].tolist() == [int(v) for v in g["depths"]]
    assert float(t.phi[0]) == pytest.approx(g["phi"][0], rel=1e-6)
    assert float(t.theta[0]) == pytest.approx(g["theta"][0], rel=1e-6)
    assert int(t.status[0]) == 0
    full = O.build_tree(logits, K=3, B_max=12, cost_coef=coef, flags=O.FLAG_FIXED_BUDGET)
    assert int(full.n_nodes[0]) == 12 and int(full.status[0]) & O.ST_FRONTIER_EXHAUSTED
    assert full.token_ids[0, 1:13].tolist() == [int(v) for v in g["full_order_tokens"]]
    assert full.parent_idx[0, 1:13].tolist() == [int(v) for v in g["full_order_parents"]]
    np.testing.assert_allclose(full.node_logprob[0, 1:13].exp().numpy(), g["full_order_prob"], rtol=1e-6)


# ---------------------------------------------------------------- the margins that gate parity exemptions
def test_exemption_margins_on_the_hand_worked_example():
    """pop_gap[j] = 1 - (best strictly smaller prefix probability in the heap) / (prefix probability of pop j),
    1 when the heap holds nothing smaller; stop_gap = |theta_new - theta_prev| / theta_prev at the test that
    stopped the loop.  On the two-position example every value is a rational worked out by hand from the heap
    contents (Algorithm 1: the heap holds the next sibling and the first child of what was popped)."""
    from fractions import Fraction as Fr
    g = _golden()
    logits = torch.tensor(np.log(np.array([[g["q1"], g["q2"]]])), dtype=torch.float32)
    coef = torch.tensor([g["cost"]], dtype=torch.float64)
    # heap when row j is popped (prefix probabilities), popped value first:
    #  1: {1/2}                       2: {1/3, 1/4}            3: {1/4, 1/12}          4: {1/4, 1/6, 1/12}
    #  5: {1/6, 1/6, 1/12}            6: {1/6, 1/12, 1/24}     7: {1/12, 1/24, 1/24}   8: {1/12, 1/24, 1/24}
    #  9..12: only 1/24 entries left
    # pops 5 and 6 tie exactly at 1/6 while both are in the heap: the margin is the one to 1/12, not 0
    want = [Fr(1), 1 - Fr(1, 4) / Fr(1, 3), 1 - Fr(1, 12) / Fr(1, 4), 1 - Fr(1, 6) / Fr(1, 4),
            1 - Fr(1, 12) / Fr(1, 6), 1 - Fr(1, 12) / Fr(1, 6), 1 - Fr(1, 24) / Fr(1, 12), 1 - Fr(1, 24) / Fr(1, 12),
            Fr(1), Fr(1), Fr(1), Fr(1)]
    assert [float(w) for w in want[:8]] == pytest.approx([1, 1 / 4, 2 / 3, 1 / 3, 1 / 2, 1 / 2, 1 / 2, 1 / 2])
    full = O.build_tree(logits, K=3, B_max=12, cost_coef=coef, flags=O.FLAG_FIXED_BUDGET)
    np.testing.assert_allclose(full.pop_gap[0, 1:13].numpy(), [float(w) for w in want], rtol=1e-5)
    assert float(full.pop_gap[0, 0]) == 1.0                                  # the root is not a pop
    stop = O.build_tree(logits, K=3, B_max=12, cost_coef=coef)
    np.testing.assert_allclose(stop.pop_gap[0, 1:5].numpy(), [float(w) for w in want[:4]], rtol=1e-5)
    assert bool((stop.pop_gap[0, 5:] == 1.0).all())                          # padding rows
    # the loop stopped on theta(5) = 10/13 <= theta(4) = 7/9
    assert float(stop.stop_gap[0]) == pytest.approx(float(abs(Fr(10, 13) - Fr(7, 9)) / Fr(7, 9)), rel=1e-4)
    assert float(abs(Fr(10, 13) - Fr(7, 9)) / Fr(7, 9)) == pytest.approx(1 / 91)
    # nothing stops a fixed-budget run: the smallest margin over the accepted nodes is reported
    probs = [Fr(1, 2), Fr(1, 3), Fr(1, 4), Fr(1, 4), Fr(1, 6), Fr(1, 6), Fr(1, 12), Fr(1, 12)] + [Fr(1, 24)] * 4
    theta, phi = [Fr(1, 2)], Fr(0)
    for n, pr in enumerate(probs, 1):
        phi += pr
        theta.append((1 + phi) / (2 + Fr(n, 4)))
    assert theta[4] == Fr(7, 9) and theta[5] == Fr(10, 13)
    smallest = min(abs(theta[n] - theta[n - 1]) / theta[n - 1] for n in range(1, 13))
    assert float(full.stop_gap[0]) == pytest.approx(float(smallest), rel=1e-4)


def frontier_margins(x_row_major, K, paths, scores):
    """Margins by the definition, from the pop order alone: when the j-th node is popped the heap holds exactly the
    unpopped nodes whose parent (a prefix) and whose previous sibling (same prefix, rank - 1) were popped before.
    Scores are library log-softmax sums; scores closer than 1e-12 count as equal."""
    L, V = x_row_major.shape
    lps, toks = [], []
    for i in range(L):
        lp = log_softmax(x_row_major[i])
        order = np.argsort(-x_row_major[i], kind="stable")[:K]
        lps.append(lp[order]); toks.append([int(t) for t in order])
    score = lambda path: sum(lps[i][toks[i].index(t)] for i, t in enumerate(path))
    popped, out = {()}, []
    for j, path in enumerate(paths):
        heap = []
        for pre in popped:                                       # children of popped nodes
            d = len(pre)
            if d == L:
                continue
            for r, t in enumerate(toks[d]):
                c = pre + (t,)
                if c in popped:
                    continue
                if r == 0 or pre + (toks[d][r - 1],) in popped:
                    heap.append(score(c))
        assert abs(max(heap) - scores[j]) < 1e-12                # the popped node is the heap's maximum
        smaller = [s for s in heap if s < scores[j] - 1e-12]
        out.append(1.0 - math.exp(max(smaller) - scores[j]) if smaller else 1.0)
        popped.add(path)
    return out


@pytest.mark.parametrize("K,L,V,seed,quant", [(2, 3, 5, 0, None), (3, 3, 6, 1, 2), (4, 3, 9, 2, 4), (2, 5, 4, 3, 1), (3, 2, 40, 4, None)])
def test_pop_gap_equals_runner_up_margin_by_definition(K, L, V, seed, quant):
    x = rand_logits(seed + 7, 1, L, V, quant=quant)
    B = sum(min(K, V) ** d for d in range(1, L + 1))
    t = O.build_tree(x, K, B_max=B, cost_coef=quad_coef(1, 1.0, 1.0, 0.0, 0.0), flags=O.FLAG_FIXED_BUDGET)
    assert int(t.n_nodes[0]) == B
    want = frontier_margins(f64(x[0]), K, tree_paths(t), t.node_logprob[0, 1:B + 1].numpy())
    got = t.pop_gap[0, 1:B + 1].numpy()
    np.testing.assert_allclose(got, want, rtol=1e-9, atol=1e-12)
    if quant:                                                    # quantised logits: exact ties occur and are skipped over
        sig = t.node_logprob[0, 1:B + 1].numpy()
        assert np.any(np.diff(sig) == 0.0) and np.all(got > 1e-3)


def test_margins_of_a_constructed_near_tie():
    """Depth-1 runner-up against the first child of the best token, 1e-9 apart in probability: the margin must come
    out as that 1e-9 (not 0, not the gap to some farther score), and an exact tie beside it must be skipped."""
    # position 2: p = softmax(0, -1, r); log p_0 moves by ~e^r per unit of r, so r near -20 tunes it in steps of
    # ~1e-15; position 1: tokens 0 and 1 differ by d = fp32(log p_0) (so the sibling ties the child up to rounding)
    d32 = np.float32(-math.log(1 + math.exp(-1.0)))
    best = None
    for r in np.arange(-21.0, -19.0, 1.0 / 1024, dtype=np.float32):
        lp0 = log_softmax(np.array([0.0, -1.0, float(r)]))[0]
        gap = 1.0 - math.exp(lp0 - float(d32)) if lp0 < float(d32) else None       # child just below the sibling
        if gap is not None and (best is None or abs(gap - 1e-9) < abs(best[1] - 1e-9)):
            best = (float(r), gap)
    r, gap = best
    assert 0.2e-9 < gap < 5e-9
    x = torch.tensor([[[0.0, float(d32), float(d32), -30.0], [0.0, -1.0, r, -40.0]]], dtype=torch.float32)
    t = O.build_tree(x, K=3, B_max=4, cost_coef=quad_coef(1, 1.0, 1.0, 0.0, 0.0), flags=O.FLAG_FIXED_BUDGET)
    # pops: token 0; then its sibling token 1 (depth 1) against the child (0, 0), 1e-9 below it
    assert t.token_ids[0, 1:4].tolist() == [0, 1, 2] and t.depth[0, 1:4].tolist() == [1, 1, 1]
    assert float(t.pop_gap[0, 2]) == pytest.approx(gap, rel=1e-5)
    # third pop: token 2 ties token 1 exactly (already popped, so not in the heap); the child (0, 0) is the nearest
    # distinct score and the margin is again the constructed one
    assert float(t.pop_gap[0, 3]) == pytest.approx(gap, rel=1e-5)
    # fourth pop: the child (0, 0) itself; below it are (1, 0) and (2, 0), which tie each other exactly at
    # p_1(1) p_2(0): margin 1 - p_1(1) / p_1(0) = 1 - e^d
    assert t.depth[0, 4].item() == 2 and t.parent_idx[0, 4].item() == 1
    assert float(t.pop_gap[0, 4]) == pytest.approx(1.0 - math.exp(float(d32)), rel=1e-9)


# ---------------------------------------------------------------- O3: pop order = plain definition
def enumerate_nodes(x_row_major, K):
    """All nodes of the K-ary depth-L candidate tree with their log prefix probability,
    straight from Eq. 5: the sum of library log-softmax values along the path."""
    L = x_row_major.shape[0]
    lps, toks = [], []
    for i in range(L):
        x = x_row_major[i]
        lp = log_softmax(x)
        order = np.argsort(-x, kind="stable")[:K]
        lps.append(lp[order]); toks.append(order)
    nodes = []           # (score, depth, path-of-tokens)
    for d in range(1, L + 1):
        for ranks in itertools.product(range(min(K, x_row_major.shape[1])), repeat=d):
            s = sum(lps[i][r] for i, r in enumerate(ranks))
            nodes.append((s, d, tuple(int(toks[i][r]) for i, r in enumerate(ranks))))
    return nodes


def tree_paths(t, b=0):
    n = int(t.n_nodes[b])
    paths = [()]
    for j in range(1, n + 1):
        p = int(t.parent_idx[b, j])
        assert 0 <= p < j
        paths.append(paths[p] + (int(t.token_ids[b, j]),))
    return paths[1:]


@pytest.mark.parametrize("K,L,V,seed", [(2, 3, 5, 0), (3, 3, 6, 1), (4, 4, 9, 2), (2, 6, 4, 3), (5, 2, 40, 4)])
def test_pop_order_equals_sorted_enumeration(K, L, V, seed):
    x = rand_logits(seed, 1, L, V)
    nodes = enumerate_nodes(f64(x[0]), K)
    nodes.sort(key=lambda t: (-t[0], t[1], t[2][-1]))
    B = len(nodes)
    t = O.build_tree(x, K, B_max=B, cost_coef=quad_coef(1, 1.0, 1.0, 0.0, 0.0), flags=O.FLAG_FIXED_BUDGET)
    assert int(t.n_nodes[0]) == B
    assert tree_paths(t) == [nd[2] for nd in nodes]
    np.testing.assert_allclose(t.node_logprob[0, 1:B + 1].numpy(), [nd[0] for nd in nodes], rtol=0, atol=1e-12)
    # Eq. 6: Phi*(n) is the prefix sum of the sorted prefix probabilities
    assert float(t.phi[0]) == pytest.approx(sum(math.exp(nd[0]) for nd in nodes), rel=1e-12)


def test_pop_order_config1_top_nodes():
    """Config-1 shape (K=4, L=8: 87380 candidate nodes): the first 32 pops are the 32 best nodes."""
    from paper_2606_01813_b200 import synth
    cfg = synth.CONFIGS["c1"]
    d = synth.make_draft_inputs(cfg, 0)
    x = f64(d.logits[0])
    K, L = cfg.K, cfg.L
    lps, toks = [], []
    for i in range(L):
        lp = log_softmax(x[i]); order = np.argsort(-x[i], kind="stable")[:K]
        lps.append(lp[order]); toks.append(order)
    all_scores, all_depth = [], []
    prev = np.zeros(1)
    for i in range(L):                                   # vectorised enumeration, depth by depth
        prev = (prev[:, None] + lps[i][None, :]).reshape(-1)
        all_scores.append(prev); all_depth.append(np.full(prev.shape, i + 1))
    scores = np.concatenate(all_scores)
    assert scores.size == sum(K ** d for d in range(1, L + 1)) == 87380
    top = np.sort(scores)[::-1][:cfg.B_max]
    t = O.build_tree(d.logits, K, cfg.B_max, cost_coef=quad_coef(1, 1.0, 1.0, 0.0, 0.0), flags=O.FLAG_FIXED_BUDGET)
    assert int(t.n_nodes[0]) == cfg.B_max and int(t.status[0]) & O.ST_CAP_HIT
    np.testing.assert_allclose(t.node_logprob[0, 1:].numpy(), top, rtol=0, atol=1e-12)


# ---------------------------------------------------------------- Prop. 1: brute force over all valid trees
def all_tree_size_phi(lp, K, L):
    """(size, Phi) of every prefix-closed tree of the full K-ary depth-L candidate tree.
    lp[i][k] = log q_{i+1} of the k-th candidate at position i+1."""
    def below(depth, logpi):
        # options for the forest below a node at `depth` with log prefix prob `logpi`
        if depth == L:
            return np.zeros(1, dtype=np.int64), np.zeros(1)
        sizes, phis = np.zeros(1, dtype=np.int64), np.zeros(1)
        for k in range(K):
            child = logpi + lp[depth][k]
            s_sub, p_sub = below(depth + 1, child)
            s_opt = np.concatenate([[0], 1 + s_sub])                 # child absent | present + subtree
            p_opt = np.concatenate([[0.0], math.exp(child) + p_sub])
            sizes = (sizes[:, None] + s_opt[None, :]).reshape(-1)
            phis = (phis[:, None] + p_opt[None, :]).reshape(-1)
        return sizes, phis
    return below(0, 0.0)


@pytest.mark.parametrize("K,L,count", [(2, 2, 25), (2, 3, 676), (3, 2, 729), (4, 2, 83521), (2, 4, 458329)])
def test_brute_force_all_prefix_closed_trees(K, L, count):
    for seed in range(2):
        x = rand_logits(100 * K + 10 * L + seed, 1, L, K, scale=1.5)       # V = K: every token is a candidate
        xs = f64(x[0])
        lp = [np.sort(log_softmax(xs[i]))[::-1] for i in range(L)]
        sizes, phis = all_tree_size_phi(lp, K, L)
        assert sizes.size == count
        n_all = sum(K ** d for d in range(1, L + 1))
        t_d, a, b, c = 0.7, 1.0, 0.15, 0.02
        coef = quad_coef(1, t_d, a, b, c)
        full = O.build_tree(x, K, B_max=n_all, cost_coef=coef, flags=O.FLAG_FIXED_BUDGET)
        delta = np.exp(full.node_logprob[0, 1:n_all + 1].numpy())
        phistar = np.concatenate([[0.0], np.cumsum(delta)])
        for n in range(n_all + 1):                                          # Eq. 6 / Prop. 1, first part
            assert phis[sizes == n].max() == pytest.approx(phistar[n], rel=1e-12, abs=1e-15)
        cost = t_d + a + b * sizes + c * sizes.astype(np.float64) ** 2
        theta_all = (1.0 + phis) / cost
        t = O.build_tree(x, K, B_max=n_all, cost_coef=coef)
        assert float(t.theta[0]) == pytest.approx(theta_all.max(), rel=1e-12)   # Prop. 1, Eq. (decomposition)
        assert float(t.phi[0]) == pytest.approx(phistar[int(t.n_nodes[0])], rel=1e-12)
        best_sizes = sizes[theta_all >= theta_all.max() * (1 - 1e-13)]
        assert int(t.n_nodes[0]) == best_sizes.min()


# ---------------------------------------------------------------- stopping rule invariants
def cost_fn(coef, n):
    n = np.asarray(n, dtype=np.float64)
    return coef[1] + coef[2] * n + coef[3] * n * n


@pytest.mark.parametrize("seed", range(6))
def test_invariants_lemma1_unimodal_greedy(seed):
    rng = np.random.default_rng(seed)
    batch, L, V, K, B = 3, int(rng.integers(2, 7)), int(rng.integers(20, 400)), int(rng.integers(2, 6)), 120
    x = rand_logits(seed + 50, batch, L, V, dtype=torch.bfloat16 if seed % 2 else torch.float32,
                    scale=float(rng.uniform(1, 4)))
    coefs = torch.tensor([[rng.uniform(0.1, 1), rng.uniform(0.2, 2), rng.uniform(1e-3, 5e-2), rng.uniform(0, 1e-3)]
                          for _ in range(batch)], dtype=torch.float64)
    full = O.build_tree(x, K, B, cost_coef=coefs, flags=O.FLAG_FIXED_BUDGET)
    stop = O.build_tree(x, K, B, cost_coef=coefs)
    for b in range(batch):
        N = int(full.n_nodes[b]); cf = coefs[b].numpy(); C_d = cf[0]
        sig = full.node_logprob[b, 1:N + 1].numpy()
        delta = np.exp(sig)
        assert np.all(np.diff(sig) <= 0)                                   # delta_n non-increasing
        phi = np.concatenate([[0.0], np.cumsum(delta)])
        assert np.all(np.diff(phi) >= 0)                                   # Phi* non-decreasing
        n = np.arange(N + 1)
        theta = (1.0 + phi) / (C_d + cost_fn(cf, n))                       # Eq. 7 / Prop. 1
        np.testing.assert_allclose(full.theta_curve[b, :N + 1].numpy(), theta, rtol=1e-13)
        c = np.diff(cost_fn(cf, n))                                        # marginal costs c_1..c_N
        rho = delta / c
        assert np.all(np.diff(rho) <= 1e-15 * rho[:-1])                    # Cor. 2: convex cost => Assumption 1
        w = (C_d + cost_fn(cf, n[:-1])) / (C_d + cost_fn(cf, n[1:]))
        np.testing.assert_allclose(theta[1:], w * theta[:-1] + (1 - w) * rho, rtol=1e-12)   # Lemma 1, Eq. 10
        rises = theta[1:] > theta[:-1]
        differs = rises != (rho > theta[:-1])                              # Eq. 11, up to rounding at equality
        assert np.all(np.abs(rho - theta[:-1])[differs] < 1e-12)
        first_fail = int(np.argmin(rises)) if not rises.all() else N       # Thm 1: unimodal
        assert not rises[first_fail:].any()
        n_star = int(stop.n_nodes[b])
        assert n_star == first_fail == int(np.argmax(theta))               # Cor. 1: smallest global maximiser
        assert float(stop.theta[b]) == pytest.approx(theta.max(), rel=1e-13)
        assert float(stop.phi[b]) == pytest.approx(phi[n_star], rel=1e-13)
        # the stopped tree is the prefix of the full expansion
        assert torch.equal(stop.token_ids[b, :n_star + 1], full.token_ids[b, :n_star + 1])
        assert torch.equal(stop.parent_idx[b, :n_star + 1], full.parent_idx[b, :n_star + 1])
        if n_star < B:
            assert int(stop.token_ids[b, n_star + 1:].max()) == -1      # padding rows


def test_table_cost_equals_quadratic_and_step_table():
    from paper_2606_01813_b200 import synth
    x = rand_logits(7, 2, 5, 300, dtype=torch.bfloat16, scale=3.0)
    B = 64
    n = torch.arange(B + 1, dtype=torch.float64)
    table = (0.9 + 0.01 * n + 0.0004 * n * n)[None, :]
    tq = O.build_tree(x, 4, B, cost_coef=quad_coef(2, 0.3, 0.9, 0.01, 0.0004))
    tt = O.build_tree(x, 4, B, cost_kind=O.COST_TABLE, cost_table=table, table_idx=torch.zeros(2, dtype=torch.int32),
                      t_draft=torch.full((2,), 0.3, dtype=torch.float64))
    assert torch.equal(tq.n_nodes, tt.n_nodes) and torch.equal(tq.token_ids, tt.token_ids)
    np.testing.assert_allclose(tq.theta.numpy(), tt.theta.numpy(), rtol=1e-14)
    tab = synth.convex_step_table((1.0, 0.0015, 0.00001), 256, 0.5, 512).numpy()
    assert np.all(np.diff(tab, 2) >= -1e-12) and np.all(np.diff(tab) > 0)          # convex, increasing
    c0 = 1.0 + 0.0015 * np.arange(513) + 0.00001 * np.arange(513) ** 2
    np.testing.assert_allclose(tab[256:], c0[256:] + 0.5, rtol=1e-15)
    np.testing.assert_allclose(tab[:33], c0[:33], rtol=1e-15)                       # quadratic wins for B <= 32
    assert tab[33] > c0[33]
    assert tab[100] == pytest.approx(2.53936 + 0.00662 * (100 - 256), rel=1e-12)


def test_constant_cost_expands_to_cap_and_larger_cost_smaller_budget():
    x = rand_logits(11, 4, 6, 200, scale=3.0)
    t = O.build_tree(x, 4, 50, cost_coef=quad_coef(4, 1.0, 2.0, 0.0, 0.0))        # constant-cost ablation
    assert t.n_nodes.tolist() == [50] * 4 and all(int(s) & O.ST_CAP_HIT for s in t.status)
    prev = None
    for scale in (0.25, 0.5, 1.0, 2.0, 4.0):                                       # costlier nodes => smaller trees
        n = O.build_tree(x, 4, 50, cost_coef=quad_coef(4, 1.0, 1.0, 0.02 * scale, 0.001 * scale)).n_nodes
        if prev is not None:
            assert torch.all(n <= prev)
        prev = n
    t = O.build_tree(x, 4, 50, cost_coef=quad_coef(4, 1.0, 1.0, 1e6, 0.0))        # huge marginal cost
    assert t.n_nodes.tolist() == [0] * 4
    assert t.theta.tolist() == pytest.approx([0.5] * 4)


def test_closed_forms_chain_onehot_uniform():
    L, V = 6, 50
    x = rand_logits(3, 1, L, V, scale=2.0)
    t = O.build_tree(x, 1, 40, cost_coef=quad_coef(1, 1.0, 1.0, 0.0, 0.0))        # K = 1: a chain
    assert int(t.n_nodes[0]) == L and int(t.status[0]) & O.ST_FRONTIER_EXHAUSTED
    lp = [log_softmax(f64(x[0, i])).max() for i in range(L)]
    np.testing.assert_allclose(t.node_logprob[0, 1:L + 1].numpy(), np.cumsum(lp), atol=1e-12)
    assert t.parent_idx[0, 1:L + 1].tolist() == list(range(L))
    assert t.token_ids[0, 1:L + 1].tolist() == [int(np.argmax(f64(x[0, i]))) for i in range(L)]
    # near-one-hot marginals: theta(n) = (1+n)/(C_d+C_v(n)) for n <= L, rank-1 chain
    x = torch.zeros(1, L, V); toks = [3, 7, 1, 0, 49, 20]
    for i, tk in enumerate(toks):
        x[0, i, tk] = 60.0
    coef = quad_coef(1, 1.0, 1.0, 0.05, 0.0)
    t = O.build_tree(x, 3, 40, cost_coef=coef)
    assert int(t.n_nodes[0]) == L and t.token_ids[0, 1:L + 1].tolist() == toks
    assert float(t.theta[0]) == pytest.approx((1 + L) / (2.0 + 0.05 * L), rel=1e-12)
    # uniform logits: order fixed purely by the tie-break
    x = torch.zeros(1, 2, 5)
    t = O.build_tree(x, 3, 12, cost_coef=coef, flags=O.FLAG_FIXED_BUDGET)
    assert t.token_ids[0, 1:13].tolist() == [0, 1, 2, 0, 0, 0, 1, 1, 1, 2, 2, 2]
    assert t.parent_idx[0, 1:13].tolist() == [0, 0, 0, 1, 2, 3, 1, 2, 3, 1, 2, 3]
    np.testing.assert_allclose(t.node_logprob[0, 1:4].numpy(), -math.log(5), rtol=1e-15)
    np.testing.assert_allclose(t.node_logprob[0, 4:13].numpy(), -2 * math.log(5), rtol=1e-15)


# ---------------------------------------------------------------- O4: arrays and mask
def check_tree_structure(t, b, K=None):
    n = int(t.n_nodes[b]); R = t.token_ids.shape[1]
    par, dep, tok = t.parent_idx[b].tolist(), t.depth[b].tolist(), t.token_ids[b].tolist()
    assert par[0] == -1 and dep[0] == 0
    mask = t.mask_bits[b].numpy().view(np.uint32)
    bits = lambda j: {c for c in range(R) if (int(mask[j, c >> 5]) >> (c & 31)) & 1}
    assert bits(0) == {0}
    seen = set()
    for j in range(1, n + 1):
        assert 0 <= par[j] < j and dep[j] == dep[par[j]] + 1
        assert bits(j) == bits(par[j]) | {j} and len(bits(j)) == dep[j] + 1
        assert (par[j], tok[j]) not in seen                # siblings carry distinct tokens
        seen.add((par[j], tok[j]))
    for j in range(n + 1, R):
        assert tok[j] == -1 and par[j] == -1 and dep[j] == 0 and not bits(j)


def test_tree_arrays_and_mask():
    x = rand_logits(21, 3, 5, 120, dtype=torch.bfloat16, scale=3.0, quant=4)
    ctx = torch.tensor([5, 0, 1000], dtype=torch.int32); bonus = torch.tensor([9, 8, 7], dtype=torch.int32)
    t = O.build_tree(x, 4, 70, R=75, cost_coef=quad_coef(3, 0.3, 1.0, 0.002, 0.00002), bonus_token=bonus,
                     ctx_len=ctx, dense_mask=True)
    for b in range(3):
        check_tree_structure(t, b)
        n = int(t.n_nodes[b])
        assert t.token_ids[b, 0] == bonus[b]
        assert torch.equal(t.position_ids[b, :n + 1], ctx[b] + t.depth[b, :n + 1])
        dense = t.mask_dense[b].numpy(); mask = t.mask_bits[b].numpy().view(np.uint32)
        for j in range(75):
            for c in range(75):
                assert dense[j, c] == (int(mask[j, c >> 5]) >> (c & 31)) & 1


# ---------------------------------------------------------------- O5 / O6: verification
def test_argmax_matches_numpy_first_occurrence():
    g = torch.Generator().manual_seed(5)
    for dtype in (torch.float32, torch.bfloat16):
        for V in (1, 9, 1000, 151936):
            row = torch.randn(V, generator=g).to(dtype)
            assert O.row_argmax(row) == int(np.argmax(f64(row)))
    row = torch.tensor([1.0, 3.0, float("nan"), 3.0, -1.0])
    assert O.row_argmax(row) == 1
    row = torch.tensor([float("nan"), -float("inf")])
    assert O.row_argmax(row) == 0


def brute_force_accept(n, tok, par, g):
    """Mark every node whose whole root path matches the target's argmax at each parent."""
    ok = {0}
    depth = {0: 0}
    for j in range(1, n + 1):
        depth[j] = depth[par[j]] + 1
        if par[j] in ok and tok[j] == g[par[j]]:
            ok.add(j)
    best = max(ok, key=lambda j: depth[j])
    path = []
    j = best
    while j != 0:
        path.append(j); j = par[j]
    return depth[best], path[::-1], g[best]


@pytest.mark.parametrize("seed", range(4))
def test_walk_matches_brute_force(seed):
    batch, L, V, K = 4, 5, 12, 3
    x = rand_logits(seed, batch, L, V, scale=1.0)
    t = O.build_tree(x, K, 40, cost_coef=quad_coef(batch, 1.0, 1.0, 0.0, 0.0), flags=O.FLAG_FIXED_BUDGET)
    g = torch.Generator().manual_seed(seed + 99)
    y = torch.randn(batch, 41, V, generator=g)
    for b in range(batch):                      # make the target agree with the drafter's best token often
        for j in range(41):
            d = int(t.depth[b, j])
            if d < L and torch.rand(1, generator=g).item() < 0.7:
                y[b, j, int(torch.argmax(x[b, d]))] += 6.0
    for mode in (O.ROWS_LIVE, O.ROWS_DENSE):
        v = O.verify_tree(y, L, t.n_nodes, t.token_ids, t.parent_idx, rows_mode=mode)
        for b in range(batch):
            n = int(t.n_nodes[b])
            gm = np.argmax(f64(y[b]), axis=1)
            rows = n + 1 if mode == O.ROWS_LIVE else 41
            assert v.node_argmax[b, :rows].tolist() == gm[:rows].tolist()
            assert (v.node_argmax[b, rows:] == -1).all()
            alpha, path, nb = brute_force_accept(n, t.token_ids[b].tolist(), t.parent_idx[b].tolist(), gm.tolist())
            assert int(v.accepted_len[b]) == alpha
            assert v.accepted_nodes[b, :alpha].tolist() == path and (v.accepted_nodes[b, alpha:] == -1).all()
            assert int(v.next_bonus[b]) == nb
    assert int(v.accepted_len.max()) >= 2       # the case is not trivial


# ---------------------------------------------------------------- edge cases and status flags
def test_edge_cases_and_status():
    x = rand_logits(1, 3, 4, 30, scale=2.0)
    coef = quad_coef(3, 1.0, 1.0, 0.01, 0.0)
    t = O.build_tree(x, 4, 0, cost_coef=coef)                                   # B_max = 0
    assert t.n_nodes.tolist() == [0, 0, 0] and all(int(s) & O.ST_CAP_HIT for s in t.status)
    t = O.build_tree(x, 4, 20, cost_coef=coef, l_eff=torch.tensor([0, 2, 9], dtype=torch.int32))
    assert int(t.n_nodes[0]) == 0 and int(t.depth[1].max()) <= 2
    assert int(t.status[2]) & O.ST_L_EFF_CLAMPED and not int(t.status[1]) & O.ST_L_EFF_CLAMPED
    x2 = x.clone(); x2[0, 1, 5] = float("inf"); x2[1, 0, 3] = float("nan"); x2[2, 1, :] = -float("inf")
    t = O.build_tree(x2, 4, 20, cost_coef=coef, flags=O.FLAG_FIXED_BUDGET)
    assert int(t.n_nodes[0]) == 0 and int(t.status[0]) & O.ST_NONFINITE          # +Inf: empty tree
    assert int(t.n_nodes[1]) == 20 and int(t.status[1]) & O.ST_NONFINITE         # NaN: ordered as -Inf
    assert 3 not in t.token_ids[1, t.depth[1] == 1].tolist()
    assert int(t.depth[2].max()) == 1 and int(t.status[2]) & O.ST_FEWER_THAN_K   # position 2 has no finite logit
    assert int(t.n_nodes[2]) == 4 and int(t.status[2]) & O.ST_FRONTIER_EXHAUSTED
    t = O.build_tree(x, 4, 20, cost_coef=quad_coef(3, -2.0, 1.0, 0.01, 0.0))
    assert t.n_nodes.tolist() == [0, 0, 0] and all(int(s) & O.ST_COST_NONPOSITIVE for s in t.status)
    xs = rand_logits(2, 1, 2, 3)                                                 # K > V
    t = O.build_tree(xs, 5, 20, cost_coef=quad_coef(1, 1.0, 1.0, 0.0, 0.0), flags=O.FLAG_FIXED_BUDGET)
    assert int(t.n_nodes[0]) == 12 and int(t.status[0]) & O.ST_FEWER_THAN_K
    with pytest.raises(ValueError):
        O.build_tree(x, 4, 20, R=20, cost_coef=coef)                             # R < B_max + 1
    # a table index that names no table: flagged, empty tree, the other requests as with a valid index
    n = torch.arange(21, dtype=torch.float64)
    table = torch.stack([1.0 + 0.01 * n, 1.0 + 0.2 * n])
    td = torch.full((3,), 1.0, dtype=torch.float64)
    t = O.build_tree(x, 4, 20, cost_kind=O.COST_TABLE, cost_table=table, t_draft=td,
                     table_idx=torch.tensor([2, 0, -1], dtype=torch.int32))
    assert [bool(int(v) & O.ST_BAD_TABLE_IDX) for v in t.status] == [True, False, True]
    assert int(t.n_nodes[0]) == 0 == int(t.n_nodes[2]) and int(t.token_ids[0, 1:].max()) == -1
    ref = O.build_tree(x, 4, 20, cost_coef=coef)                                 # table 0 is that quadratic
    assert int(t.n_nodes[1]) == int(ref.n_nodes[1]) > 0 and torch.equal(t.token_ids[1], ref.token_ids[1])


def test_cross_depth_exact_tie_prefers_lower_depth():
    """q_1 = (1/2, 1/2), q_2 = (1, 0): all four nodes have prefix probability exactly 1/2, so the
    order is fixed by the tie-break alone: both depth-1 nodes (token order) before the depth-2 ones
    (same token, lower parent row first)."""
    ninf = -float("inf")
    x = torch.tensor([[[0.0, 0.0, ninf], [ninf, 2.0, ninf]]])
    t = O.build_tree(x, 2, 8, cost_coef=quad_coef(1, 1.0, 1.0, 0.0, 0.0), flags=O.FLAG_FIXED_BUDGET)
    assert int(t.n_nodes[0]) == 4
    assert t.depth[0, 1:5].tolist() == [1, 1, 2, 2]
    assert t.token_ids[0, 1:5].tolist() == [0, 1, 1, 1]
    assert t.parent_idx[0, 1:5].tolist() == [0, 0, 1, 2]
    np.testing.assert_allclose(t.node_logprob[0, 1:5].numpy(), math.log(0.5), rtol=1e-15)


# ---------------- context interpolation of the cost tables (Eq. 13) ----------------
def test_context_interpolated_cost():
    from paper_2606_01813_b200 import synth
    B = 96
    tables, grid = synth.make_context_cost_tables(B)
    assert np.all(np.diff(tables.numpy(), 2, axis=1) >= -1e-12) and np.all(np.diff(tables.numpy(), axis=1) > 0)
    x = rand_logits(31, 6, 5, 400, dtype=torch.bfloat16, scale=3.0)
    td = torch.full((6,), 0.3, dtype=torch.float64)
    kw = dict(cost_kind=O.COST_TABLE_INTERP, cost_table=tables, ctx_grid=grid, t_draft=td)
    # on a grid point, below and above the profiled range: exactly one table
    ctx = torch.tensor([0, 2048, 8192, 20000, 3072, 1024], dtype=torch.int32)
    ti = O.build_tree(x, 4, B, ctx_len=ctx, **kw)
    tt = O.build_tree(x, 4, B, ctx_len=ctx, cost_kind=O.COST_TABLE, cost_table=tables, t_draft=td,
                      table_idx=torch.tensor([0, 2, 8, 8, 3, 1], dtype=torch.int32))
    assert torch.equal(ti.n_nodes, tt.n_nodes) and torch.equal(ti.token_ids, tt.token_ids)
    np.testing.assert_allclose(ti.theta.numpy(), tt.theta.numpy(), rtol=1e-15)
    # between two grid points: the blend is itself a table; it stays convex and increasing (the remark after Eq. 13)
    ctx = torch.tensor([512, 1536, 2300, 5000, 7000, 8191], dtype=torch.int32)
    blended = []
    for l in ctx.tolist():
        j = max(k for k in range(len(grid)) if int(grid[k]) <= l)
        alpha = (l - int(grid[j])) / (int(grid[j + 1]) - int(grid[j]))
        assert 0.0 <= alpha < 1.0
        blended.append((1 - alpha) * tables[j] + alpha * tables[j + 1])
    blended = torch.stack(blended)
    assert np.all(np.diff(blended.numpy(), 2, axis=1) >= -1e-12) and np.all(np.diff(blended.numpy(), axis=1) > 0)
    ti = O.build_tree(x, 4, B, ctx_len=ctx, **kw)
    tt = O.build_tree(x, 4, B, ctx_len=ctx, cost_kind=O.COST_TABLE, cost_table=blended, t_draft=td,
                      table_idx=torch.arange(6, dtype=torch.int32))
    assert torch.equal(ti.n_nodes, tt.n_nodes) and torch.equal(ti.token_ids, tt.token_ids)
    np.testing.assert_allclose(ti.theta.numpy(), tt.theta.numpy(), rtol=1e-14)
    # a longer context costs more per node, so the chosen budget cannot grow (Section 5.3, third observation)
    same = x[:1].expand(9, -1, -1).contiguous()
    sweep = O.build_tree(same, 4, B, ctx_len=torch.tensor([0, 700, 1500, 2600, 4000, 5500, 6100, 7900, 9000], dtype=torch.int32),
                         cost_kind=O.COST_TABLE_INTERP, cost_table=tables, ctx_grid=grid, t_draft=torch.full((9,), 0.3, dtype=torch.float64))
    assert np.all(np.diff(sweep.n_nodes.numpy()) <= 0) and np.all(np.diff(sweep.theta.numpy()) < 0)


# ---- logits from hidden states and the output projection (Section 3.1) ----

def test_head_logits_against_library_matmul_and_loops():
    g = torch.Generator().manual_seed(3)
    h = torch.randn(2, 3, 24, generator=g).bfloat16()
    w = torch.randn(7, 24, generator=g).bfloat16()
    y = O.head_logits(h, w)
    ref = torch.einsum("brk,vk->brv", h.double(), w.double())              # library contraction
    assert torch.allclose(y, ref, rtol=1e-14, atol=1e-14)
    for (b, r, v) in [(0, 0, 0), (1, 2, 6), (0, 1, 3)]:                      # plain loops
        acc = 0.0
        for k in range(24):
            acc += float(h[b, r, k]) * float(w[v, k])
        assert abs(float(y[b, r, v]) - acc) < 1e-12


def test_head_logits_closed_forms():
    hidden, V = 16, 5
    w = (torch.arange(V * hidden, dtype=torch.float32).reshape(V, hidden) % 7 - 3).bfloat16()
    h = torch.zeros(1, hidden, hidden)
    h[0] = torch.eye(hidden)                                                # row j selects column j of W
    y = O.head_logits(h.bfloat16(), w)
    assert torch.equal(y[0], w.double().T)
    # a transposed operand or a wrong stride would fail here: W rows are not symmetric
    h2 = torch.ones(1, 1, hidden).bfloat16()
    assert torch.equal(O.head_logits(h2, w)[0, 0], w.double().sum(dim=1))


def test_fused_head_verdict_on_a_hand_made_tree():
    # root (token 9) with children tokens 1 and 2; node 1 has child token 3.  W = identity rows scaled, so the
    # argmax at a node is the index of the largest coordinate of its hidden state.
    V = hidden = 8
    w = torch.eye(V).bfloat16()
    n_nodes = torch.tensor([3], dtype=torch.int32)
    token_ids = torch.tensor([[9, 1, 2, 3, -1]], dtype=torch.int32)
    parent_idx = torch.tensor([[-1, 0, 0, 1, -1]], dtype=torch.int32)
    h = torch.zeros(1, 5, hidden)
    h[0, 0, 1] = 2.0      # root predicts token 1 -> accept node 1
    h[0, 1, 3] = 1.0      # node 1 predicts token 3 -> accept node 3
    h[0, 3, 5] = 1.0      # node 3 predicts token 5 -> no such child: stop, bonus 5
    h[0, 2, 2] = 1.0
    h[0, 1, 6] = 1.0      # tie at node 1 between tokens 3 and 6: the lower id wins
    ov, y64 = O.verify_tree_fused_head(h.bfloat16(), w, 4, n_nodes, token_ids, parent_idx, rows_mode=O.ROWS_LIVE)
    assert ov.node_argmax[0].tolist() == [1, 3, 2, 5, -1]
    assert int(ov.accepted_len[0]) == 2 and ov.accepted_nodes[0].tolist() == [1, 3, -1, -1] and int(ov.next_bonus[0]) == 5


# ---- offline cost fitting: convex, non-decreasing least squares (Eq. 12) ----

def _kkt_violation(y, f):
    """Optimality of f over the cone of convex non-decreasing sequences, checked from the definition with plain
    numpy: feasibility; residual orthogonal to constants; <r, hinge_k> <= 0 for every hinge max(0, i - k), with
    equality wherever the fit actually bends (or rises, for k = 0)."""
    import numpy as np
    y, f = np.asarray(y, dtype=np.float64), np.asarray(f, dtype=np.float64)
    N = len(y)
    scale = max(1.0, float(np.abs(y).max()))
    r = y - f
    slopes = np.diff(f)
    bends = np.concatenate([slopes[:1], np.diff(slopes)])          # beta_k, k = 0..N-2
    worst = max(0.0, float(-bends.min()) / scale) if N > 1 else 0.0   # feasibility
    worst = max(worst, abs(float(r.sum())) / (scale * N))
    i = np.arange(N)
    for k in range(N - 1):
        g = float((np.maximum(0, i - k) * r).sum()) / (scale * N * N)
        worst = max(worst, g)                                       # dual feasibility
        if bends[k] > 1e-9 * scale:
            worst = max(worst, abs(g))                              # complementary slackness
    return worst


def test_convex_fit_satisfies_kkt_on_noisy_data():
    g = torch.Generator().manual_seed(8)
    n = torch.arange(200, dtype=torch.float64)
    clean = torch.stack([2.0 + 0.01 * n + 2e-4 * n * n, 5.0 + 0.03 * n + torch.clamp(n - 120, min=0) * 0.2])
    y = clean + 0.3 * torch.randn(2, 200, generator=g, dtype=torch.float64)
    f = O.fit_convex_nondecreasing(y)
    for t in range(2):
        assert _kkt_violation(y[t].numpy(), f[t].numpy()) < 1e-8
        assert float(((f[t] - clean[t]) ** 2).mean()) < float(((y[t] - clean[t]) ** 2).mean())   # it denoises


def test_convex_fit_closed_forms():
    n = torch.arange(50, dtype=torch.float64)
    convex = 1.0 + 0.5 * n + 0.02 * n * n
    assert torch.allclose(O.fit_convex_nondecreasing(convex[None])[0], convex, rtol=0, atol=1e-9)   # exact recovery
    falling = 10.0 - 0.3 * n
    assert torch.allclose(O.fit_convex_nondecreasing(falling[None])[0], torch.full_like(n, float(falling.mean())), atol=1e-9)
    concave = torch.sqrt(n + 1.0)                                    # best convex fit of a concave rise: its regression line
    X = torch.stack([torch.ones_like(n), n], dim=1)
    line = X @ torch.linalg.lstsq(X, concave[:, None]).solution[:, 0]
    assert torch.allclose(O.fit_convex_nondecreasing(concave[None])[0], line, atol=1e-9)


def test_convex_fit_brute_force_over_active_sets():
    """N = 6: the solution is the feasible least-squares fit with the smallest error over all 2^5 choices of which
    hinges may be non-zero."""
    import itertools
    import numpy as np
    rng = np.random.default_rng(4)
    N = 6
    i = np.arange(N, dtype=np.float64)
    for trial in range(20):
        y = np.cumsum(rng.normal(0.3, 1.0, N))
        best, best_f = None, None
        for mask in itertools.product([0, 1], repeat=N - 1):
            cols = [np.ones(N)] + [np.maximum(0, i - k) for k in range(N - 1) if mask[k]]
            A = np.stack(cols, axis=1)
            coef = np.linalg.lstsq(A, y, rcond=None)[0]
            if (coef[1:] < -1e-12).any():
                continue
            f = A @ coef
            sse = float(((y - f) ** 2).sum())
            if best is None or sse < best - 1e-12:
                best, best_f = sse, f
        f = O.fit_convex_nondecreasing(torch.from_numpy(y)[None])[0].numpy()
        assert abs(float(((y - f) ** 2).sum()) - best) < 1e-9 and np.allclose(f, best_f, atol=1e-7)


# ---------------------------------------------------------------------------------------------------------
# Sampling-mode verification: the inverse-CDF draw and the walk with drawn tokens
# ---------------------------------------------------------------------------------------------------------
def test_row_sample_closed_forms():
    # all logits equal: the CDF is (v+1)/V, so the draw is floor(u * V)
    for V in (1, 2, 10, 1000):
        row = torch.full((V,), 1.25, dtype=torch.float32)
        for u in (0.0, 0.049, 0.31, 0.5 + 1e-9, 0.999999):
            assert O.row_sample(row, u)[0] == int(math.floor(u * V))
    # two tokens with probabilities 1/4 and 3/4 at T = 1 ...
    row = torch.tensor([0.0, math.log(3.0)], dtype=torch.float64)
    assert [O.row_sample(row, u)[0] for u in (0.0, 0.2499, 0.2501, 0.99)] == [0, 0, 1, 1]
    # ... and the same probabilities from logits twice as far apart at T = 2
    row2 = torch.tensor([0.0, 2.0 * math.log(3.0)], dtype=torch.float64)
    assert [O.row_sample(row2, u, 2.0)[0] for u in (0.0, 0.2499, 0.2501, 0.99)] == [0, 0, 1, 1]
    # one token holds all the mass; a tiny temperature turns the draw into the arg-max
    row = torch.zeros(50, dtype=torch.float32)
    row[37] = 2000.0                                   # exp(-2000) underflows: the others carry no mass at all
    assert all(O.row_sample(row, u)[0] == 37 for u in (0.0, 0.5, 0.999999999))
    g = torch.Generator().manual_seed(4)
    y = torch.randn(300, generator=g, dtype=torch.float64)
    assert all(O.row_sample(y, u, 1e-4)[0] == int(y.argmax()) for u in (0.0, 0.3, 0.999))
    # values without mass are never drawn; a row with nothing finite gives token 0
    row = torch.tensor([float("-inf"), float("nan"), 0.0, float("inf"), 0.0], dtype=torch.float32)
    assert [O.row_sample(row, u)[0] for u in (0.0, 0.49, 0.51, 0.999)] == [2, 2, 4, 4]
    assert O.row_sample(torch.full((7,), float("nan")), 0.4)[0] == 0
    # margin: distance of u to the nearer interval end
    row = torch.zeros(4, dtype=torch.float64)
    tok, margin = O.row_sample(row, 0.30)
    assert tok == 1 and abs(margin - 0.05) < 1e-12


@pytest.mark.parametrize("T", [0.7, 1.0, 1.6])
def test_row_sample_frequencies_on_a_uniform_grid(T):
    """Over the equispaced uniforms (i + 1/2) / N an inverse-CDF sampler returns token v exactly
    N * p_v times up to one grid point per interval end, with p from the library softmax."""
    from scipy.special import softmax
    g = torch.Generator().manual_seed(8)
    y = (torch.randn(40, generator=g, dtype=torch.float64) * 2.0)
    p = softmax(y.numpy() / T)
    N = 4000
    counts = np.zeros(40, dtype=np.int64)
    prev = -1
    for i in range(N):
        v, _ = O.row_sample(y, (i + 0.5) / N, T)
        assert v >= prev                      # monotone in u: intervals lie in token order
        prev = v
        counts[v] += 1
    assert np.abs(counts - N * p).max() <= 1.0 + 1e-9


def test_accept_walk_with_given_tokens_matches_the_greedy_walk():
    """Pins the Python walk to the C one: one-hot target logits make the arg-max equal to the given tokens."""
    g = torch.Generator().manual_seed(12)
    V, R, L = 12, 9, 4
    for trial in range(40):
        n = int(torch.randint(0, R, (1,), generator=g))
        par = torch.zeros(1, R, dtype=torch.int32)
        tok = torch.zeros(1, R, dtype=torch.int32)
        for c in range(1, n + 1):
            par[0, c] = int(torch.randint(0, c, (1,), generator=g))
            tok[0, c] = int(torch.randint(0, 3, (1,), generator=g))       # few tokens: matches are frequent
        given = torch.randint(0, 3, (1, R), generator=g, dtype=torch.int32)
        y = torch.zeros(1, R, V, dtype=torch.float32)
        y.scatter_(2, given.long().unsqueeze(-1), 5.0)
        ref = O.verify_tree(y, L, torch.tensor([n], dtype=torch.int32), tok, par, O.ROWS_DENSE)
        acc, nxt = O.accept_walk(L, n, tok[0], par[0], given[0])
        assert len(acc) == int(ref.accepted_len[0]) and nxt == int(ref.next_bonus[0])
        assert acc == [int(c) for c in ref.accepted_nodes[0, : len(acc)]]


def test_sampled_verification_limits_and_losslessness():
    g = torch.Generator().manual_seed(5)
    batch, R, V, L = 3, 7, 30, 3
    y = torch.randn(batch, R, V, generator=g, dtype=torch.float32) * 3.0
    par = torch.tensor([[0, 0, 0, 1, 1, 3, 2]] * batch, dtype=torch.int32)
    tok = torch.randint(0, V, (batch, R), generator=g, dtype=torch.int32)
    n = torch.tensor([6, 4, 0], dtype=torch.int32)
    u = torch.rand(batch, R, generator=g, dtype=torch.float64)
    # T -> 0: the greedy verdict, whatever the uniforms
    cold, _ = O.verify_tree_sampled(y, u, L, n, tok, par, O.ROWS_LIVE, 1e-4)
    ref = O.verify_tree(y, L, n, tok, par, O.ROWS_LIVE)
    for f in ("node_argmax", "accepted_len", "accepted_nodes", "next_bonus", "status"):
        assert torch.equal(getattr(cold, f), getattr(ref, f)), f
    # LIVE leaves the rows beyond n unread
    warm, mg = O.verify_tree_sampled(y, u, L, n, tok, par, O.ROWS_LIVE, 1.0)
    assert int(warm.node_argmax[1, 5]) == -1 and int(warm.node_argmax[2, 1]) == -1 and int(warm.accepted_len[2]) == 0
    assert torch.isinf(mg[1, 5])
    # losslessness at the root: over a grid of root uniforms the first emitted token (the accepted child's token, or
    # the bonus when nothing is accepted) is distributed as softmax(y_root)
    from scipy.special import softmax
    p = softmax(y[0, 0].double().numpy())
    N = 2000
    counts = np.zeros(V)
    accepted = 0
    for i in range(N):
        u[0, 0] = (i + 0.5) / N
        v, _ = O.verify_tree_sampled(y[:1], u[:1], L, n[:1], tok[:1], par[:1], O.ROWS_LIVE, 1.0)
        first = int(tok[0, int(v.accepted_nodes[0, 0])]) if int(v.accepted_len[0]) > 0 else int(v.next_bonus[0])
        counts[first] += 1
        accepted += int(v.accepted_len[0]) > 0
    assert np.abs(counts - N * p).max() <= 1.0 + 1e-9
    kids = {int(tok[0, c]) for c in (1, 2)}
    assert abs(accepted - N * sum(p[t] for t in kids)) <= len(kids) + 1e-9
