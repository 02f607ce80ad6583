"""GPU parity of the verification fused into the output projection (tensor-core path) against the CPU oracle."""
import pytest
import torch

from oracle import cadd_oracle as O
from paper_2606_01813_b200 import binding as G
from paper_2606_01813_b200 import synth
from parity_util import compare_build, to_cpu

pytestmark = pytest.mark.gpu


def planted_head_inputs(tree: O.OracleTree, L: int, hidden: int, V: int, seed: int, agreement: float = 0.6):
    """Hidden states and weight such that the target's argmax at a node is, with probability `agreement`, the token
    of one of its children (so that walks of several steps occur), else some other token."""
    g = torch.Generator().manual_seed(seed)
    batch, R = tree.token_ids.shape
    w = torch.randn(V, hidden, generator=g)
    h = 0.3 * torch.randn(batch, R, hidden, generator=g)
    for b in range(batch):
        n = int(tree.n_nodes[b])
        for j in range(R):
            kids = [c for c in range(1, n + 1) if int(tree.parent_idx[b, c]) == j] if j <= n else []
            if kids and (j == 0 or torch.rand((), generator=g) < agreement):     # the root always agrees
                t = int(tree.token_ids[b, kids[int(torch.randint(len(kids), (), generator=g))]])
            else:
                t = int(torch.randint(V, (), generator=g))
            h[b, j] += 4.0 * w[t] / w[t].norm()
    return h.bfloat16(), w.bfloat16()


def check_head(h, w, tree, L, rows_mode):
    ov, y64 = O.verify_tree_fused_head(h, w, L, tree.n_nodes, tree.token_ids, tree.parent_idx, rows_mode=rows_mode)
    dev = lambda t: t.cuda()
    gv = G.cadd_verify_tree_fused_head(h.cuda(), w.cuda(), L, dev(tree.n_nodes), dev(tree.token_ids), dev(tree.parent_idx), rows_mode)
    torch.cuda.synchronize()
    ga, oa = to_cpu(gv.node_argmax), ov.node_argmax
    assert int(to_cpu(gv.status).max()) & G.STATUS_INTERNAL_TIMEOUT == 0
    # fp32 accumulation of `hidden` products in an order the hardware chooses: |error| <= hidden * 2^-24 * sum |terms|
    # in the worst case; a differing pick is admissible only inside that bound (and then nothing downstream is compared)
    absdot = h.double().abs().reshape(-1, h.shape[2]) @ w.double().abs().T
    batch, R, V = y64.shape
    exempt = 0
    for b in range(batch):
        for j in range(R):
            if ga[b, j] == oa[b, j]:
                continue
            assert ga[b, j] >= 0 and oa[b, j] >= 0, (b, j, int(ga[b, j]), int(oa[b, j]))
            tol = h.shape[2] * 2.0 ** -24 * float(absdot[b * R + j, [int(ga[b, j]), int(oa[b, j])]].max())
            gap = float(y64[b, j, int(oa[b, j])] - y64[b, j, int(ga[b, j])])
            assert abs(gap) <= tol, (b, j, int(ga[b, j]), int(oa[b, j]), gap, tol)
            exempt += 1
    if exempt == 0:
        assert torch.equal(to_cpu(gv.accepted_len), ov.accepted_len)
        assert torch.equal(to_cpu(gv.accepted_nodes), ov.accepted_nodes)
        assert torch.equal(to_cpu(gv.next_bonus), ov.next_bonus)
    return exempt, ov


@pytest.mark.parametrize("shape", [
    # batch, hidden, V      (R comes from the tree; ragged row tiles, column tiles and k-steps on purpose)
    (1, 64, 300),
    (2, 256, 4099),
    (3, 200, 1000),
    (2, 1032, 2500),
])
@pytest.mark.parametrize("rows_mode", [G.ROWS_LIVE, G.ROWS_DENSE])
def test_fused_head_small(shape, rows_mode):
    batch, hidden, V = shape
    cfg = synth.scaled(synth.CONFIGS["c2"], batch=batch, V=max(V, 64))
    d = synth.make_draft_inputs(cfg, 11)
    c = synth.make_cost_inputs(cfg, 11)
    tree = O.build_tree(d.logits, cfg.K, cfg.B_max, cfg.R, l_eff=d.l_eff, bonus_token=d.bonus_token, ctx_len=d.ctx_len,
                        cost_coef=c.coef, flags=O.FLAG_FIXED_BUDGET)        # fixed budget: trees with many nodes
    h, w = planted_head_inputs(tree, cfg.L, hidden, V, seed=5)
    exempt, ov = check_head(h, w, tree, cfg.L, rows_mode)
    assert exempt <= 2
    assert int(ov.accepted_len.max()) >= 1                                  # the walk has something to follow


def test_fused_head_matches_materialised_logits():
    """Same answer as forming the logits with a library GEMM and calling cadd_verify_tree on them (up to the two
    GEMMs' own rounding: rows whose top two logits are closer than that are skipped)."""
    cfg = synth.scaled(synth.CONFIGS["c2"], batch=2, V=5000)
    d = synth.make_draft_inputs(cfg, 12)
    c = synth.make_cost_inputs(cfg, 12)
    tree = O.build_tree(d.logits, cfg.K, cfg.B_max, cfg.R, l_eff=d.l_eff, bonus_token=d.bonus_token, ctx_len=d.ctx_len,
                        cost_coef=c.coef, flags=O.FLAG_FIXED_BUDGET)
    h, w = planted_head_inputs(tree, cfg.L, 512, 5000, seed=6)
    hc, wc = h.cuda(), w.cuda()
    dev = lambda t: t.cuda()
    y = (hc.float() @ wc.float().T)
    top2 = y.topk(2, dim=-1).values
    clear = (top2[..., 0] - top2[..., 1]) > 1e-3
    g1 = G.cadd_verify_tree_fused_head(hc, wc, cfg.L, dev(tree.n_nodes), dev(tree.token_ids), dev(tree.parent_idx), G.ROWS_DENSE)
    g2 = G.cadd_verify_tree(y.contiguous(), cfg.L, dev(tree.n_nodes), dev(tree.token_ids), dev(tree.parent_idx), G.ROWS_DENSE)
    torch.cuda.synchronize()
    assert clear.float().mean() > 0.9
    assert torch.equal(g1.node_argmax[clear], g2.node_argmax[clear])


def test_fused_head_rejects_bad_arguments():
    h = torch.zeros(1, 3, 64, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(10, 64, dtype=torch.bfloat16, device="cuda")
    z = torch.zeros(1, dtype=torch.int32, device="cuda")
    t = torch.zeros(1, 3, dtype=torch.int32, device="cuda")
    with pytest.raises(ValueError):
        G.cadd_verify_tree_fused_head(h.float(), w, 4, z, t, t)
    with pytest.raises(G.CaddError):                                       # stride not a multiple of 8 elements
        G.cadd_verify_tree_fused_head(torch.zeros(1, 3, 68, dtype=torch.bfloat16, device="cuda")[:, :, :60],
                                      torch.zeros(10, 60, dtype=torch.bfloat16, device="cuda"), 4, z, t, t)


def test_fused_head_full_size_sampled_rows():
    """Config 2's verification shape (8224 rows, V = 151936) with hidden size 4096, in the launch configuration the
    bench times; the oracle recomputes a seeded sample of rows (one row costs V x hidden fp64 products)."""
    cfg = synth.CONFIGS["c2"]
    hidden = 4096
    g = torch.Generator(device="cuda").manual_seed(77)
    h = torch.randn(cfg.batch, cfg.R, hidden, device="cuda", dtype=torch.bfloat16, generator=g)
    w = torch.randn(cfg.V, hidden, device="cuda", dtype=torch.bfloat16, generator=g)
    n_nodes = torch.full((cfg.batch,), 7, dtype=torch.int32, device="cuda")
    tok = torch.zeros(cfg.batch, cfg.R, dtype=torch.int32, device="cuda")
    par = torch.zeros(cfg.batch, cfg.R, dtype=torch.int32, device="cuda")
    out = G.cadd_verify_tree_fused_head(h, w, cfg.L, n_nodes, tok, par, G.ROWS_DENSE)
    torch.cuda.synchronize()
    assert int(out.status.max()) == 0
    ga = to_cpu(out.node_argmax).reshape(-1)
    assert int(ga.min()) >= 0 and int(ga.max()) < cfg.V
    rows = torch.randint(0, cfg.batch * cfg.R, (12,), generator=torch.Generator().manual_seed(5)).tolist() + [0, cfg.batch * cfg.R - 1]
    hs = h.reshape(-1, hidden)[rows].cpu().unsqueeze(0)
    wc = w.cpu()
    y64 = O.head_logits(hs, wc)[0]
    absw = wc.double().abs()
    for i, r in enumerate(rows):
        o = int(y64[i].to(torch.float32).argmax())          # decision in the precision the GPU reports its logits in
        gpick = int(ga[r])
        if o != gpick:
            tol = hidden * 2.0 ** -24 * float((hs[0, i].double().abs() * absw[[o, gpick]]).sum(dim=1).max())
            assert abs(float(y64[i, o] - y64[i, gpick])) <= tol, (r, o, gpick)


# ---------------- tree construction fused into the drafter's output projection ----------------

def planted_draft_inputs(batch, L, hidden, V, seed, sigma=1.5):
    """Hidden states whose logits h . W^T are N(0, sigma^2) noise plus one boosted token per position."""
    g = torch.Generator().manual_seed(seed)
    w = torch.randn(V, hidden, generator=g)
    h = torch.randn(batch, L, hidden, generator=g) * (sigma / hidden ** 0.5)
    for b in range(batch):
        for i in range(L):
            t = int(torch.randint(V, (), generator=g))
            boost = float(4.0 + 6.0 * torch.rand((), generator=g)) * 0.9 ** i
            h[b, i] += boost * w[t] / float(w[t] @ w[t])
    return h.bfloat16(), w.bfloat16()


def check_fused_build(h, w, cfg, seed, **extra):
    c = synth.make_cost_inputs(cfg, seed)
    fixed = extra.pop("flags", 0)
    kw = dict(cost_coef=c.coef, **extra)
    ot, y64 = O.build_tree_fused_head(h, w, cfg.K, cfg.B_max, cfg.R, flags=fixed, **kw)
    gt = G.cadd_build_tree_fused_head(h.cuda(), w.cuda(), cfg.K, cfg.B_max, cfg.R, flags=G.FLAG_EMIT_TOPK | fixed,
                                      **{k: (v.cuda() if torch.is_tensor(v) else v) for k, v in kw.items()})
    torch.cuda.synchronize()
    # a logit is an fp32 accumulation of `hidden` products: |error| <= e = hidden * 2^-24 * sum_k |h_k W_vk| in the
    # worst case; a log-prob (logit - log Z) then carries at most 2e, a score over L depths at most 2 L e
    absdot = h.double().abs().reshape(-1, h.shape[2]) @ w.double().abs().T
    e = h.shape[2] * 2.0 ** -24 * float(absdot.max())
    diag = compare_build(gt, ot, cfg.K, check_topk=False, rel_tol=1e-5 + 2 * cfg.L * 2 * e, near_tie=max(1e-6, 2 * cfg.L * 2 * e))
    # top-K: token ids equal unless the oracle's own gap at the K-th place is inside the bound
    tt_g, tt_o = gt.topk_token.cpu(), ot.topk_token
    mism = (tt_g != tt_o).any(dim=-1)
    y = y64.reshape(-1, y64.shape[-1])
    for r in torch.nonzero(mism.reshape(-1)).flatten().tolist():
        top = torch.sort(y[r], descending=True).values[: cfg.K + 1]
        assert float((top[:-1] - top[1:]).min()) <= 2 * e, f"row {r}: top-K differs without a near-tie"
    lg, lo = gt.topk_logprob.cpu()[~mism], ot.topk_logprob[~mism]
    fin = torch.isfinite(lo)                                   # masked positions and short lists carry no log-probs
    assert torch.equal(torch.isfinite(lg), fin)
    if fin.any():
        assert float((lg[fin] - lo[fin]).abs().max()) <= 2 * e + 1e-7
    return diag, int(mism.sum()), ot


@pytest.mark.parametrize("shape", [
    # batch, L, hidden, V, K
    (1, 4, 64, 300, 4),
    (2, 16, 256, 4099, 8),
    (3, 16, 200, 20000, 16),
    (9, 16, 512, 2500, 32),      # 144 rows: two row tiles, the second ragged
])
def test_fused_draft_head_small(shape):
    batch, L, hidden, V, K = shape
    cfg = synth.scaled(synth.CONFIGS["c2"], batch=batch, L=L, V=V, K=K, B_max=64)
    h, w = planted_draft_inputs(batch, L, hidden, V, seed=hidden)
    diag, mism, ot = check_fused_build(h, w, cfg, 3)
    assert len(diag["exempt"]) <= 1 and mism <= 1
    assert int(ot.n_nodes.max()) >= 2


def test_fused_draft_head_masked_positions_and_fixed_budget():
    batch, L, hidden, V = 5, 16, 128, 3000
    cfg = synth.scaled(synth.CONFIGS["c5"], batch=batch, L=L, V=V, K=8, B_max=96)
    h, w = planted_draft_inputs(batch, L, hidden, V, seed=31)
    l_eff = torch.tensor([4, 16, 0, 9, 1], dtype=torch.int32)
    bonus = torch.arange(batch, dtype=torch.int32)
    diag, mism, ot = check_fused_build(h, w, cfg, 4, l_eff=l_eff, bonus_token=bonus, flags=O.FLAG_FIXED_BUDGET)
    assert int(ot.n_nodes[2]) == 0 and int(ot.n_nodes.max()) == 96


def test_fused_draft_head_full_size_sampled_rows():
    """Config 2's draft shape (512 rows, V = 151936, K = 8) with hidden size 4096, in the launch configuration the
    bench times.  The oracle recomputes the logits of a seeded sample of requests' rows; their top-K lists and
    log-probabilities must agree (near-ties inside the accumulation bound excepted), and the whole tree of every
    sampled request must be the oracle's."""
    cfg = synth.CONFIGS["c2"]
    hidden = 4096
    h, w = planted_draft_inputs(cfg.batch, cfg.L, hidden, cfg.V, seed=99)
    c = synth.make_cost_inputs(cfg, 3)
    gt = G.cadd_build_tree_fused_head(h.cuda(), w.cuda(), cfg.K, cfg.B_max, cfg.R, cost_coef=c.coef.cuda(), flags=G.FLAG_EMIT_TOPK)
    torch.cuda.synchronize()
    assert int(gt.status.max()) & G.STATUS_INTERNAL_TIMEOUT == 0
    sample = [0, 13, 31]
    ot, y64 = O.build_tree_fused_head(h[sample], w, cfg.K, cfg.B_max, cfg.R, cost_coef=c.coef[sample])
    absdot = h[sample].double().abs().reshape(-1, hidden) @ w.double().abs().T
    e = hidden * 2.0 ** -24 * float(absdot.max())
    sub = G.Tree(**{f: (getattr(gt, f)[sample] if getattr(gt, f) is not None else None) for f in gt.__dataclass_fields__})
    diag = compare_build(sub, ot, cfg.K, check_topk=False, rel_tol=1e-5 + 2 * cfg.L * 2 * e, near_tie=max(1e-6, 2 * cfg.L * 2 * e))
    assert len(diag["exempt"]) <= 1
    mism = (sub.topk_token.cpu() != ot.topk_token).any(dim=-1)
    assert int(mism.sum()) <= 1
    lg, lo = sub.topk_logprob.cpu()[~mism], ot.topk_logprob[~mism]
    assert float((lg - lo).abs().max()) <= 2 * e + 1e-7
