"""GPU parity tests: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import cadd_oracle as O
from paper_2606_01813_b200 import binding as G
from paper_2606_01813_b200 import synth
from parity_util import compare_build, compare_verify, run_both_build, to_cpu, LOGZ_TOL

pytestmark = pytest.mark.gpu


def quad_coef(batch, t_draft, a, b, c):
    return torch.tensor([[t_draft, a, b, c]] * batch, dtype=torch.float64)


def cost_kwargs(c: synth.CostInputs):
    if c.kind == synth.COST_TABLE:
        return dict(cost_kind=G.COST_TABLE, cost_table=c.table, table_idx=c.table_idx, t_draft=c.t_draft)
    return dict(cost_kind=G.COST_QUADRATIC, cost_coef=c.coef)


@pytest.fixture(autouse=True, params=["one-launch where small", "regular"])
def launch_path(request):
    """Small problems are served by one kernel per call; every test of this file runs once as a caller would and once
    with all calls forced onto the regular two-kernel path, so that both are held to the oracle on the same cases."""
    G.FORCE_REGULAR_PATH = request.param == "regular"
    yield
    G.FORCE_REGULAR_PATH = False


def round_trip(cfg, seed, rows_mode=G.ROWS_LIVE, dense_mask=False):
    """One full round (build, target logits for the built tree, verify) on both sides."""
    d = synth.make_draft_inputs(cfg, seed)
    c = synth.make_cost_inputs(cfg, seed)
    flags = (G.FLAG_FIXED_BUDGET if cfg.fixed_budget else 0) | (G.FLAG_EMIT_DENSE_MASK if dense_mask else 0)
    gt, ot = run_both_build(d.logits, cfg.K, cfg.B_max, cfg.R, l_eff=d.l_eff, bonus_token=d.bonus_token,
                            ctx_len=d.ctx_len, flags=flags, **cost_kwargs(c))
    diag = compare_build(gt, ot, cfg.K)
    if dense_mask:
        assert torch.equal(to_cpu(gt.mask_dense), ot.mask_dense)
    y = synth.make_target_logits(cfg, seed, d, ot.depth)
    ov = O.verify_tree(y, cfg.L, ot.n_nodes, ot.token_ids, ot.parent_idx, rows_mode=rows_mode)
    dev = lambda t: t.cuda()
    gv = G.cadd_verify_tree(y.cuda(), cfg.L, dev(ot.n_nodes), dev(ot.token_ids), dev(ot.parent_idx), rows_mode=rows_mode)
    torch.cuda.synchronize()
    compare_verify(gv, ov)
    return diag, ot, ov


def test_library_reports_version():
    assert G.cadd_version() == 4
    assert G.cadd_status_string(0) == "ok"


@pytest.mark.parametrize("seed", [0, 1, 2])
@pytest.mark.parametrize("rows_mode", [G.ROWS_LIVE, G.ROWS_DENSE])
def test_config1_full_round(seed, rows_mode):
    diag, ot, ov = round_trip(synth.CONFIGS["c1"], seed, rows_mode, dense_mask=True)
    assert not diag["exempt"]
    assert diag["max_logZ_err"] < LOGZ_TOL


# Reduced-size versions of configs 2-5: same generators, dtype, V and structure, fewer requests so the
# oracle finishes in seconds.  V = 151936 spans many tiles, several segments and is not a power of two.
SMALL = {
    "c2": dict(batch=3),
    "c3": dict(batch=3, B_max=128),
    "c4": dict(batch=2, L=8, B_max=96),
    "c4_stress": dict(batch=2, L=8, B_max=200),
    "c5": dict(batch=6),
}


@pytest.mark.parametrize("name", list(SMALL))
def test_reduced_configs_full_round(name):
    cfg = synth.scaled(synth.CONFIGS[name], **SMALL[name])
    diag, ot, ov = round_trip(cfg, synth.config_seed(cfg), G.ROWS_LIVE)
    print(name, "n*", ot.n_nodes.tolist(), "alpha", ov.accepted_len.tolist(), diag)
    assert diag["exempt"] == []
    assert diag["max_logZ_err"] < LOGZ_TOL


def test_config5_rounds_with_fresh_seeds():
    """Configuration 5 is defined as many rounds with a fresh seed each (varying L_eff and jittered costs per
    request): a reduced batch over a run of consecutive rounds, both verification modes."""
    cfg = synth.scaled(synth.CONFIGS["c5"], batch=4)
    exempt = 0
    for rnd in range(8):
        for mode in (G.ROWS_LIVE, G.ROWS_DENSE):
            diag, ot, ov = round_trip(cfg, synth.config_seed(cfg, rnd), mode)
            exempt += len(diag["exempt"])
            assert diag["max_logZ_err"] is None or diag["max_logZ_err"] < LOGZ_TOL
    assert exempt == 0


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("V", [1, 2, 7, 8, 9, 63, 257, 1000, 4099, 40000])
def test_random_small_cases(dtype, V):
    rng = np.random.default_rng(V)
    for trial in range(6):
        batch, L = int(rng.integers(1, 5)), int(rng.integers(1, 9))
        K, B = int(rng.integers(1, 12)), int(rng.integers(0, 90))
        g = torch.Generator().manual_seed(1000 * V + trial)
        scale = float(rng.uniform(0.5, 5))
        x = torch.randn(batch, L, V, generator=g) * scale
        if trial % 2:
            x = torch.round(x * 2) / 2                    # heavy ties
        x = x.to(dtype)
        coef = torch.tensor([[rng.uniform(0.1, 1), rng.uniform(0.2, 2), rng.uniform(1e-3, 5e-2), rng.uniform(0, 1e-3)]
                             for _ in range(batch)], dtype=torch.float64)
        flags = G.FLAG_FIXED_BUDGET if trial % 3 == 0 else 0
        R = B + 1 + int(rng.integers(0, 40))
        gt, ot = run_both_build(x, K, B, R, cost_coef=coef, flags=flags,
                                ctx_len=torch.arange(batch, dtype=torch.int32) * 7)
        diag = compare_build(gt, ot, K)
        assert not diag["exempt"], diag
        assert diag["max_logZ_err"] < 1e-6


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_random_small_problems_wide_lists_masked_positions_offsets(seed):
    """Random small problems with what the cases above leave out: lists of up to 64 tokens (more than a warp has lanes),
    rows that start at odd offsets inside a wider tensor, masked positions, non-finite logits, all-equal rows."""
    rng = np.random.default_rng(4242 + seed)
    g = torch.Generator().manual_seed(99 + seed)
    for trial in range(12):
        batch, L = int(rng.choice([1, 2, 3, 5])), int(rng.choice([1, 2, 3, 5, 8, 13, 16]))
        V = int(rng.choice([1, 2, 7, 33, 100, 257, 1000, 1024, 2047, 2048]))
        K, B = int(rng.choice([1, 2, 4, 8, 13, 32, 40, 64])), int(rng.choice([0, 1, 5, 32, 100, 300]))
        dtype = torch.float32 if rng.integers(0, 2) else torch.bfloat16
        off = int(rng.choice([0, 1, 3, 4, 5]))
        mode = ["normal", "ties", "flat", "nonfinite"][int(rng.integers(0, 4))]
        x = torch.randn(batch, L, V + 8, generator=g) * float(rng.choice([0.5, 1.0, 3.0]))
        if mode == "ties":
            x = torch.round(x * 2) / 2
        elif mode == "flat":
            x = torch.zeros_like(x)
        elif mode == "nonfinite":
            m = torch.rand(x.shape, generator=g)
            x[m < 0.05] = float("-inf")
            x[(m > 0.05) & (m < 0.07)] = float("nan")
        x = x.to(dtype)
        # (the marginal cost is kept positive: with a constant cost the rule stops where a node's probability drops below
        # the rounding of 1 + Phi, which is not a property of the tree)
        coef = torch.tensor([[rng.choice([0.3, 1.0]), rng.choice([0.5, 2.0]), rng.choice([0.002, 0.01, 0.05]), rng.choice([0.0, 0.0005])]
                             for _ in range(batch)], dtype=torch.float64)
        le = torch.tensor(rng.integers(0, L + 1, size=batch), dtype=torch.int32)
        flags = G.FLAG_FIXED_BUDGET if rng.integers(0, 2) else 0
        ot = O.build_tree(x[:, :, off:off + V].contiguous(), K, B, cost_coef=coef, l_eff=le, flags=flags)
        gt = G.cadd_build_tree(x.cuda()[:, :, off:off + V], K, B, cost_coef=coef, l_eff=le, flags=flags | G.FLAG_EMIT_TOPK)
        torch.cuda.synchronize()
        diag = compare_build(gt, ot, K)
        assert not diag["exempt"], (diag, batch, L, V, K, B, dtype, off, mode)
        assert diag["max_logZ_err"] < 1e-6


@pytest.mark.parametrize("seed", [0, 1])
def test_random_midsize_problems_wide_lists_masked_positions_offsets(seed):
    """The same mix on vocabularies of thousands to 150 thousand tokens (several tiles and segments per row, records of up
    to 256 keys), where every call takes the two-kernel path."""
    rng = np.random.default_rng(777 + seed)
    g = torch.Generator().manual_seed(5 + seed)
    for trial in range(10):
        batch, L = int(rng.choice([1, 2, 3])), int(rng.choice([1, 2, 5, 8, 16, 32]))
        V = int(rng.choice([2049, 3000, 8192, 20000, 50001, 151936]))
        K, B = int(rng.choice([1, 2, 4, 8, 13, 32, 40, 64])), int(rng.choice([0, 1, 5, 32, 100, 300]))
        dtype = torch.float32 if rng.integers(0, 2) else torch.bfloat16
        off = int(rng.choice([0, 1, 3, 4, 5]))
        mode = ["normal", "ties", "flat", "nonfinite"][int(rng.integers(0, 4))]
        x = torch.randn(batch, L, V + 8, generator=g) * float(rng.choice([0.5, 1.0, 3.0]))
        if mode == "ties":
            x = torch.round(x * 2) / 2
        elif mode == "flat":
            x = torch.zeros_like(x)
        elif mode == "nonfinite":
            m = torch.rand(x.shape, generator=g)
            x[m < 0.05] = float("-inf")
            x[(m > 0.05) & (m < 0.07)] = float("nan")
        x = x.to(dtype)
        coef = torch.tensor([[rng.choice([0.3, 1.0]), rng.choice([0.5, 2.0]), rng.choice([0.002, 0.01, 0.05]), rng.choice([0.0, 0.0005])]
                             for _ in range(batch)], dtype=torch.float64)
        le = torch.tensor(rng.integers(0, L + 1, size=batch), dtype=torch.int32)
        flags = G.FLAG_FIXED_BUDGET if rng.integers(0, 2) else 0
        ot = O.build_tree(x[:, :, off:off + V].contiguous(), K, B, cost_coef=coef, l_eff=le, flags=flags)
        gt = G.cadd_build_tree(x.cuda()[:, :, off:off + V], K, B, cost_coef=coef, l_eff=le, flags=flags | G.FLAG_EMIT_TOPK)
        torch.cuda.synchronize()
        diag = compare_build(gt, ot, K)
        assert not diag["exempt"], (diag, batch, L, V, K, B, dtype, off, mode)
        assert diag["max_logZ_err"] < 1e-6


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_random_rounds_verification_both_row_modes(seed):
    """Random full rounds on small and mid-size vocabularies: the tree from the builder, target logits that agree with the
    tree's tokens at a random share of the nodes (and tie, or hold NaN, in places), verification in both row modes."""
    rng = np.random.default_rng(31337 + seed)
    g = torch.Generator().manual_seed(17 + seed)
    for trial in range(8):
        batch, L = int(rng.choice([1, 2, 4])), int(rng.choice([1, 3, 8, 16]))
        V = int(rng.choice([2, 33, 257, 1024, 4099, 8192, 20000]))
        K, B = int(rng.choice([1, 2, 4, 8])), int(rng.choice([1, 8, 32, 100]))
        dtype = torch.float32 if rng.integers(0, 2) else torch.bfloat16
        x = (torch.randn(batch, L, V, generator=g) * 2.0).to(dtype)
        coef = torch.tensor([[0.3, 0.5, 0.002, 0.0]] * batch, dtype=torch.float64)
        gt, ot = run_both_build(x, K, B, cost_coef=coef, flags=G.FLAG_FIXED_BUDGET if trial % 2 else 0)
        assert not compare_build(gt, ot, K)["exempt"]
        R = B + 1
        y = torch.randn(batch, R, V, generator=g)
        if trial % 3 == 0:
            y = torch.round(y)                                  # arg-max ties: the lowest id wins
        agree = float(rng.choice([0.3, 0.7, 1.0]))
        tok, par = ot.token_ids, ot.parent_idx
        for b in range(batch):                                  # plant the child's token at its parent's row
            for j in range(1, int(ot.n_nodes[b]) + 1):
                if rng.random() < agree:
                    y[b, int(par[b, j]), int(tok[b, j])] = 50.0 + j
        if trial % 4 == 1:
            y[:, :, 0] = float("nan")
        y = y.to(dtype)
        for rows_mode in (G.ROWS_LIVE, G.ROWS_DENSE):
            ov = O.verify_tree(y, L, ot.n_nodes, ot.token_ids, ot.parent_idx, rows_mode)
            gv = G.cadd_verify_tree(y.cuda(), L, gt.n_nodes, gt.token_ids, gt.parent_idx, rows_mode)
            torch.cuda.synchronize()
            compare_verify(gv, ov)


def test_unaligned_rows_and_strides():
    """Row starts that are not 16-byte aligned (odd V, offset base) go through the scalar head/tail path."""
    g = torch.Generator().manual_seed(5)
    for dtype in (torch.bfloat16, torch.float32):
        for V in (1001, 4099):
            big = (torch.randn(3, 4, V + 13, generator=g) * 3).to(dtype)
            x = big[:, :, 5:5 + V]                         # strided view, unaligned rows
            coef = quad_coef(3, 0.3, 1.0, 0.002, 0.00002)
            ot = O.build_tree(x.contiguous(), 8, 64, cost_coef=coef)
            gt = G.cadd_build_tree(big.cuda()[:, :, 5:5 + V], 8, 64, cost_coef=coef, flags=G.FLAG_EMIT_TOPK)
            torch.cuda.synchronize()
            compare_build(gt, ot, 8)
            y = (torch.randn(3, 65, V + 3, generator=g)).to(dtype)
            ov = O.verify_tree(y[:, :, 1:1 + V].contiguous(), 4, ot.n_nodes, ot.token_ids, ot.parent_idx, rows_mode=O.ROWS_DENSE)
            gv = G.cadd_verify_tree(y.cuda()[:, :, 1:1 + V], 4, ot.n_nodes.cuda(), ot.token_ids.cuda(), ot.parent_idx.cuda(),
                                    rows_mode=G.ROWS_DENSE)
            torch.cuda.synchronize()
            compare_verify(gv, ov)


def test_nonfinite_and_degenerate_inputs():
    g = torch.Generator().manual_seed(9)
    x = (torch.randn(6, 4, 3000, generator=g) * 2).to(torch.bfloat16)
    x[0, 1, 5] = float("inf")                  # +Inf: empty tree
    x[1, 0, 3] = float("nan")                  # NaN: ordered as -Inf
    x[1, 2, 100:2000] = float("nan")
    x[2, 1, :] = -float("inf")                 # a position with no finite logit
    x[3, :, 7:] = -float("inf")                # only 7 finite logits per row: fewer than K
    x[4] = 0.5                                 # all logits equal: order fixed by the tie-break alone
    x[5, :, :] = torch.sort(x[5].float(), dim=-1).values.to(torch.bfloat16)   # ascending: every element a new best
    coef = quad_coef(6, 0.3, 1.0, 0.002, 0.00002)
    for flags in (0, G.FLAG_FIXED_BUDGET):
        gt, ot = run_both_build(x, 9, 50, 60, cost_coef=coef, flags=flags,
                                l_eff=torch.tensor([4, 4, 4, 4, 9, -1], dtype=torch.int32))
        diag = compare_build(gt, ot, 9)
        assert not diag["exempt"]
    coef_bad = quad_coef(6, -2.0, 1.0, 0.002, 0.0)
    gt, ot = run_both_build(x, 9, 50, 60, cost_coef=coef_bad)
    compare_build(gt, ot, 9)
    assert all(int(s) & G.STATUS_COST_NONPOSITIVE for s in to_cpu(gt.status))


def test_table_cost_and_limits():
    g = torch.Generator().manual_seed(10)
    x = (torch.randn(2, 64, 500, generator=g) * 2).to(torch.float32)      # L = 64, K = 64: the limits of the ABI
    n = torch.arange(301, dtype=torch.float64)
    table = torch.stack([0.9 + 0.01 * n + 0.0004 * n * n, 0.5 + 0.002 * n])
    kw = dict(cost_kind=G.COST_TABLE, cost_table=table, table_idx=torch.tensor([1, 0], dtype=torch.int32),
              t_draft=torch.tensor([0.3, 0.2], dtype=torch.float64))
    for flags in (0, G.FLAG_FIXED_BUDGET):
        gt, ot = run_both_build(x, 64, 300, **kw, flags=flags)
        assert not compare_build(gt, ot, 64)["exempt"]
    x = (torch.randn(1, 3, 300, generator=g)).to(torch.bfloat16)          # B_max = 2048: the largest cap
    gt, ot = run_both_build(x, 16, 2048, cost_coef=quad_coef(1, 1.0, 1.0, 0.0, 0.0), flags=G.FLAG_FIXED_BUDGET)
    assert not compare_build(gt, ot, 16)["exempt"]
    assert int(ot.n_nodes[0]) == 2048


def test_table_index_out_of_range_is_flagged_and_reads_nothing():
    """A table index that names no table must not be dereferenced: the request is flagged and gets the empty tree,
    its neighbours are untouched."""
    g = torch.Generator().manual_seed(12)
    x = (torch.randn(4, 5, 700, generator=g) * 2).to(torch.bfloat16)
    n = torch.arange(41, dtype=torch.float64)
    table = torch.stack([0.9 + 0.01 * n + 0.0004 * n * n, 0.5 + 0.002 * n])
    kw = dict(cost_kind=G.COST_TABLE, cost_table=table, table_idx=torch.tensor([-1, 1, 2, 1 << 30], dtype=torch.int32),
              t_draft=torch.tensor([0.3, 0.2, 0.3, 0.3], dtype=torch.float64))
    for flags in (0, G.FLAG_FIXED_BUDGET):
        gt, ot = run_both_build(x, 6, 40, **kw, flags=flags)
        assert not compare_build(gt, ot, 6)["exempt"]
        st = to_cpu(gt.status)
        assert [bool(int(v) & G.STATUS_BAD_TABLE_IDX) for v in st] == [True, False, True, True]
        assert to_cpu(gt.n_nodes)[[0, 2, 3]].tolist() == [0, 0, 0] and int(gt.n_nodes[1]) > 0


def test_argmax_ties_nan_and_walk():
    g = torch.Generator().manual_seed(11)
    batch, R, V, L = 3, 40, 151936, 6
    y = torch.randn(batch, R, V, generator=g).to(torch.bfloat16)           # bf16 N(0,1): frequent exact ties at the top
    y[0, 3, :] = float("nan")
    y[0, 4, :] = -float("inf")
    y[0, 5, 100] = float("nan"); y[0, 5, 7] = 9.0; y[0, 5, 150000] = 9.0
    y[1, 2, V - 1] = 50.0
    y[1, 3, 0] = 50.0
    y[2, 0, :] = 0.0; y[2, 0, 5] = -0.0
    x = (torch.randn(batch, L, 40, generator=g) * 2).to(torch.float32)
    ot = O.build_tree(x, 4, R - 1, cost_coef=quad_coef(batch, 1.0, 1.0, 0.0, 0.0), flags=O.FLAG_FIXED_BUDGET)
    for b in range(batch):                      # make the walk non-trivial: target agrees with the tree often
        for j in range(R):
            kids = [c for c in range(1, R) if int(ot.parent_idx[b, c]) == j]
            if kids and j % 7 != 6 and not (b == 0 and j in (3, 4, 5)) and not (b == 2 and j == 0):
                y[b, j, int(ot.token_ids[b, kids[0]])] = 60.0
    for mode in (G.ROWS_LIVE, G.ROWS_DENSE):
        n_nodes = ot.n_nodes.clone()
        if mode == G.ROWS_LIVE:
            n_nodes[1] = 17
        ov = O.verify_tree(y, L, n_nodes, ot.token_ids, ot.parent_idx, rows_mode=mode)
        gv = G.cadd_verify_tree(y.cuda(), L, n_nodes.cuda(), ot.token_ids.cuda(), ot.parent_idx.cuda(), rows_mode=mode)
        torch.cuda.synchronize()
        compare_verify(gv, ov)
        assert int(ov.accepted_len.max()) >= 3
    bad = ot.n_nodes.clone(); bad[0] = -5; bad[2] = 1000
    ov = O.verify_tree(y, L, bad, ot.token_ids, ot.parent_idx)
    gv = G.cadd_verify_tree(y.cuda(), L, bad.cuda(), ot.token_ids.cuda(), ot.parent_idx.cuda())
    torch.cuda.synchronize()
    compare_verify(gv, ov)
    assert int(ov.status[0]) & O.ST_BAD_N_NODES


def test_deterministic_and_reused_buffers():
    cfg = synth.scaled(synth.CONFIGS["c2"], batch=2)
    d = synth.make_draft_inputs(cfg, 3)
    c = synth.make_cost_inputs(cfg, 3)
    x = d.logits.cuda()
    ws = torch.empty(G.cadd_build_workspace_bytes(cfg.batch, cfg.L, cfg.V, cfg.K, cfg.B_max, cfg.R, x.dtype),
                     dtype=torch.uint8, device="cuda")
    ws.fill_(0xAB)                              # scratch needs no initialisation
    t1 = G.cadd_build_tree(x, cfg.K, cfg.B_max, cost_coef=c.coef, workspace=ws, flags=G.FLAG_EMIT_TOPK)
    t2 = G.cadd_build_tree(x, cfg.K, cfg.B_max, cost_coef=c.coef, workspace=ws, flags=G.FLAG_EMIT_TOPK, out=None)
    torch.cuda.synchronize()
    for f in ("n_nodes", "token_ids", "parent_idx", "depth", "position_ids", "mask_bits", "topk_token", "status"):
        assert torch.equal(getattr(t1, f), getattr(t2, f)), f
    # evicted top-K candidates are folded into the partition sums in the order shared-memory atomics
    # happened to hand out buffer slots (each thread folds with its own fp32 reference exponent), so
    # floating-point outputs repeat to about 1e-10 in log space, not bit for bit
    for f in ("node_logprob", "phi", "theta", "topk_logprob"):
        a, b = getattr(t1, f), getattr(t2, f)
        fin = torch.isfinite(a)
        assert torch.equal(fin, torch.isfinite(b)) and torch.allclose(a[fin], b[fin], rtol=0, atol=2e-9), f


def test_round_replays_from_a_cuda_graph():
    """Both entry points only enqueue kernels on the given stream, so one round can be captured once and
    replayed; a replay on fresh inputs of the same shape gives the oracle's answer."""
    cfg = synth.scaled(synth.CONFIGS["c2"], batch=2, V=32000)
    d0, d1 = synth.make_draft_inputs(cfg, 5), synth.make_draft_inputs(cfg, 6)
    c = synth.make_cost_inputs(cfg, 5)
    x = d0.logits.cuda()
    y = torch.zeros(cfg.batch, cfg.R, cfg.V, dtype=x.dtype, device="cuda")
    kw = dict(l_eff=d0.l_eff.cuda(), bonus_token=d0.bonus_token.cuda(), ctx_len=d0.ctx_len.cuda(), cost_coef=c.coef.cuda())
    ws = torch.empty(G.cadd_build_workspace_bytes(cfg.batch, cfg.L, cfg.V, cfg.K, cfg.B_max, cfg.R, x.dtype),
                     dtype=torch.uint8, device="cuda")
    tree = G.cadd_build_tree(x, cfg.K, cfg.B_max, cfg.R, workspace=ws, **kw)            # first call outside capture
    verdict = G.cadd_verify_tree(y, cfg.L, tree.n_nodes, tree.token_ids, tree.parent_idx, G.ROWS_LIVE)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        G.cadd_build_tree(x, cfg.K, cfg.B_max, cfg.R, workspace=ws, out=tree, **kw)
        G.cadd_verify_tree(y, cfg.L, tree.n_nodes, tree.token_ids, tree.parent_idx, G.ROWS_LIVE, out=verdict)
    for d in (d1, d0):
        x.copy_(d.logits)
        ot = O.build_tree(d.logits, cfg.K, cfg.B_max, cfg.R, l_eff=d0.l_eff, bonus_token=d0.bonus_token, ctx_len=d0.ctx_len,
                          cost_coef=c.coef)
        yy = synth.make_target_logits(cfg, 5, d, ot.depth)
        y.copy_(yy)
        g.replay()
        torch.cuda.synchronize()
        compare_build(tree, ot, cfg.K)
        compare_verify(verdict, O.verify_tree(yy, cfg.L, ot.n_nodes, ot.token_ids, ot.parent_idx, rows_mode=G.ROWS_LIVE))


def test_context_interpolated_cost_and_theta_curve():
    """Table cost blended by context length (Eq. 13) and the theta*(n) curve output, against the oracle."""
    B = 200
    tables, grid = synth.make_context_cost_tables(B)
    gen = torch.Generator().manual_seed(77)
    x = (torch.randn(8, 6, 5000, generator=gen) * 3).to(torch.bfloat16)
    ctx = torch.tensor([0, 512, 1024, 2300, 5000, 8191, 8192, 30000], dtype=torch.int32)
    td = torch.full((8,), 0.25, dtype=torch.float64)
    for flags in (0, G.FLAG_FIXED_BUDGET):
        kw = dict(ctx_len=ctx, cost_kind=G.COST_TABLE_INTERP, cost_table=tables, ctx_grid=grid, t_draft=td)
        ot = O.build_tree(x, 6, B, flags=flags, **kw)
        gt = G.cadd_build_tree(x.cuda(), 6, B, flags=flags | G.FLAG_EMIT_TOPK, theta_curve=True, **kw)
        torch.cuda.synchronize()
        assert not compare_build(gt, ot, 6)["exempt"]
        np.testing.assert_allclose(to_cpu(gt.theta_curve).numpy(), ot.theta_curve.numpy(), rtol=1e-5, atol=0)
    assert int(ot.n_nodes.min()) == B                      # the fixed-budget run is a whole budget sweep
    curve = to_cpu(gt.theta_curve).numpy()
    stop = O.build_tree(x, 6, B, **kw)
    for b in range(8):                                     # Corollary 1: the rule stops at the curve's first maximum
        assert int(stop.n_nodes[b]) == int(np.argmax(curve[b] >= curve[b].max() * (1 - 1e-12)))


def test_adversarial_rows_full_vocabulary():
    """Rows that defeat the streaming top-K heuristics at V = 151936: ascending (every element a new best: the
    candidate ring overflows and the careful path takes over), descending, all equal, two values alternating,
    large magnitudes, denormals, and a row whose mass sits in one token.  K = 64 is the largest list."""
    V, L = 151936, 8
    g = torch.Generator().manual_seed(123)
    base = torch.randn(L, V, generator=g) * 2
    x = torch.empty(1, L, V)
    x[0, 0] = torch.sort(base[0]).values                           # ascending
    x[0, 1] = torch.sort(base[1], descending=True).values          # descending
    x[0, 2] = 1.5                                                   # all equal
    x[0, 3] = torch.where(torch.arange(V) % 2 == 0, torch.tensor(0.25), torch.tensor(-0.25))
    x[0, 4] = base[4] * 1e4                                         # large magnitudes (the documented range is |x| <= 1e6)
    x[0, 5] = base[5] * 1e-40                                       # denormals in fp32, zeros in bf16
    x[0, 6] = base[6]; x[0, 6, 77777] = 80.0                        # one dominant token
    x[0, 7] = torch.round(base[7])                                  # a handful of distinct values, massive ties
    coef = quad_coef(1, 0.3, 1.0, 0.002, 0.00002)
    for dtype in (torch.bfloat16, torch.float32):
        xs = x.to(dtype)
        for K, B in ((64, 300), (3, 40)):
            for flags in (0, G.FLAG_FIXED_BUDGET):
                gt, ot = run_both_build(xs, K, B, cost_coef=coef, flags=flags)
                diag = compare_build(gt, ot, K)
                assert not diag["exempt"], diag
                assert diag["max_logZ_err"] < 1e-6, diag


def scaled_cost_kwargs(c, cd_scale: float, cv_scale: float):
    """The cost inputs with the draft cost C_d and the verification cost C_v(.) multiplied by constants."""
    if c.kind == synth.COST_TABLE:
        return dict(cost_kind=G.COST_TABLE, cost_table=c.table * cv_scale, table_idx=c.table_idx, t_draft=c.t_draft * cd_scale)
    coef = c.coef.clone()
    coef[:, 0] *= cd_scale
    coef[:, 1:] *= cv_scale
    return dict(cost_kind=G.COST_QUADRATIC, cost_coef=coef)


@pytest.mark.parametrize("name", ["c2", "c3", "c5"])
def test_cost_sensitivity_analogue(name):
    """Synthetic analogue of the paper's sensitivity ablation (Section 5, Table "Sensitivity ... to cost parameter
    perturbations"): the builder is run with C_d and C_v each scaled by 0.5 and 2.  Parity with the oracle at every
    setting, plus what Eq. 11 implies: the stop test compares delta/(1+Phi) with (C_v(n+1)-C_v(n))/(C_d+C_v(n)), whose
    right side falls when C_d grows and rises when C_v is scaled up, so n* is non-decreasing in the C_d scale and
    non-increasing in the C_v scale, request by request."""
    cfg = synth.scaled(synth.CONFIGS[name], **SMALL[name])
    seed = synth.config_seed(cfg)
    d = synth.make_draft_inputs(cfg, seed)
    c = synth.make_cost_inputs(cfg, seed)
    n_star = {}
    for cd, cv in ((1.0, 1.0), (0.5, 1.0), (2.0, 1.0), (1.0, 0.5), (1.0, 2.0)):
        gt, ot = run_both_build(d.logits, cfg.K, cfg.B_max, cfg.R, l_eff=d.l_eff, bonus_token=d.bonus_token,
                                ctx_len=d.ctx_len, **scaled_cost_kwargs(c, cd, cv))
        diag = compare_build(gt, ot, cfg.K)
        assert diag["exempt"] == [], diag
        n_star[(cd, cv)] = to_cpu(gt.n_nodes)
    assert bool((n_star[(0.5, 1.0)] <= n_star[(1.0, 1.0)]).all()) and bool((n_star[(1.0, 1.0)] <= n_star[(2.0, 1.0)]).all())
    assert bool((n_star[(1.0, 0.5)] >= n_star[(1.0, 1.0)]).all()) and bool((n_star[(1.0, 1.0)] >= n_star[(1.0, 2.0)]).all())
    if name == "c3":                                                              # large enough trees: the perturbation does move them
        assert int(n_star[(1.0, 0.5)].sum()) > int(n_star[(1.0, 2.0)].sum())


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_live_verification_with_several_rows_per_cta(dtype):
    """LIVE verification with a small node cap lets one CTA read several rows of a request one after the other
    (its ring of tiles carries on from row to row): requests with 0, a few and all rows live, rows that start off a
    16-byte boundary, against the oracle; the padding rows read -1 and DENSE agrees on the live rows."""
    g = torch.Generator().manual_seed(44)
    batch, R, V, L = 4, 201, 9001, 6
    big = (torch.randn(batch, R, V + 5, generator=g) * 2.0).to(dtype)
    y = big[:, :, 3: 3 + V]                                        # unaligned rows, odd row stride
    n = torch.tensor([0, 5, 200, 37], dtype=torch.int32)
    par = torch.zeros(batch, R, dtype=torch.int32)
    for c in range(1, R):
        par[:, c] = torch.randint(0, c, (batch,), generator=g, dtype=torch.int32)
    tok = torch.randint(0, V, (batch, R), generator=g, dtype=torch.int32)
    am = y.float().argmax(-1).to(torch.int32)
    for b in range(batch):                                         # plant a chain so that the walk accepts a few nodes
        cur = 0
        for c in range(1, min(int(n[b]), 4) + 1):
            par[b, c] = cur
            tok[b, c] = am[b, cur]
            cur = c
    yd = big.cuda()[:, :, 3: 3 + V]
    dev = lambda t: t.cuda()
    live = G.cadd_verify_tree(yd, L, dev(n), dev(tok), dev(par), rows_mode=G.ROWS_LIVE)
    dense = G.cadd_verify_tree(yd, L, dev(n), dev(tok), dev(par), rows_mode=G.ROWS_DENSE)
    torch.cuda.synchronize()
    ov = O.verify_tree(y.contiguous(), L, n, tok, par, rows_mode=O.ROWS_LIVE)
    compare_verify(live, ov)
    la, da = to_cpu(live.node_argmax), to_cpu(dense.node_argmax)
    for b in range(batch):
        nb = int(n[b])
        assert torch.equal(la[b, : nb + 1], da[b, : nb + 1]) and bool((la[b, nb + 1:] == -1).all())
    assert torch.equal(to_cpu(live.accepted_len), to_cpu(dense.accepted_len))
    assert to_cpu(live.accepted_len).tolist() == [0, 4, 4, 4]
