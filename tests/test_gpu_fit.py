"""GPU parity of the offline cost fitting (convex, non-decreasing least squares, Eq. 12) against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import cadd_oracle as O
from paper_2606_01813_b200 import binding as G
from paper_2606_01813_b200 import synth

pytestmark = pytest.mark.gpu

REL_TOL = 1e-5          # floating-point outputs: relative to the data's scale


def kkt_violation(y, f):
    """Feasibility, residual orthogonal to constants, <r, hinge_k> <= 0 with equality where the fit bends."""
    y, f = np.asarray(y, dtype=np.float64), np.asarray(f, dtype=np.float64)
    N = len(y)
    scale = max(1.0, float(np.abs(y).max()))
    r = y - f
    if N == 1:
        return abs(float(r[0])) / scale
    slopes = np.diff(f)
    bends = np.concatenate([slopes[:1], np.diff(slopes)])
    worst = max(0.0, float(-bends.min()) / scale, abs(float(r.sum())) / (scale * N))
    s1 = np.concatenate([np.cumsum(r[::-1])[::-1][1:], [0.0]])       # sum_{i>m} r_i
    w = np.cumsum(s1[::-1])[::-1][: N - 1]                           # sum_i max(0, i-k) r_i
    g = w / (scale * N * N)
    worst = max(worst, float(g.max()))
    active = bends > 1e-9 * scale
    if active.any():
        worst = max(worst, float(np.abs(g[active]).max()))
    return worst


def check(y: torch.Tensor, tol=REL_TOL):
    f_o = O.fit_convex_nondecreasing(y)
    f_g, nb, st = G.cadd_fit_cost_tables(y.cuda())
    torch.cuda.synchronize()
    f_g = f_g.cpu()
    assert int(st.max()) == 0
    scale = float(y.abs().max().clamp(min=1.0))
    assert float((f_g - f_o).abs().max()) <= tol * scale
    for t in range(y.shape[0]):
        assert kkt_violation(y[t].numpy(), f_g[t].numpy()) < 1e-9
    return f_g, nb.cpu()


def test_fit_latency_grids_full_size():
    """Nine context lengths x 1024 node counts, the shape of the paper's profiling grid: smooth convex latency
    curves (a step in marginal cost at 256 nodes, as in configuration 3's table) plus measurement noise."""
    g = torch.Generator().manual_seed(21)
    n = torch.arange(1, 1025, dtype=torch.float64)
    rows = []
    for j in range(9):
        base = 18.0 + 2.0 * j + (0.010 + 0.002 * j) * n + (2e-5 + 2e-6 * j) * n * n + 0.004 * torch.clamp(n - 256, min=0)
        rows.append(base + (0.2 + 0.05 * j) * torch.randn(1024, generator=g, dtype=torch.float64))
    y = torch.stack(rows)
    f, nb = check(y)
    assert int(nb.min()) >= 2 and int(nb.max()) < 200
    assert float(torch.diff(f, dim=1).min()) >= -1e-12 and float(torch.diff(f, n=2, dim=1).min()) >= -1e-9


@pytest.mark.parametrize("N", [1, 2, 3, 7, 64, 257, 1000, 2048])
def test_fit_sizes_and_special_cases(N):
    g = torch.Generator().manual_seed(N)
    n = torch.arange(N, dtype=torch.float64)
    y = torch.stack([
        1.0 + 0.3 * n + 0.01 * n * n,                                                  # convex already: recovered
        5.0 - 0.2 * n,                                                                 # falling: the mean
        torch.sqrt(n + 1.0),                                                           # concave: a line
        torch.cumsum(torch.randn(N, generator=g, dtype=torch.float64), 0),             # a random walk
        3.0 + torch.randn(N, generator=g, dtype=torch.float64) * 1e-3,                 # almost flat
        1e6 * (1.0 + 0.001 * n) + 10.0 * torch.randn(N, generator=g, dtype=torch.float64),   # large offset
    ])
    f, _ = check(y)
    # data that is convex already comes back (every point is a kink: the degenerate end of the active-set method)
    assert torch.allclose(f[0], y[0], rtol=0, atol=1e-6 * float(y[0].abs().max().clamp(min=1)))
    assert torch.allclose(f[1], torch.full_like(n, float(y[1].mean())), atol=1e-9)


def test_fitted_tables_drive_the_tree_builder():
    """Fit -> cost_table -> cadd_build_tree with context interpolation, against the same chain on the oracle side."""
    cfg = synth.scaled(synth.CONFIGS["c3"], batch=3, V=20000)
    d = synth.make_draft_inputs(cfg, 9)
    g = torch.Generator().manual_seed(2)
    n = torch.arange(cfg.B_max + 1, dtype=torch.float64)
    raw = torch.stack([1.0 + 0.2 * j + 0.0015 * n + 1e-5 * n * n + 0.01 * torch.randn(cfg.B_max + 1, generator=g, dtype=torch.float64)
                       for j in range(3)])
    fit_g, _, st = G.cadd_fit_cost_tables(raw.cuda())
    fit_o = O.fit_convex_nondecreasing(raw)
    assert int(st.max()) == 0 and float((fit_g.cpu() - fit_o).abs().max()) < 1e-8
    grid = torch.tensor([0, 4096, 8192], dtype=torch.int32)
    ctx = torch.tensor([100, 5000, 9000], dtype=torch.int32)
    t_draft = torch.full((cfg.batch,), 0.25, dtype=torch.float64)
    kw = dict(l_eff=d.l_eff, bonus_token=d.bonus_token, ctx_len=ctx, t_draft=t_draft, ctx_grid=grid)
    ot = O.build_tree(d.logits, cfg.K, cfg.B_max, cfg.R, cost_kind=O.COST_TABLE_INTERP, cost_table=fit_o, **kw)
    gt = G.cadd_build_tree(d.logits.cuda(), cfg.K, cfg.B_max, cfg.R, cost_kind=G.COST_TABLE_INTERP, cost_table=fit_g,
                           **{k: v.cuda() for k, v in kw.items()})
    torch.cuda.synchronize()
    assert torch.equal(gt.n_nodes.cpu(), ot.n_nodes)
    assert torch.equal(gt.token_ids.cpu(), ot.token_ids) and torch.equal(gt.parent_idx.cpu(), ot.parent_idx)


def test_fit_rejects_bad_arguments():
    with pytest.raises(ValueError):
        G.cadd_fit_cost_tables(torch.zeros(2, 8, dtype=torch.float32, device="cuda"))
    with pytest.raises(G.CaddError):
        G.cadd_fit_cost_tables(torch.zeros(1, 4096, dtype=torch.float64, device="cuda"))
