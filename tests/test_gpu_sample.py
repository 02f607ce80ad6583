"""GPU parity of tree verification under sampling (one inverse-CDF draw per node from softmax(y / T), then the
accept walk with the drawn tokens) against the CPU oracle.

The drawn token is an integer decided by floating point: u * Z falls into the token's interval of the CDF.  Both
sides form the masses exp((y - max) / T) and sum them in token order, the oracle in fp64 throughout, the kernel with
fp32 ex2 terms per 2 KB run and fp64 sums.  The relative error of the kernel's CDF is below 1e-5 (fp32 rounding of
the scaled exponent, <= 2^-24 * 150, times the approximation error of ex2), so a row whose uniform lies within
MARGIN = 1e-5 of an interval end may resolve to the neighbouring token with mass; every other row is bit-exact.
The walk is checked for every request on the tokens the kernel drew (bit-exact)."""
import math

import numpy as np
import pytest
import torch

from oracle import cadd_oracle as O
from paper_2606_01813_b200 import binding as G
from paper_2606_01813_b200 import synth

pytestmark = pytest.mark.gpu

MARGIN = 1e-5


def neighbour_with_mass(row: torch.Tensor, tok: int, step: int) -> int:
    """Next token in direction `step` whose logit is finite (carries mass), or -1."""
    v = tok + step
    while 0 <= v < row.numel():
        if math.isfinite(float(row[v])):
            return v
        v += step
    return -1


def compare_sampled(gv, y_cpu, u_cpu, L, n, tok, par, rows_mode, T, max_exempt=0):
    ov, mg = O.verify_tree_sampled(y_cpu, u_cpu, L, n, tok, par, rows_mode, T)
    got = gv.node_argmax.cpu()
    exempt = 0
    batch, R, _ = y_cpu.shape
    for b in range(batch):
        for j in range(R):
            g, o = int(got[b, j]), int(ov.node_argmax[b, j])
            if g == o:
                continue
            assert o >= 0 and float(mg[b, j]) < MARGIN, f"row ({b},{j}): drew {g}, oracle {o}, margin {float(mg[b, j]):.3e}"
            assert g in (neighbour_with_mass(y_cpu[b, j], o, -1), neighbour_with_mass(y_cpu[b, j], o, +1))
            exempt += 1
    assert exempt <= max_exempt, f"{exempt} rows at a CDF boundary"
    check_walk(gv, L, n, tok, par)
    if exempt == 0:
        for f in ("accepted_len", "accepted_nodes", "next_bonus", "status"):
            assert torch.equal(getattr(gv, f).cpu(), getattr(ov, f)), f
    return ov


def check_walk(gv, L, n, tok, par):
    """The walk on the tokens the kernel drew, against the oracle's walk on the same tokens."""
    got = gv.node_argmax.cpu()
    al, an, nb = gv.accepted_len.cpu(), gv.accepted_nodes.cpu(), gv.next_bonus.cpu()
    R = got.shape[1]
    for b in range(got.shape[0]):
        nn = min(max(int(n[b]), 0), R - 1)
        acc, nxt = O.accept_walk(L, nn, tok[b], par[b], got[b])
        assert int(al[b]) == len(acc) and int(nb[b]) == nxt, f"request {b}"
        assert an[b].tolist() == acc + [-1] * (L - len(acc)), f"request {b}"


def random_tree(g, batch, R, V, hot):
    """Random parent arrays; child tokens drawn among the `hot` most likely tokens so that matches happen."""
    par = torch.zeros(batch, R, dtype=torch.int32)
    for c in range(1, R):
        par[:, c] = torch.randint(0, c, (batch,), generator=g, dtype=torch.int32)
    tok = hot[torch.randint(0, hot.numel(), (batch, R), generator=g)].to(torch.int32)
    n = torch.randint(0, R, (batch,), generator=g, dtype=torch.int32)
    return n, tok, par


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("V", [1, 7, 1000, 4097, 20000, 151936])
def test_sampled_small(dtype, V):
    g = torch.Generator().manual_seed(V)
    batch, R, L = 3, 9, 4
    y = (torch.randn(batch, R, V, generator=g) * 2.5).to(dtype)
    hot = torch.arange(min(V, 6))
    y[..., : hot.numel()] += 6.0                      # a handful of likely tokens
    n, tok, par = random_tree(g, batch, R, V, hot)
    u = torch.rand(batch, R, generator=g, dtype=torch.float64)
    for rows_mode in (G.ROWS_LIVE, G.ROWS_DENSE):
        for T in (0.6, 1.0, 1.4):
            gv = G.cadd_verify_tree_sampled(y.cuda(), u.cuda(), L, n.cuda(), tok.cuda(), par.cuda(), rows_mode, temperature=T)
            torch.cuda.synchronize()
            compare_sampled(gv, y, u, L, n, tok, par, rows_mode, T)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_sampled_unaligned_rows_and_strides(dtype):
    """Rows that start off a 16-byte boundary (scalar head and tail elements) inside a wider buffer."""
    g = torch.Generator().manual_seed(77)
    batch, R, V, L = 2, 5, 5003, 3
    big = (torch.randn(batch, R + 1, V + 13, generator=g) * 3.0).to(dtype)
    y = big[:, 1:, 3: 3 + V]
    hot = torch.tensor([0, 1, V // 2, V - 2, V - 1])
    y[..., hot] += 7.0
    n, tok, par = random_tree(g, batch, R, V, hot)
    u = torch.rand(batch, R, generator=g, dtype=torch.float64)
    yd = big.cuda()[:, 1:, 3: 3 + V]
    gv = G.cadd_verify_tree_sampled(yd, u.cuda(), L, n.cuda(), tok.cuda(), par.cuda(), G.ROWS_DENSE, temperature=0.9)
    torch.cuda.synchronize()
    ov = compare_sampled(gv, y.contiguous(), u, L, n, tok, par, G.ROWS_DENSE, 0.9)
    assert set(ov.node_argmax.flatten().tolist()) & {0, 1, V - 2, V - 1}      # head and tail runs were drawn from


def test_sampled_edge_cases():
    V, R, L = 3000, 6, 3
    y = torch.zeros(1, R, V, dtype=torch.float32)
    y[0, 0, 5] = 2000.0                                # all the mass on one token
    y[0, 1] = float("nan")                             # nothing finite: token 0
    y[0, 2, :] = float("-inf")
    y[0, 2, 2999] = 0.0                                # the only finite value is the last
    y[0, 3, 100:] = float("-inf")                      # mass on the first hundred tokens only
    y[0, 4, 7] = float("inf")                          # +Inf carries no mass; the rest is uniform
    u = torch.tensor([[0.0, 0.5, 1.0 - 2.0 ** -53, 1.0 - 2.0 ** -53, 0.0, 0.5]], dtype=torch.float64)
    n = torch.tensor([5], dtype=torch.int32)
    tok = torch.tensor([[0, 5, 0, 2999, 99, 0]], dtype=torch.int32)
    par = torch.tensor([[0, 0, 1, 1, 3, 4]], dtype=torch.int32)
    gv = G.cadd_verify_tree_sampled(y.cuda(), u.cuda(), L, n.cuda(), tok.cuda(), par.cuda(), G.ROWS_DENSE)
    torch.cuda.synchronize()
    assert gv.node_argmax.cpu().tolist() == [[5, 0, 2999, 99, 0, 1500]]
    compare_sampled(gv, y, u, L, n, tok, par, G.ROWS_DENSE, 1.0)
    assert int(gv.accepted_len[0]) == 2 and int(gv.next_bonus[0]) == 2999      # root -> row 1 (token 5) -> row 2 (token 0)
    # a cold temperature reproduces greedy verification, whatever the uniforms
    g = torch.Generator().manual_seed(3)
    y = (torch.randn(2, R, V, generator=g) * 3).to(torch.bfloat16).float()
    y.scatter_add_(2, y.argmax(-1, keepdim=True), torch.ones(2, R, 1))      # a clear winner in every row
    u = torch.rand(2, R, generator=g, dtype=torch.float64)
    n = torch.tensor([5, 3], dtype=torch.int32)
    tok = y.argmax(-1).to(torch.int32).roll(1, dims=1)                    # row j carries the arg-max of row j-1: a chain
    par = torch.tensor([[0, 0, 1, 2, 3, 4]] * 2, dtype=torch.int32)
    cold = G.cadd_verify_tree_sampled(y.cuda(), u.cuda(), L, n.cuda(), tok.cuda(), par.cuda(), G.ROWS_LIVE, temperature=1e-3)
    ref = G.cadd_verify_tree(y.cuda(), L, n.cuda(), tok.cuda(), par.cuda(), G.ROWS_LIVE)
    torch.cuda.synchronize()
    for f in ("node_argmax", "accepted_len", "accepted_nodes", "next_bonus"):
        assert torch.equal(getattr(cold, f), getattr(ref, f)), f
    assert cold.accepted_len.tolist() == [3, 3]


def test_sampled_rejects_bad_arguments():
    y = torch.zeros(1, 2, 8, dtype=torch.float32, device="cuda")
    u = torch.zeros(1, 2, dtype=torch.float64, device="cuda")
    i = lambda *s: torch.zeros(*s, dtype=torch.int32, device="cuda")
    with pytest.raises(G.CaddError):
        G.cadd_verify_tree_sampled(y, u, 1, i(1), i(1, 2), i(1, 2), temperature=0.0)
    with pytest.raises(G.CaddError):
        G.cadd_verify_tree_sampled(y, u, 1, i(1), i(1, 2), i(1, 2), temperature=float("nan"))
    with pytest.raises(ValueError):
        G.cadd_verify_tree_sampled(y, u.float(), 1, i(1), i(1, 2), i(1, 2))
    with pytest.raises(ValueError):
        G.cadd_verify_tree_sampled(y.cpu(), u, 1, i(1), i(1, 2), i(1, 2))


def test_sampled_frequencies_on_a_uniform_grid():
    """A property that holds at any size: over the equispaced uniforms (i + 1/2) / N the kernel returns token v
    N * p_v times up to the interval ends (one grid point each, plus the CDF's rounding)."""
    from scipy.special import softmax
    g = torch.Generator().manual_seed(31)
    V, N, T = 3001, 4096, 1.2
    row = torch.randn(V, generator=g) * 2.0
    row[:20] += 5.0
    y = row.expand(N, V).contiguous().view(1, N, V)
    u = ((torch.arange(N, dtype=torch.float64) + 0.5) / N).view(1, N)
    i = lambda *s: torch.zeros(*s, dtype=torch.int32, device="cuda")
    gv = G.cadd_verify_tree_sampled(y.cuda(), u.cuda(), 1, i(1), i(1, N), i(1, N), G.ROWS_DENSE, temperature=T)
    torch.cuda.synchronize()
    drawn = gv.node_argmax.cpu().view(-1)
    assert bool((drawn[1:] >= drawn[:-1]).all())                       # monotone in u
    counts = np.bincount(drawn.numpy(), minlength=V)
    p = softmax(row.double().numpy() / T)
    assert np.abs(counts - N * p).max() <= 1.0 + 0.05


def test_sampled_full_size_config2():
    """Configuration 2's verification tensor (32 x 257 rows of 151936 bf16 logits, dense), as bench.py launches it:
    the oracle re-draws a seeded sample of rows one by one and re-walks every request on the kernel's tokens."""
    cfg = synth.CONFIGS["c2"]
    seed = synth.config_seed(cfg)
    d = synth.make_draft_inputs(cfg, seed, device="cuda")
    c = synth.make_cost_inputs(cfg, seed)
    gt = G.cadd_build_tree(d.logits, cfg.K, cfg.B_max, cfg.R, l_eff=d.l_eff, bonus_token=d.bonus_token, ctx_len=d.ctx_len,
                           cost_kind=G.COST_QUADRATIC, cost_coef=c.coef)
    torch.cuda.synchronize()
    y = synth.make_target_logits(cfg, seed, d, gt.depth, device="cuda")
    gu = torch.Generator().manual_seed(seed + 1)
    u = torch.rand(cfg.batch, cfg.R, generator=gu, dtype=torch.float64)
    T = 1.0
    gv = G.cadd_verify_tree_sampled(y, u.cuda(), cfg.L, gt.n_nodes, gt.token_ids, gt.parent_idx, G.ROWS_DENSE, temperature=T)
    torch.cuda.synchronize()
    drawn = gv.node_argmax.cpu()
    assert int(drawn.min()) >= 0 and int(drawn.max()) < cfg.V
    check_walk(gv, cfg.L, gt.n_nodes.cpu(), gt.token_ids.cpu(), gt.parent_idx.cpu())
    rng = np.random.default_rng(seed)
    total = cfg.batch * cfg.R
    picks = rng.choice(total, size=160, replace=False)
    rows = y.view(total, cfg.V)[torch.from_numpy(picks).cuda()].cpu()
    near = 0
    for k, r in enumerate(picks):
        o, mg = O.row_sample(rows[k], float(u.view(-1)[r]), T)
        g_tok = int(drawn.view(-1)[r])
        if g_tok != o:
            assert mg < MARGIN and abs(g_tok - o) == 1, f"row {int(r)}: drew {g_tok}, oracle {o}, margin {mg:.3e}"
            near += 1
    assert near <= 1
    # the planted target tokens take most of the mass: acceptance must be far above chance and below greedy + noise
    al = gv.accepted_len.cpu()
    assert int(al.min()) >= 0 and bool((al <= d.l_eff.cpu()).all())
    print(f"sampled c2: accepted mean {al.float().mean():.2f}; boundary rows in the sample {near}")
