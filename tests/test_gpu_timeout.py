"""The bounded waits of the streaming kernels, exercised in a form that cannot hang or fault a GPU: with the test flag
of the C ABI the copy of one tile per row is never issued and the wait for that tile alone gives up after a few tries;
nothing is in flight for the barrier that is given up on, copies into the other ring stages are waited for before the
CTA leaves, and the context stays usable.  Each streaming kernel must report CADD_STATUS_INTERNAL_TIMEOUT, and nothing
else, with the empty tree (build) or an empty accepted path (verification); the very next ordinary call must be exact."""
import pytest
import torch

from oracle import cadd_oracle as O
from paper_2606_01813_b200 import binding as G
from paper_2606_01813_b200 import synth
from parity_util import compare_build, compare_verify, to_cpu

pytestmark = pytest.mark.gpu


def _inputs(V=60000, batch=3, seed=5):
    cfg = synth.scaled(synth.CONFIGS["c2"], batch=batch, V=V)          # several 16 KB tiles per row
    d = synth.make_draft_inputs(cfg, seed)
    c = synth.make_cost_inputs(cfg, seed)
    kw = dict(l_eff=d.l_eff, bonus_token=d.bonus_token, ctx_len=d.ctx_len, cost_coef=c.coef)
    return cfg, d, kw


@pytest.mark.parametrize("V", [60000, 5000])                            # many tiles per row / a single tile per row
def test_softmax_topk_wait_runs_out(V):
    cfg, d, kw = _inputs(V)
    x = d.logits.cuda()
    bad = G.cadd_build_tree(x, cfg.K, cfg.B_max, cfg.R, flags=G.FLAG_TEST_DROP_TILE | G.FLAG_EMIT_TOPK, **kw)
    torch.cuda.synchronize()
    st = to_cpu(bad.status)
    assert [int(v) for v in st] == [G.STATUS_INTERNAL_TIMEOUT] * cfg.batch
    assert to_cpu(bad.n_nodes).tolist() == [0] * cfg.batch
    assert int(to_cpu(bad.token_ids)[:, 1:].max()) == -1 and int(to_cpu(bad.parent_idx)[:, 1:].max()) == -1
    assert to_cpu(bad.token_ids)[:, 0].tolist() == d.bonus_token.tolist()          # the root row is still emitted
    # the context is intact: the same call without the flag is exact
    good = G.cadd_build_tree(x, cfg.K, cfg.B_max, cfg.R, flags=G.FLAG_EMIT_TOPK, **kw)
    torch.cuda.synchronize()
    ot = O.build_tree(d.logits, cfg.K, cfg.B_max, cfg.R, **kw)
    assert compare_build(good, ot, cfg.K)["exempt"] == []


@pytest.mark.parametrize("rows_mode", [G.ROWS_DENSE, G.ROWS_LIVE])
def test_row_argmax_wait_runs_out(rows_mode):
    cfg, d, kw = _inputs()
    ot = O.build_tree(d.logits, cfg.K, cfg.B_max, cfg.R, flags=O.FLAG_FIXED_BUDGET, **kw)
    y = synth.make_target_logits(cfg, 5, d, ot.depth)
    yd, dev = y.cuda(), (lambda t: t.cuda())
    args = (yd, cfg.L, dev(ot.n_nodes), dev(ot.token_ids), dev(ot.parent_idx), rows_mode)
    bad = G.cadd_verify_tree(*args, flags=G.FLAG_TEST_DROP_TILE)
    torch.cuda.synchronize()
    assert [int(v) for v in to_cpu(bad.status)] == [G.STATUS_INTERNAL_TIMEOUT] * cfg.batch
    assert to_cpu(bad.accepted_len).tolist() == [0] * cfg.batch
    assert int(to_cpu(bad.accepted_nodes).max()) == -1
    am = to_cpu(bad.node_argmax)
    for b in range(cfg.batch):                                           # every row that was read is marked as not decided
        n = int(ot.n_nodes[b])
        live = cfg.R if rows_mode == G.ROWS_DENSE else n + 1
        assert am[b, :live].tolist() == [-2] * live and am[b, live:].tolist() == [-1] * (cfg.R - live)
    good = G.cadd_verify_tree(*args)
    torch.cuda.synchronize()
    compare_verify(good, O.verify_tree(y, cfg.L, ot.n_nodes, ot.token_ids, ot.parent_idx, rows_mode))


@pytest.mark.parametrize("rows_mode", [G.ROWS_DENSE, G.ROWS_LIVE])
def test_row_sample_wait_runs_out(rows_mode):
    cfg, d, kw = _inputs()
    ot = O.build_tree(d.logits, cfg.K, cfg.B_max, cfg.R, flags=O.FLAG_FIXED_BUDGET, **kw)
    y = synth.make_target_logits(cfg, 5, d, ot.depth)
    u = torch.rand(cfg.batch, cfg.R, dtype=torch.float64, generator=torch.Generator().manual_seed(2))
    dev = lambda t: t.cuda()
    args = (y.cuda(), u.cuda(), cfg.L, dev(ot.n_nodes), dev(ot.token_ids), dev(ot.parent_idx), rows_mode)
    bad = G.cadd_verify_tree_sampled(*args, flags=G.FLAG_TEST_DROP_TILE)
    torch.cuda.synchronize()
    assert [int(v) for v in to_cpu(bad.status)] == [G.STATUS_INTERNAL_TIMEOUT] * cfg.batch
    assert to_cpu(bad.accepted_len).tolist() == [0] * cfg.batch
    good = G.cadd_verify_tree_sampled(*args)
    again = G.cadd_verify_tree_sampled(*args)
    torch.cuda.synchronize()
    assert int(to_cpu(good.status).max()) == 0 and int(to_cpu(good.node_argmax).max()) >= 0
    assert torch.equal(good.node_argmax, again.node_argmax) and torch.equal(good.accepted_len, again.accepted_len)
