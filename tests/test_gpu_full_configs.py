"""The five benchmark configurations at their full sizes, in the launch configuration bench.py times
(inputs generated on the device, buffers reused, dense verification).  Trees are compared with the
oracle for every request; per-node argmax and the accepted path are compared on every live row and on
every padding row for configurations 1 and 2, a seeded sample (>= 1 %) of them for the larger ones; the oracle
computes those one row at a time."""
import numpy as np
import pytest
import torch

from oracle import cadd_oracle as O
from paper_2606_01813_b200 import binding as G
from paper_2606_01813_b200 import synth
from parity_util import compare_build, to_cpu, LOGZ_TOL

pytestmark = pytest.mark.gpu


def cost_kwargs(c):
    if c.kind == synth.COST_TABLE:
        return dict(cost_kind=G.COST_TABLE, cost_table=c.table, table_idx=c.table_idx, t_draft=c.t_draft)
    return dict(cost_kind=G.COST_QUADRATIC, cost_coef=c.coef)


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4", "c4_stress", "c5"])
def test_full_size_round(name):
    cfg = synth.CONFIGS[name]
    seed = synth.config_seed(cfg)
    dev = "cuda"
    d = synth.make_draft_inputs(cfg, seed, device=dev)
    c = synth.make_cost_inputs(cfg, seed)
    flags = (G.FLAG_FIXED_BUDGET if cfg.fixed_budget else 0) | G.FLAG_EMIT_TOPK
    kw = dict(l_eff=d.l_eff, bonus_token=d.bonus_token, ctx_len=d.ctx_len, **cost_kwargs(c))
    gt = G.cadd_build_tree(d.logits, cfg.K, cfg.B_max, cfg.R, flags=flags, **kw)
    torch.cuda.synchronize()
    ot = O.build_tree(d.logits.cpu(), cfg.K, cfg.B_max, cfg.R, flags=flags & O.FLAG_FIXED_BUDGET, **kw)
    diag = compare_build(gt, ot, cfg.K)
    n = ot.n_nodes
    print(f"{name}: n* mean {n.float().mean():.1f} max {int(n.max())}; exempt {diag['exempt']}; "
          f"max |dlogZ| {diag['max_logZ_err']:.2e}")
    assert diag["exempt"] == [], f"requests decided inside the oracle's own rounding margin: {diag['exempt']}"
    assert diag["max_logZ_err"] < LOGZ_TOL
    if name == "c4_stress":
        assert int(n.min()) == cfg.B_max

    # ---- verification over the dense [batch, R, V] target tensor ----
    y = synth.make_target_logits(cfg, seed, d, ot.depth, device=dev)
    gv = G.cadd_verify_tree(y, cfg.L, gt.n_nodes, gt.token_ids, gt.parent_idx, G.ROWS_DENSE)
    torch.cuda.synchronize()
    # requests whose live rows the oracle re-verifies in full (all of them when the trees are small)
    live_rows = int((n + 1).sum())
    reqs = list(range(cfg.batch)) if live_rows <= 6000 else list(range(0, cfg.batch, max(1, cfg.batch // 3)))[:3]
    for b in reqs:
        rl = int(n[b]) + 1
        yb = y[b:b + 1, :rl].cpu()
        ov = O.verify_tree(yb, cfg.L, n[b:b + 1], ot.token_ids[b:b + 1, :rl], ot.parent_idx[b:b + 1, :rl], O.ROWS_LIVE)
        assert torch.equal(to_cpu(gv.node_argmax[b, :rl]), ov.node_argmax[0]), f"argmax, request {b}"
        assert int(gv.accepted_len[b]) == int(ov.accepted_len[0]), f"accepted_len, request {b}"
        assert torch.equal(to_cpu(gv.accepted_nodes[b]), ov.accepted_nodes[0]), f"accepted path, request {b}"
        assert int(gv.next_bonus[b]) == int(ov.next_bonus[0]), f"next bonus, request {b}"
    # configurations 1 and 2: every row of the dense tensor, live or padding; the larger ones: a seeded sample of
    # at least 1 % of all rows (one oracle argmax per row)
    rng = np.random.default_rng(seed)
    total = cfg.batch * cfg.R
    k = total if name in ("c1", "c2") else min(total, max(64, total // 100))
    picks = rng.choice(total, size=k, replace=False)
    rows = torch.from_numpy(picks).to(dev)
    sample = y.view(total, cfg.V)[rows].cpu()
    got = to_cpu(gv.node_argmax.view(total)[rows])
    for i in range(k):
        assert int(got[i]) == O.row_argmax(sample[i]), f"argmax of row {int(picks[i])}"
    # properties that hold at any size
    am = to_cpu(gv.node_argmax)
    assert int(am.min()) >= 0 and int(am.max()) < cfg.V
    al = to_cpu(gv.accepted_len)
    assert int(al.min()) >= 0 and bool((al <= d.l_eff).all())
    print(f"{name}: accepted mean {al.float().mean():.2f} max {int(al.max())}; sampled rows {k}")
