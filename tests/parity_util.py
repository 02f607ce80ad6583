"""Element-by-element comparison of the CUDA path with the CPU oracle on the same inputs.

Acceptance bar: token ids, parent indices, depths, chosen budget n*, masks, positions, status bits,
top-K token ids, per-node argmax, accepted length / path and next bonus are bit-exact.  Probabilities
(exp of log-probs), expected acceptance Phi and throughput theta match within 1e-5 relative.
The only exemption: where the ORACLE's own competing scores (or throughputs at the stopping test)
differ by less than 1e-6 relative, a different choice is admissible; such requests are counted,
reported and compared on expected acceptance instead."""
from __future__ import annotations

import numpy as np
import torch

from oracle import cadd_oracle as O
from paper_2606_01813_b200 import binding as G

REL_TOL = 1e-5          # probabilities, Phi, theta
NEAR_TIE = 1e-6         # oracle margin below which a different decision is admissible
LOGZ_TOL = 2e-7         # |log Z_gpu - log Z_oracle| bound checked by the parity tests


def to_cpu(t):
    return None if t is None else t.detach().cpu()


def compare_build(gt: G.Tree, ot: O.OracleTree, K: int, check_topk: bool = True, rel_tol: float = None, near_tie: float = None):
    """Returns a dict of diagnostics; raises AssertionError on a parity failure.  rel_tol / near_tie override the
    module's bars for paths whose logits themselves carry a stated rounding error (the fused output projection)."""
    REL_TOL_ = REL_TOL if rel_tol is None else rel_tol
    NEAR_TIE_ = NEAR_TIE if near_tie is None else near_tie
    n_g, n_o = to_cpu(gt.n_nodes).numpy(), ot.n_nodes.numpy()
    batch, R = ot.token_ids.shape
    tok_g, par_g, dep_g = to_cpu(gt.token_ids).numpy(), to_cpu(gt.parent_idx).numpy(), to_cpu(gt.depth).numpy()
    tok_o, par_o, dep_o = ot.token_ids.numpy(), ot.parent_idx.numpy(), ot.depth.numpy()
    lp_g, lp_o = to_cpu(gt.node_logprob).numpy(), ot.node_logprob.numpy()
    phi_g, phi_o = to_cpu(gt.phi).numpy(), ot.phi.numpy()
    th_g, th_o = to_cpu(gt.theta).numpy(), ot.theta.numpy()
    st_g, st_o = to_cpu(gt.status).numpy(), ot.status.numpy()
    pos_g, pos_o = to_cpu(gt.position_ids).numpy(), ot.position_ids.numpy()
    mb_g, mb_o = to_cpu(gt.mask_bits).numpy(), ot.mask_bits.numpy()
    exempt = []
    for b in range(batch):
        same_n = n_g[b] == n_o[b]
        k = min(n_g[b], n_o[b]) + 1
        same_rows = (np.array_equal(tok_g[b, :k], tok_o[b, :k]) and np.array_equal(par_g[b, :k], par_o[b, :k])
                     and np.array_equal(dep_g[b, :k], dep_o[b, :k]))
        if same_n and same_rows:
            assert np.array_equal(tok_g[b], tok_o[b]) and np.array_equal(par_g[b], par_o[b]) and np.array_equal(dep_g[b], dep_o[b]), f"padding rows differ (request {b})"
            assert st_g[b] == st_o[b], f"status differs (request {b}): gpu {st_g[b]} oracle {st_o[b]}"
            assert np.array_equal(pos_g[b], pos_o[b]), f"position ids differ (request {b})"
            assert np.array_equal(mb_g[b], mb_o[b]), f"mask differs (request {b})"
            np.testing.assert_allclose(np.exp(lp_g[b]), np.exp(lp_o[b]), rtol=REL_TOL_, err_msg=f"node prob (request {b})")
        else:
            # admissible only if the oracle's own decision at the first difference was a near-tie
            if not same_rows:
                j = next(j for j in range(k) if (tok_g[b, j], par_g[b, j], dep_g[b, j]) != (tok_o[b, j], par_o[b, j], dep_o[b, j]))
                margin = float(ot.pop_gap[b, j])
                what = f"pop {j}"
            else:
                margin = float(ot.stop_gap[b])
                what = "stop test"
            assert margin < NEAR_TIE_, (f"request {b}: trees differ at {what} but the oracle's margin there is "
                                       f"{margin:.3e} >= {NEAR_TIE_}")
            exempt.append((b, what, margin))
        np.testing.assert_allclose(phi_g[b], phi_o[b], rtol=REL_TOL_, err_msg=f"Phi (request {b})")
        np.testing.assert_allclose(th_g[b], th_o[b], rtol=REL_TOL_, err_msg=f"theta (request {b})")
    diag = {"exempt": exempt, "max_logprob_err": float(np.max(np.abs(np.where(tok_o >= 0, lp_g - lp_o, 0.0)))) if not exempt else None}
    if check_topk and gt.topk_token is not None:
        tt_g, tt_o = to_cpu(gt.topk_token).numpy(), ot.topk_token.numpy()
        assert np.array_equal(tt_g, tt_o), "top-K token ids differ"
        tl_g, tl_o = to_cpu(gt.topk_logprob).numpy(), ot.topk_logprob.numpy()
        fin = np.isfinite(tl_o)
        assert np.array_equal(np.isfinite(tl_g), fin)
        err = np.abs(tl_g[fin] - tl_o[fin])
        diag["max_logZ_err"] = float(err.max()) if err.size else 0.0
        np.testing.assert_allclose(np.exp(tl_g[fin]), np.exp(tl_o[fin]), rtol=REL_TOL_)
    return diag


def compare_verify(gv: G.Verdict, ov: O.OracleVerify):
    for name in ("node_argmax", "accepted_len", "accepted_nodes", "next_bonus", "status"):
        g, o = to_cpu(getattr(gv, name)).numpy(), getattr(ov, name).numpy()
        assert np.array_equal(g, o), f"{name} differs: {np.argwhere(g != o)[:5].tolist()}"


def run_both_build(x_cpu, K, B_max, R=None, device="cuda", **kw):
    """Run oracle (CPU) and CUDA path on the same bits; returns (gpu_tree, oracle_tree)."""
    flags = kw.pop("flags", 0)
    ot = O.build_tree(x_cpu, K, B_max, R, flags=flags & O.FLAG_FIXED_BUDGET, dense_mask=bool(flags & G.FLAG_EMIT_DENSE_MASK), **kw)
    gt = G.cadd_build_tree(x_cpu.to(device), K, B_max, R, flags=flags | G.FLAG_EMIT_TOPK, **kw)
    torch.cuda.synchronize()
    return gt, ot
