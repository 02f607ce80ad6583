"""ctypes wrapper around the plain-C fp64 oracle (cadd_oracle.c).

TEST INFRASTRUCTURE.  Only tests, the smoke check and the benchmark's CPU-baseline leg may use
this module; the product path (the package and its CUDA library) never does.  Inputs are torch
CPU tensors; outputs are torch CPU tensors allocated here.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cadd_oracle.c")
_LIB = os.path.join(_HERE, "libcadd_oracle.so")

DT_BF16, DT_FP32 = 0, 1
COST_QUADRATIC, COST_TABLE, COST_TABLE_INTERP = 0, 1, 2
FLAG_FIXED_BUDGET = 4
ROWS_LIVE, ROWS_DENSE = 0, 1
ST_NONFINITE, ST_FEWER_THAN_K, ST_CAP_HIT, ST_FRONTIER_EXHAUSTED = 1, 2, 4, 8
ST_L_EFF_CLAMPED, ST_COST_NONPOSITIVE, ST_BAD_N_NODES = 16, 32, 64
ST_BAD_TABLE_IDX = 256


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, -O2, OpenMP over requests)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                               "-ffp-contract=off", "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.cadd_oracle_row_argmax.restype = C.c_int32
    return _lib


def num_threads() -> int:
    return int(lib().cadd_oracle_num_threads())


def set_num_threads(n: int) -> None:
    """Threads the oracle's per-request loops use from now on (for timing the same code on one core)."""
    lib().cadd_oracle_set_num_threads(int(n))


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return DT_BF16
    if t.dtype == torch.float32:
        return DT_FP32
    raise TypeError(f"unsupported logits dtype {t.dtype}")


def _p(t: Optional[torch.Tensor]):
    return C.c_void_p(0 if t is None else t.data_ptr())


@dataclass
class OracleTree:
    n_nodes: torch.Tensor
    token_ids: torch.Tensor
    parent_idx: torch.Tensor
    depth: torch.Tensor
    position_ids: torch.Tensor
    node_logprob: torch.Tensor
    phi: torch.Tensor
    theta: torch.Tensor
    mask_bits: torch.Tensor
    mask_dense: Optional[torch.Tensor]
    topk_token: torch.Tensor
    topk_logprob: torch.Tensor
    status: torch.Tensor
    logZ: torch.Tensor
    pop_gap: torch.Tensor
    stop_gap: torch.Tensor
    theta_curve: torch.Tensor
    node_rank: torch.Tensor


def row_softmax_topk(row: torch.Tensor, K: int):
    """O1+O2 for one row: returns (m, logZ, tok[K], a[K], lp[K], k_eff, nonfinite, has_pinf)."""
    assert row.dim() == 1 and row.is_contiguous() and row.device.type == "cpu"
    tok = torch.empty(K, dtype=torch.int32)
    a = torch.empty(K, dtype=torch.float64)
    lp = torch.empty(K, dtype=torch.float64)
    m, lz = C.c_double(), C.c_double()
    ke, nf, pinf = C.c_int32(), C.c_int32(), C.c_int32()
    lib().cadd_oracle_row_softmax_topk(_p(row), _dt(row), C.c_int64(row.numel()), K,
                                       C.byref(m), C.byref(lz), _p(tok), _p(a), _p(lp),
                                       C.byref(ke), C.byref(nf), C.byref(pinf))
    return m.value, lz.value, tok, a, lp, ke.value, nf.value, pinf.value


def build_tree(draft_logits: torch.Tensor, K: int, B_max: int, R: Optional[int] = None, *,
               l_eff=None, bonus_token=None, ctx_len=None,
               cost_kind: int = COST_QUADRATIC, cost_coef=None, cost_table=None, table_idx=None,
               t_draft=None, ctx_grid=None, flags: int = 0, dense_mask: bool = False) -> OracleTree:
    """O1-O4 for a batch of requests; draft_logits is a CPU tensor [batch, L, V] (V contiguous)."""
    x = draft_logits
    assert x.device.type == "cpu" and x.dim() == 3 and x.stride(2) == 1
    batch, L, V = x.shape
    R = B_max + 1 if R is None else R
    W = (R + 31) // 32
    i32 = lambda *s: torch.empty(*s, dtype=torch.int32)
    f64 = lambda *s: torch.empty(*s, dtype=torch.float64)
    out = OracleTree(
        n_nodes=i32(batch), token_ids=i32(batch, R), parent_idx=i32(batch, R), depth=i32(batch, R),
        position_ids=i32(batch, R), node_logprob=f64(batch, R), phi=f64(batch), theta=f64(batch),
        mask_bits=torch.empty(batch, R, W, dtype=torch.int32),
        mask_dense=torch.empty(batch, R, R, dtype=torch.uint8) if dense_mask else None,
        topk_token=i32(batch, L, K), topk_logprob=f64(batch, L, K), status=i32(batch),
        logZ=f64(batch, L), pop_gap=f64(batch, R), stop_gap=f64(batch), theta_curve=f64(batch, R),
        node_rank=i32(batch, R))
    cv = lambda t, dt: None if t is None else t.to("cpu", dt).contiguous()
    l_eff, bonus_token, ctx_len = cv(l_eff, torch.int32), cv(bonus_token, torch.int32), cv(ctx_len, torch.int32)
    cost_coef, cost_table = cv(cost_coef, torch.float64), cv(cost_table, torch.float64)
    table_idx, t_draft = cv(table_idx, torch.int32), cv(t_draft, torch.float64)
    ctx_grid = cv(ctx_grid, torch.int32)
    n_tables = 0 if cost_table is None else int(cost_table.shape[0])
    if cost_kind == COST_TABLE_INTERP:
        assert cost_table is not None and ctx_grid is not None and t_draft is not None
        assert cost_table.shape[1] == B_max + 1 and ctx_grid.numel() == n_tables
        assert bool((ctx_grid[1:] > ctx_grid[:-1]).all())
    elif cost_kind == COST_TABLE:
        assert cost_table is not None and table_idx is not None and t_draft is not None
        assert cost_table.shape[1] == B_max + 1
    else:
        assert cost_coef is not None and tuple(cost_coef.shape) == (batch, 4)
    rc = lib().cadd_oracle_build_tree(
        batch, L, C.c_int64(V), K, B_max, R, _dt(x), _p(x), C.c_int64(x.stride(0)), C.c_int64(x.stride(1)),
        _p(l_eff), _p(bonus_token), _p(ctx_len), cost_kind, _p(cost_coef), _p(cost_table), _p(table_idx),
        _p(t_draft), n_tables, _p(ctx_grid), C.c_uint32(flags),
        _p(out.n_nodes), _p(out.token_ids), _p(out.parent_idx), _p(out.depth), _p(out.position_ids),
        _p(out.node_logprob), _p(out.phi), _p(out.theta), _p(out.mask_bits), _p(out.mask_dense),
        _p(out.topk_token), _p(out.topk_logprob), _p(out.status),
        _p(out.logZ), _p(out.pop_gap), _p(out.stop_gap), _p(out.theta_curve), _p(out.node_rank))
    if rc != 0:
        raise ValueError(f"cadd_oracle_build_tree rejected its arguments (rc={rc})")
    return out


@dataclass
class OracleVerify:
    node_argmax: torch.Tensor
    accepted_len: torch.Tensor
    accepted_nodes: torch.Tensor
    next_bonus: torch.Tensor
    status: torch.Tensor


def row_argmax(row: torch.Tensor) -> int:
    assert row.dim() == 1 and row.is_contiguous() and row.device.type == "cpu"
    return int(lib().cadd_oracle_row_argmax(_p(row), _dt(row), C.c_int64(row.numel())))


def verify_tree(target_logits: torch.Tensor, L: int, n_nodes, token_ids, parent_idx,
                rows_mode: int = ROWS_LIVE) -> OracleVerify:
    """O5+O6 for a batch; target_logits is a CPU tensor [batch, R, V] (V contiguous)."""
    y = target_logits
    assert y.device.type == "cpu" and y.dim() == 3 and y.stride(2) == 1
    batch, R, V = y.shape
    n_nodes = n_nodes.to("cpu", torch.int32).contiguous()
    token_ids = token_ids.to("cpu", torch.int32).contiguous()
    parent_idx = parent_idx.to("cpu", torch.int32).contiguous()
    assert tuple(token_ids.shape) == (batch, R)
    out = OracleVerify(torch.empty(batch, R, dtype=torch.int32), torch.empty(batch, dtype=torch.int32),
                       torch.empty(batch, L, dtype=torch.int32), torch.empty(batch, dtype=torch.int32),
                       torch.empty(batch, dtype=torch.int32))
    rc = lib().cadd_oracle_verify_tree(
        batch, C.c_int64(V), R, L, _dt(y), _p(y), C.c_int64(y.stride(0)), C.c_int64(y.stride(1)), rows_mode,
        _p(n_nodes), _p(token_ids), _p(parent_idx),
        _p(out.node_argmax), _p(out.accepted_len), _p(out.accepted_nodes), _p(out.next_bonus), _p(out.status))
    if rc != 0:
        raise ValueError(f"cadd_oracle_verify_tree rejected its arguments (rc={rc})")
    return out


def head_logits(hidden_states: torch.Tensor, weight: torch.Tensor) -> torch.Tensor:
    """fp64 logits [batch, R, V] = hidden_states [batch, R, hidden] . weight [V, hidden]^T (Section 3.1), both bf16 on CPU."""
    h, w = hidden_states, weight
    assert h.device.type == "cpu" and w.device.type == "cpu" and h.dtype == torch.bfloat16 and w.dtype == torch.bfloat16
    assert h.dim() == 3 and w.dim() == 2 and h.shape[2] == w.shape[1]
    h, w = h.contiguous(), w.contiguous()
    batch, R, hidden = h.shape
    V = w.shape[0]
    out = torch.empty(batch, R, V, dtype=torch.float64)
    rc = lib().cadd_oracle_head_logits(C.c_int64(batch * R), C.c_int64(V), hidden, _p(h), C.c_int64(hidden), _p(w),
                                       C.c_int64(hidden), _p(out))
    if rc != 0:
        raise ValueError(f"cadd_oracle_head_logits rejected its arguments (rc={rc})")
    return out


def verify_tree_fused_head(hidden_states: torch.Tensor, weight: torch.Tensor, L: int, n_nodes, token_ids, parent_idx,
                           rows_mode: int = ROWS_LIVE):
    """O5+O6 on logits formed from hidden states and the output projection.  The decision is taken in the
    precision the GPU path reports its logits in (fp32): the exact fp64 dot products are rounded once to fp32,
    then the plain argmax (lowest id among equals) and the walk follow.  Returns (OracleVerify, fp64 logits)."""
    y64 = head_logits(hidden_states, weight)
    return verify_tree(y64.to(torch.float32), L, n_nodes, token_ids, parent_idx, rows_mode), y64


def build_tree_fused_head(hidden_states: torch.Tensor, weight: torch.Tensor, K: int, B_max: int, R: Optional[int] = None, **kw):
    """O1-O4 on draft logits formed from the drafter's hidden states [batch, L, hidden] and its output projection
    [V, hidden] (Eq. 1 with l_i = h_i . W^T).  The exact fp64 dot products are rounded once to fp32, the precision the
    GPU path holds its logits in, and handed to build_tree.  Returns (OracleTree, fp64 logits)."""
    y64 = head_logits(hidden_states, weight)
    return build_tree(y64.to(torch.float32), K, B_max, R, **kw), y64


def row_sample(row, u: float, temperature: float = 1.0):
    """One draw from softmax(row / temperature) by the inverse CDF in token order, given the uniform u in [0, 1):
    the smallest token v with  sum_{w <= v} e_w  >  u * sum_w e_w,  e_w = exp((y_w - max y) / temperature); NaN and
    infinite logits carry no mass; a row without a finite logit gives token 0.  Returns (token, margin): margin is
    the distance from u to the nearer end of the token's interval of the CDF, as a fraction of the total (rows whose
    margin is at rounding level may legitimately resolve to the neighbouring token in another summation order)."""
    import numpy as np
    y = torch.as_tensor(row).to(torch.float64).numpy()
    fin = np.isfinite(y)
    if not fin.any():
        return 0, 1.0
    e = np.where(fin, np.exp((np.where(fin, y, 0.0) - y[fin].max()) / float(temperature)), 0.0)
    cdf = np.cumsum(e)                       # ascending token order, fp64
    Z = float(cdf[-1])
    t = float(u) * Z
    v = int(np.searchsorted(cdf, t, side="right"))     # first index with cdf > t
    if v >= len(y):                          # u so close to 1 that u * Z rounds to Z: the last token with mass
        v = int(np.nonzero(e > 0)[0][-1])
    below = float(cdf[v - 1]) if v > 0 else 0.0
    margin = min(float(cdf[v]) - t, t - below if v > 0 and below > 0 else np.inf) / Z
    return v, float(margin)


def accept_walk(L: int, n: int, token_ids_b, parent_idx_b, node_token_b):
    """O6 for one request with the per-node target tokens given: from the root follow, at each node, the child
    (lowest row first) whose token equals the target's token at that node.  Returns (accepted rows, next token)."""
    cur, acc = 0, []
    while len(acc) < L:
        g = int(node_token_b[cur])
        child = next((c for c in range(1, n + 1) if int(parent_idx_b[c]) == cur and int(token_ids_b[c]) == g), -1)
        if child < 0:
            break
        acc.append(child)
        cur = child
    return acc, int(node_token_b[cur])


def verify_tree_sampled(target_logits: torch.Tensor, uniforms: torch.Tensor, L: int, n_nodes, token_ids, parent_idx,
                        rows_mode: int = ROWS_LIVE, temperature: float = 1.0):
    """Tree verification under sampling (the T > 0 setting of the paper's Section 5 tables; the tree variant is
    this repository's reading): the target's token at node j is ONE draw from softmax(y_j / T) at the supplied uniform
    uniforms[b, j] (row_sample); the walk is O6 with the drawn tokens in place of the arg-max.  The emitted tokens are
    distributed as the target's own sampling whatever the tree.  Returns (OracleVerify, margins [batch, R])."""
    y = target_logits
    assert y.device.type == "cpu" and y.dim() == 3
    batch, R, V = y.shape
    out = OracleVerify(torch.full((batch, R), -1, dtype=torch.int32), torch.zeros(batch, dtype=torch.int32),
                       torch.full((batch, L), -1, dtype=torch.int32), torch.zeros(batch, dtype=torch.int32),
                       torch.zeros(batch, dtype=torch.int32))
    margins = torch.full((batch, R), float("inf"), dtype=torch.float64)
    for b in range(batch):
        n = int(n_nodes[b])
        if n < 0 or n > R - 1:
            out.status[b] = ST_BAD_N_NODES
            n = min(max(n, 0), R - 1)
        for j in range(R):
            if j <= n or rows_mode == ROWS_DENSE:
                tok, mg = row_sample(y[b, j], float(uniforms[b, j]), temperature)
                out.node_argmax[b, j], margins[b, j] = tok, mg
        acc, nxt = accept_walk(L, n, token_ids[b], parent_idx[b], out.node_argmax[b])
        out.accepted_len[b] = len(acc)
        for i, c in enumerate(acc):
            out.accepted_nodes[b, i] = c
        out.next_bonus[b] = nxt
    return out, margins


def fit_convex_nondecreasing(y) -> "torch.Tensor":
    """Offline cost fitting (Eq. 12): for each row of y [n_tables, N] (latencies measured at N equally spaced node
    counts) the least-squares fit among all convex, non-decreasing sequences.

    Written out as the definition: a sequence f on points 0..N-1 is convex and non-decreasing iff
    f_i = a + sum_k beta_k * max(0, i - k) with beta_k >= 0 for k = 0..N-2 (beta_0 is the first slope, beta_k the
    slope increase at point k) and a free; the fit is therefore a non-negative least-squares problem in
    (a+, a-, beta), handed to the library's NNLS routine.  fp64 throughout."""
    import numpy as np
    from scipy.optimize import nnls
    y = torch.as_tensor(y, dtype=torch.float64)
    assert y.dim() == 2
    T, N = y.shape
    i = np.arange(N, dtype=np.float64)[:, None]
    k = np.arange(max(N - 1, 0), dtype=np.float64)[None, :]
    A = np.concatenate([np.ones((N, 1)), -np.ones((N, 1)), np.maximum(0.0, i - k)], axis=1)
    out = torch.empty_like(y)
    for t in range(T):
        coef, _ = nnls(A, y[t].numpy(), maxiter=50 * A.shape[1])
        out[t] = torch.from_numpy(A @ coef)
    return out
