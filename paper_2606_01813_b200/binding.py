"""Thin ctypes binding of the C ABI in include/cadd.h.  Argument marshalling only: every step of the
path runs in the CUDA kernels of libcadd.so.  There is no CPU fallback: if the library is missing
or the tensors are not on a CUDA device the calls raise.

PyTorch is used for device memory and streams.  The functions carry the names of the C entry
points (cadd_build_tree, cadd_verify_tree, ...)."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcadd.so")

OK = 0
ERR_NULL, ERR_STRUCT_SIZE, ERR_SHAPE, ERR_DTYPE, ERR_ALIGN, ERR_WORKSPACE, ERR_LAUNCH = -1, -2, -3, -4, -5, -6, -7
STATUS_NONFINITE_INPUT, STATUS_FEWER_THAN_K_FINITE, STATUS_CAP_HIT, STATUS_FRONTIER_EXHAUSTED = 1, 2, 4, 8
STATUS_L_EFF_CLAMPED, STATUS_COST_NONPOSITIVE, STATUS_BAD_N_NODES, STATUS_INTERNAL_TIMEOUT = 16, 32, 64, 128
STATUS_BAD_TABLE_IDX = 256
DTYPE_BF16, DTYPE_FP32 = 0, 1
COST_QUADRATIC, COST_TABLE, COST_TABLE_INTERP = 0, 1, 2
FLAG_EMIT_DENSE_MASK, FLAG_EMIT_TOPK, FLAG_FIXED_BUDGET = 1, 2, 4
FLAG_ONLY_TOPK, FLAG_ONLY_EXPAND = 8, 16          # measurement aids: one of the two build kernels alone
VERIFY_ONLY_ARGMAX, VERIFY_ONLY_WALK = 1, 2       # the same for cadd_verify_tree
FLAG_TEST_DROP_TILE = 0x80000000                  # test hook: one tile per row is never copied, its wait gives up
FLAG_REGULAR_PATH, VERIFY_REGULAR_PATH = 32, 4    # small problems too take the two-kernel path
# Tests set this to run small shapes through the regular two-kernel path as well (it only adds the two flags above).
FORCE_REGULAR_PATH = False
ROWS_LIVE, ROWS_DENSE = 0, 1

EXPORTS = ("cadd_version", "cadd_status_string", "cadd_build_workspace_bytes", "cadd_verify_workspace_bytes",
           "cadd_build_tree", "cadd_verify_tree", "cadd_build_tree_static_scratch", "cadd_build_launches", "cadd_verify_launches",
           "cadd_head_workspace_bytes", "cadd_verify_tree_fused_head", "cadd_fit_cost_tables",
           "cadd_build_head_workspace_bytes", "cadd_build_tree_fused_head", "cadd_verify_tree_sampled")
ERR_STATIC_SCRATCH = -8
STATIC_SCRATCH_BYTES = 8 << 20


class BuildArgs(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("flags", C.c_uint32),
        ("batch", C.c_int32), ("L", C.c_int32), ("K", C.c_int32), ("B_max", C.c_int32), ("R", C.c_int32),
        ("logits_dtype", C.c_int32), ("V", C.c_int64),
        ("draft_logits", C.c_void_p), ("stride_b", C.c_int64), ("stride_l", C.c_int64),
        ("l_eff", C.c_void_p), ("bonus_token", C.c_void_p), ("ctx_len", C.c_void_p),
        ("cost_kind", C.c_int32), ("n_tables", C.c_int32),
        ("cost_coef", C.c_void_p), ("cost_table", C.c_void_p), ("table_idx", C.c_void_p), ("t_draft", C.c_void_p),
        ("ctx_grid", C.c_void_p),
        ("n_nodes", C.c_void_p), ("token_ids", C.c_void_p), ("parent_idx", C.c_void_p), ("depth", C.c_void_p),
        ("position_ids", C.c_void_p), ("node_logprob", C.c_void_p), ("phi", C.c_void_p), ("theta", C.c_void_p),
        ("theta_curve", C.c_void_p),
        ("mask_bits", C.c_void_p), ("mask_dense", C.c_void_p), ("topk_token", C.c_void_p),
        ("topk_logprob", C.c_void_p), ("status", C.c_void_p),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
    ]


class VerifyArgs(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("flags", C.c_uint32),
        ("batch", C.c_int32), ("L", C.c_int32), ("R", C.c_int32),
        ("logits_dtype", C.c_int32), ("rows_mode", C.c_int32), ("reserved0", C.c_int32), ("V", C.c_int64),
        ("target_logits", C.c_void_p), ("stride_b", C.c_int64), ("stride_row", C.c_int64),
        ("n_nodes", C.c_void_p), ("token_ids", C.c_void_p), ("parent_idx", C.c_void_p),
        ("node_argmax", C.c_void_p), ("accepted_len", C.c_void_p), ("accepted_nodes", C.c_void_p),
        ("next_bonus", C.c_void_p), ("status", C.c_void_p),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
    ]


class HeadArgs(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("flags", C.c_uint32),
        ("batch", C.c_int32), ("L", C.c_int32), ("R", C.c_int32), ("hidden", C.c_int32),
        ("rows_mode", C.c_int32), ("reserved0", C.c_int32), ("V", C.c_int64),
        ("hidden_states", C.c_void_p), ("stride_row", C.c_int64),
        ("weight", C.c_void_p), ("stride_w", C.c_int64),
        ("n_nodes", C.c_void_p), ("token_ids", C.c_void_p), ("parent_idx", C.c_void_p),
        ("node_argmax", C.c_void_p), ("accepted_len", C.c_void_p), ("accepted_nodes", C.c_void_p),
        ("next_bonus", C.c_void_p), ("status", C.c_void_p),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
    ]


class BuildHeadArgs(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("flags", C.c_uint32), ("hidden", C.c_int32), ("reserved0", C.c_int32),
        ("hidden_states", C.c_void_p), ("stride_row", C.c_int64), ("weight", C.c_void_p), ("stride_w", C.c_int64),
        ("build", BuildArgs),
    ]


class SampleArgs(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("flags", C.c_uint32),
        ("batch", C.c_int32), ("L", C.c_int32), ("R", C.c_int32),
        ("logits_dtype", C.c_int32), ("rows_mode", C.c_int32), ("reserved0", C.c_int32), ("V", C.c_int64),
        ("temperature", C.c_double),
        ("target_logits", C.c_void_p), ("stride_b", C.c_int64), ("stride_row", C.c_int64),
        ("uniforms", C.c_void_p),
        ("n_nodes", C.c_void_p), ("token_ids", C.c_void_p), ("parent_idx", C.c_void_p),
        ("node_token", C.c_void_p), ("accepted_len", C.c_void_p), ("accepted_nodes", C.c_void_p),
        ("next_bonus", C.c_void_p), ("status", C.c_void_p),
    ]


class FitArgs(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("flags", C.c_uint32), ("n_tables", C.c_int32), ("N", C.c_int32),
        ("y", C.c_void_p), ("fit", C.c_void_p), ("n_breaks", C.c_void_p), ("status", C.c_void_p),
    ]


_lib = None


def lib() -> C.CDLL:
    """The loaded C-ABI library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2606_01813_b200.build` "
                               "(there is no CPU fallback)")
        l = C.CDLL(LIB_PATH)
        l.cadd_version.restype = C.c_int
        l.cadd_status_string.restype = C.c_char_p
        l.cadd_status_string.argtypes = [C.c_int]
        l.cadd_build_workspace_bytes.argtypes = [C.POINTER(BuildArgs), C.POINTER(C.c_size_t)]
        l.cadd_verify_workspace_bytes.argtypes = [C.POINTER(VerifyArgs), C.POINTER(C.c_size_t)]
        l.cadd_build_tree.argtypes = [C.POINTER(BuildArgs), C.c_void_p]
        l.cadd_verify_tree.argtypes = [C.POINTER(VerifyArgs), C.c_void_p]
        l.cadd_head_workspace_bytes.argtypes = [C.POINTER(HeadArgs), C.POINTER(C.c_size_t)]
        l.cadd_verify_tree_fused_head.argtypes = [C.POINTER(HeadArgs), C.c_void_p]
        l.cadd_fit_cost_tables.argtypes = [C.POINTER(FitArgs), C.c_void_p]
        l.cadd_verify_tree_sampled.argtypes = [C.POINTER(SampleArgs), C.c_void_p]
        l.cadd_build_head_workspace_bytes.argtypes = [C.POINTER(BuildHeadArgs), C.POINTER(C.c_size_t)]
        l.cadd_build_tree_fused_head.argtypes = [C.POINTER(BuildHeadArgs), C.c_void_p]
        l.cadd_build_tree_static_scratch.argtypes = [C.POINTER(BuildArgs), C.c_void_p]
        l.cadd_build_launches.argtypes = [C.POINTER(BuildArgs)]
        l.cadd_verify_launches.argtypes = [C.POINTER(VerifyArgs)]
        _lib = l
    return _lib


class CaddError(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        super().__init__(f"cadd error {code}: {lib().cadd_status_string(code).decode()}")


def cadd_version() -> int:
    return int(lib().cadd_version())


def cadd_status_string(code: int) -> str:
    return lib().cadd_status_string(code).decode()


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return DTYPE_BF16
    if t.dtype == torch.float32:
        return DTYPE_FP32
    raise TypeError(f"unsupported logits dtype {t.dtype}")


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream_of(stream: Optional[torch.cuda.Stream], dev) -> torch.cuda.Stream:
    """The stream a call is enqueued on: the given one, else the current stream OF THE TENSORS' DEVICE (which need
    not be the current device).  The same object serves the C call and record_stream."""
    return torch.cuda.current_stream(dev) if stream is None else stream


def _dev(t: Optional[torch.Tensor], device, dtype) -> Optional[torch.Tensor]:
    if t is None:
        return None
    return t.to(device=device, dtype=dtype).contiguous()


@dataclass
class Tree:
    """Outputs of cadd_build_tree (device tensors)."""
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
    topk_token: Optional[torch.Tensor]
    topk_logprob: Optional[torch.Tensor]
    status: torch.Tensor
    theta_curve: Optional[torch.Tensor] = None


@dataclass
class Verdict:
    """Outputs of cadd_verify_tree (device tensors)."""
    node_argmax: torch.Tensor
    accepted_len: torch.Tensor
    accepted_nodes: torch.Tensor
    next_bonus: torch.Tensor
    status: torch.Tensor


def _build_args(x, K, B_max, R, flags, cost_kind) -> BuildArgs:
    a = BuildArgs()
    a.struct_size = C.sizeof(BuildArgs)
    a.flags = flags
    a.batch, a.L, a.V = x.shape
    a.K, a.B_max, a.R = K, B_max, R
    a.logits_dtype = _dtype_code(x)
    a.cost_kind = cost_kind
    return a


def _marshal_build(a: BuildArgs, dev, batch, L, K, R, flags, theta_curve, out, l_eff, bonus_token, ctx_len, cost_coef,
                   cost_table, table_idx, t_draft, ctx_grid):
    """Fills the per-request inputs and the output pointers of a BuildArgs; returns (out, tensors to keep alive)."""
    keep = [_dev(l_eff, dev, torch.int32), _dev(bonus_token, dev, torch.int32), _dev(ctx_len, dev, torch.int32),
            _dev(cost_coef, dev, torch.float64), _dev(cost_table, dev, torch.float64),
            _dev(table_idx, dev, torch.int32), _dev(t_draft, dev, torch.float64), _dev(ctx_grid, dev, torch.int32)]
    a.l_eff, a.bonus_token, a.ctx_len = _ptr(keep[0]), _ptr(keep[1]), _ptr(keep[2])
    a.cost_coef, a.cost_table, a.table_idx, a.t_draft = _ptr(keep[3]), _ptr(keep[4]), _ptr(keep[5]), _ptr(keep[6])
    a.ctx_grid = _ptr(keep[7])
    a.n_tables = 0 if keep[4] is None else keep[4].shape[0]
    if out is None:
        W = (R + 31) // 32
        i32 = lambda *s: torch.empty(*s, dtype=torch.int32, device=dev)
        f64 = lambda *s: torch.empty(*s, dtype=torch.float64, device=dev)
        out = Tree(n_nodes=i32(batch), token_ids=i32(batch, R), parent_idx=i32(batch, R), depth=i32(batch, R),
                   position_ids=i32(batch, R), node_logprob=f64(batch, R), phi=f64(batch), theta=f64(batch),
                   mask_bits=i32(batch, R, W),
                   mask_dense=torch.empty(batch, R, R, dtype=torch.uint8, device=dev) if flags & FLAG_EMIT_DENSE_MASK else None,
                   topk_token=i32(batch, L, K) if flags & FLAG_EMIT_TOPK else None,
                   topk_logprob=f64(batch, L, K) if flags & FLAG_EMIT_TOPK else None,
                   status=i32(batch), theta_curve=f64(batch, R) if theta_curve else None)
    a.n_nodes, a.token_ids, a.parent_idx, a.depth = _ptr(out.n_nodes), _ptr(out.token_ids), _ptr(out.parent_idx), _ptr(out.depth)
    a.position_ids, a.node_logprob, a.phi, a.theta = _ptr(out.position_ids), _ptr(out.node_logprob), _ptr(out.phi), _ptr(out.theta)
    a.theta_curve = _ptr(out.theta_curve)
    a.mask_bits, a.mask_dense = _ptr(out.mask_bits), _ptr(out.mask_dense)
    a.topk_token, a.topk_logprob, a.status = _ptr(out.topk_token), _ptr(out.topk_logprob), _ptr(out.status)
    return out, keep


def cadd_build_workspace_bytes(batch: int, L: int, V: int, K: int, B_max: int, R: int, dtype: torch.dtype) -> int:
    a = BuildArgs()
    a.struct_size = C.sizeof(BuildArgs)
    a.batch, a.L, a.V, a.K, a.B_max, a.R = batch, L, V, K, B_max, R
    a.logits_dtype = DTYPE_BF16 if dtype == torch.bfloat16 else DTYPE_FP32
    out = C.c_size_t()
    rc = lib().cadd_build_workspace_bytes(C.byref(a), C.byref(out))
    if rc != OK:
        raise CaddError(rc)
    return int(out.value)


def cadd_round_launches(batch: int, L: int, V: int, K: int, B_max: int, R: int, dtype: torch.dtype, rows_mode: int = ROWS_LIVE) -> int:
    """Kernels one round (cadd_build_tree + cadd_verify_tree) enqueues for this shape: 4, or 2 for small problems."""
    a = BuildArgs()
    a.struct_size = C.sizeof(BuildArgs)
    a.batch, a.L, a.V, a.K, a.B_max, a.R = batch, L, V, K, B_max, R
    a.logits_dtype = DTYPE_BF16 if dtype == torch.bfloat16 else DTYPE_FP32
    v = VerifyArgs()
    v.struct_size = C.sizeof(VerifyArgs)
    v.batch, v.L, v.R, v.V = batch, L, R, V
    v.logits_dtype, v.rows_mode = a.logits_dtype, rows_mode
    nb, nv = lib().cadd_build_launches(C.byref(a)), lib().cadd_verify_launches(C.byref(v))
    if nb < 0 or nv < 0:
        raise CaddError(min(nb, nv))
    return int(nb + nv)


def cadd_build_tree(draft_logits: torch.Tensor, K: int, B_max: int, R: Optional[int] = None, *,
                    l_eff=None, bonus_token=None, ctx_len=None,
                    cost_kind: int = COST_QUADRATIC, cost_coef=None, cost_table=None, table_idx=None,
                    t_draft=None, ctx_grid=None, theta_curve: bool = False, flags: int = 0, out: Optional[Tree] = None,
                    workspace: Optional[torch.Tensor] = None,
                    stream: Optional[torch.cuda.Stream] = None) -> Tree:
    """Build the draft trees of a batch (Eq. 1, Algorithm 1, Section 3.3) on the current CUDA stream.

    draft_logits: CUDA tensor [batch, L, V], bf16 or fp32, vocabulary axis contiguous.
    Small per-request inputs (l_eff, cost model, ...) are moved to the device if they are not there.
    `out` / `workspace` let a caller reuse buffers across rounds (no allocation inside the call then).
    """
    x = draft_logits
    if not x.is_cuda:
        raise ValueError("draft_logits must be a CUDA tensor (there is no CPU path)")
    if x.dim() != 3 or x.stride(2) != 1:
        raise ValueError("draft_logits must be [batch, L, V] with a contiguous vocabulary axis")
    dev = x.device
    batch, L, V = x.shape
    R = B_max + 1 if R is None else R
    a = _build_args(x, K, B_max, R, flags | (FLAG_REGULAR_PATH if FORCE_REGULAR_PATH else 0), cost_kind)
    a.draft_logits = x.data_ptr()
    a.stride_b, a.stride_l = x.stride(0), x.stride(1)
    out, keep = _marshal_build(a, dev, batch, L, K, R, flags, theta_curve, out, l_eff, bonus_token, ctx_len, cost_coef,
                               cost_table, table_idx, t_draft, ctx_grid)
    if workspace is None:
        nbytes = cadd_build_workspace_bytes(batch, L, V, K, B_max, R, x.dtype)
        workspace = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=dev)
    a.workspace, a.workspace_bytes = workspace.data_ptr(), workspace.numel()
    st = _stream_of(stream, dev)
    with torch.cuda.device(dev):
        rc = lib().cadd_build_tree(C.byref(a), st.cuda_stream)
    if rc != OK:
        raise CaddError(rc)
    # the call is asynchronous: keep temporaries alive until the stream has consumed them
    for t in keep + [workspace]:
        if t is not None:
            t.record_stream(st)
    return out


def cadd_verify_tree(target_logits: torch.Tensor, L: int, n_nodes: torch.Tensor, token_ids: torch.Tensor,
                     parent_idx: torch.Tensor, rows_mode: int = ROWS_LIVE, *, out: Optional[Verdict] = None,
                     flags: int = 0, stream: Optional[torch.cuda.Stream] = None) -> Verdict:
    """Greedy tree verification (Sections 3.1, 3.3): per-node argmax of target_logits [batch, R, V]
    and the walk along the longest accepted path, on the current CUDA stream."""
    y = target_logits
    if not y.is_cuda:
        raise ValueError("target_logits must be a CUDA tensor (there is no CPU path)")
    if y.dim() != 3 or y.stride(2) != 1:
        raise ValueError("target_logits must be [batch, R, V] with a contiguous vocabulary axis")
    dev = y.device
    batch, R, V = y.shape
    for t in (n_nodes, token_ids, parent_idx):
        if not (t.is_cuda and t.dtype == torch.int32 and t.is_contiguous()):
            raise ValueError("tree arrays must be contiguous int32 CUDA tensors")
    a = VerifyArgs()
    a.struct_size = C.sizeof(VerifyArgs)
    a.flags = flags | (VERIFY_REGULAR_PATH if FORCE_REGULAR_PATH else 0)
    a.batch, a.L, a.R, a.V = batch, L, R, V
    a.logits_dtype = _dtype_code(y)
    a.rows_mode = rows_mode
    a.target_logits = y.data_ptr()
    a.stride_b, a.stride_row = y.stride(0), y.stride(1)
    a.n_nodes, a.token_ids, a.parent_idx = n_nodes.data_ptr(), token_ids.data_ptr(), parent_idx.data_ptr()
    if out is None:
        i32 = lambda *s: torch.empty(*s, dtype=torch.int32, device=dev)
        out = Verdict(node_argmax=i32(batch, R), accepted_len=i32(batch), accepted_nodes=i32(batch, L),
                      next_bonus=i32(batch), status=i32(batch))
    a.node_argmax, a.accepted_len, a.accepted_nodes = _ptr(out.node_argmax), _ptr(out.accepted_len), _ptr(out.accepted_nodes)
    a.next_bonus, a.status = _ptr(out.next_bonus), _ptr(out.status)
    st = _stream_of(stream, dev)
    with torch.cuda.device(dev):
        rc = lib().cadd_verify_tree(C.byref(a), st.cuda_stream)
    if rc != OK:
        raise CaddError(rc)
    return out


def cadd_head_workspace_bytes(batch: int, R: int, hidden: int, V: int, L: int = 1, rows_mode: int = ROWS_LIVE) -> int:
    """Scratch bytes of cadd_verify_tree_fused_head; LIVE mode (the default here) needs room for a packed copy of the
    live hidden states and is therefore the larger of the two."""
    a = HeadArgs()
    a.struct_size = C.sizeof(HeadArgs)
    a.batch, a.L, a.R, a.hidden, a.V = batch, L, R, hidden, V
    a.rows_mode = rows_mode
    n = C.c_size_t(0)
    rc = lib().cadd_head_workspace_bytes(C.byref(a), C.byref(n))
    if rc != OK:
        raise CaddError(rc)
    return int(n.value)


def cadd_verify_tree_fused_head(hidden_states: torch.Tensor, weight: torch.Tensor, L: int, n_nodes: torch.Tensor,
                                token_ids: torch.Tensor, parent_idx: torch.Tensor, rows_mode: int = ROWS_LIVE, *,
                                out: Optional[Verdict] = None, workspace: Optional[torch.Tensor] = None,
                                stream: Optional[torch.cuda.Stream] = None) -> Verdict:
    """Greedy tree verification from the target's last hidden states [batch, R, hidden] and its output-projection
    weight [V, hidden] (both bf16): the logits h . W^T are formed on the tensor cores and reduced to the per-node
    argmax without being written to memory (Section 3.1), then the accepted path is walked (Section 3.3)."""
    h, w = hidden_states, weight
    if not (h.is_cuda and w.is_cuda):
        raise ValueError("hidden_states and weight must be CUDA tensors (there is no CPU path)")
    if h.dtype != torch.bfloat16 or w.dtype != torch.bfloat16:
        raise ValueError("hidden_states and weight must be bfloat16")
    if h.dim() != 3 or h.stride(2) != 1 or h.stride(0) != h.shape[1] * h.stride(1):
        raise ValueError("hidden_states must be [batch, R, hidden] with contiguous rows of equal stride")
    if w.dim() != 2 or w.stride(1) != 1 or w.shape[1] != h.shape[2]:
        raise ValueError("weight must be [V, hidden] with a contiguous hidden axis")
    dev = h.device
    batch, R, hidden = h.shape
    V = w.shape[0]
    for t in (n_nodes, token_ids, parent_idx):
        if not (t.is_cuda and t.dtype == torch.int32 and t.is_contiguous()):
            raise ValueError("tree arrays must be contiguous int32 CUDA tensors")
    a = HeadArgs()
    a.struct_size = C.sizeof(HeadArgs)
    a.batch, a.L, a.R, a.hidden, a.V = batch, L, R, hidden, V
    a.rows_mode = rows_mode
    a.hidden_states, a.stride_row = h.data_ptr(), h.stride(1)
    a.weight, a.stride_w = w.data_ptr(), w.stride(0)
    a.n_nodes, a.token_ids, a.parent_idx = n_nodes.data_ptr(), token_ids.data_ptr(), parent_idx.data_ptr()
    if out is None:
        i32 = lambda *s: torch.empty(*s, dtype=torch.int32, device=dev)
        out = Verdict(node_argmax=i32(batch, R), accepted_len=i32(batch), accepted_nodes=i32(batch, L),
                      next_bonus=i32(batch), status=i32(batch))
    a.node_argmax, a.accepted_len, a.accepted_nodes = _ptr(out.node_argmax), _ptr(out.accepted_len), _ptr(out.accepted_nodes)
    a.next_bonus, a.status = _ptr(out.next_bonus), _ptr(out.status)
    if workspace is None:
        workspace = torch.empty(cadd_head_workspace_bytes(batch, R, hidden, V, L, rows_mode), dtype=torch.uint8, device=dev)
    a.workspace, a.workspace_bytes = workspace.data_ptr(), workspace.numel()
    st = _stream_of(stream, dev)
    with torch.cuda.device(dev):
        rc = lib().cadd_verify_tree_fused_head(C.byref(a), st.cuda_stream)
    if rc != OK:
        raise CaddError(rc)
    workspace.record_stream(st)
    return out


def _build_head_args(batch, L, V, hidden, K, B_max, R, flags, cost_kind) -> BuildHeadArgs:
    h = BuildHeadArgs()
    h.struct_size = C.sizeof(BuildHeadArgs)
    h.hidden = hidden
    a = h.build
    a.struct_size = C.sizeof(BuildArgs)
    a.flags = flags
    a.batch, a.L, a.V = batch, L, V
    a.K, a.B_max, a.R = K, B_max, R
    a.logits_dtype = DTYPE_FP32
    a.cost_kind = cost_kind
    return h


def cadd_build_head_workspace_bytes(batch: int, L: int, V: int, hidden: int, K: int, B_max: int, R: int) -> int:
    h = _build_head_args(batch, L, V, hidden, K, B_max, R, 0, COST_QUADRATIC)
    n = C.c_size_t(0)
    rc = lib().cadd_build_head_workspace_bytes(C.byref(h), C.byref(n))
    if rc != OK:
        raise CaddError(rc)
    return int(n.value)


def cadd_build_tree_fused_head(hidden_states: torch.Tensor, weight: torch.Tensor, K: int, B_max: int, R: Optional[int] = None, *,
                               l_eff=None, bonus_token=None, ctx_len=None,
                               cost_kind: int = COST_QUADRATIC, cost_coef=None, cost_table=None, table_idx=None,
                               t_draft=None, ctx_grid=None, theta_curve: bool = False, flags: int = 0,
                               out: Optional[Tree] = None, workspace: Optional[torch.Tensor] = None,
                               stream: Optional[torch.cuda.Stream] = None) -> Tree:
    """cadd_build_tree from the drafter's last hidden states [batch, L, hidden] and its output-projection weight
    [V, hidden] (both bf16): the draft logits are formed on the tensor cores and consumed by the softmax statistics
    and the top-K selection without being written to memory (Eq. 1, Algorithm 1)."""
    hs, w = hidden_states, weight
    if not (hs.is_cuda and w.is_cuda):
        raise ValueError("hidden_states and weight must be CUDA tensors (there is no CPU path)")
    if hs.dtype != torch.bfloat16 or w.dtype != torch.bfloat16:
        raise ValueError("hidden_states and weight must be bfloat16")
    if hs.dim() != 3 or hs.stride(2) != 1 or hs.stride(0) != hs.shape[1] * hs.stride(1):
        raise ValueError("hidden_states must be [batch, L, hidden] with contiguous rows of equal stride")
    if w.dim() != 2 or w.stride(1) != 1 or w.shape[1] != hs.shape[2]:
        raise ValueError("weight must be [V, hidden] with a contiguous hidden axis")
    dev = hs.device
    batch, L, hidden = hs.shape
    V = w.shape[0]
    R = B_max + 1 if R is None else R
    h = _build_head_args(batch, L, V, hidden, K, B_max, R, flags, cost_kind)
    h.hidden_states, h.stride_row = hs.data_ptr(), hs.stride(1)
    h.weight, h.stride_w = w.data_ptr(), w.stride(0)
    out, keep = _marshal_build(h.build, dev, batch, L, K, R, flags, theta_curve, out, l_eff, bonus_token, ctx_len, cost_coef,
                               cost_table, table_idx, t_draft, ctx_grid)
    if workspace is None:
        workspace = torch.empty(cadd_build_head_workspace_bytes(batch, L, V, hidden, K, B_max, R), dtype=torch.uint8, device=dev)
    h.build.workspace, h.build.workspace_bytes = workspace.data_ptr(), workspace.numel()
    st = _stream_of(stream, dev)
    with torch.cuda.device(dev):
        rc = lib().cadd_build_tree_fused_head(C.byref(h), st.cuda_stream)
    if rc != OK:
        raise CaddError(rc)
    for t in keep + [workspace]:
        if t is not None:
            t.record_stream(st)
    return out


def cadd_verify_tree_sampled(target_logits: torch.Tensor, uniforms: torch.Tensor, L: int, n_nodes: torch.Tensor,
                             token_ids: torch.Tensor, parent_idx: torch.Tensor, rows_mode: int = ROWS_LIVE, *,
                             temperature: float = 1.0, out: Optional[Verdict] = None, flags: int = 0,
                             stream: Optional[torch.cuda.Stream] = None) -> Verdict:
    """Tree verification under sampling: one token is drawn per node from softmax(target_logits / temperature) by the
    inverse CDF at uniforms[b, j]; the walk follows the child that carries the drawn token.  Verdict.node_argmax holds
    the drawn tokens."""
    y = target_logits
    if not (y.is_cuda and uniforms.is_cuda):
        raise ValueError("target_logits and uniforms must be CUDA tensors (there is no CPU path)")
    if y.dim() != 3 or y.stride(2) != 1:
        raise ValueError("target_logits must be [batch, R, V] with a contiguous vocabulary axis")
    dev = y.device
    batch, R, V = y.shape
    if uniforms.dtype != torch.float64 or tuple(uniforms.shape) != (batch, R) or not uniforms.is_contiguous():
        raise ValueError("uniforms must be a contiguous float64 tensor [batch, R]")
    for t in (n_nodes, token_ids, parent_idx):
        if not (t.is_cuda and t.dtype == torch.int32 and t.is_contiguous()):
            raise ValueError("tree arrays must be contiguous int32 CUDA tensors")
    a = SampleArgs()
    a.struct_size = C.sizeof(SampleArgs)
    a.flags = flags
    a.batch, a.L, a.R, a.V = batch, L, R, V
    a.logits_dtype = _dtype_code(y)
    a.rows_mode = rows_mode
    a.temperature = float(temperature)
    a.target_logits = y.data_ptr()
    a.stride_b, a.stride_row = y.stride(0), y.stride(1)
    a.uniforms = uniforms.data_ptr()
    a.n_nodes, a.token_ids, a.parent_idx = n_nodes.data_ptr(), token_ids.data_ptr(), parent_idx.data_ptr()
    if out is None:
        i32 = lambda *s: torch.empty(*s, dtype=torch.int32, device=dev)
        out = Verdict(node_argmax=i32(batch, R), accepted_len=i32(batch), accepted_nodes=i32(batch, L),
                      next_bonus=i32(batch), status=i32(batch))
    a.node_token, a.accepted_len, a.accepted_nodes = _ptr(out.node_argmax), _ptr(out.accepted_len), _ptr(out.accepted_nodes)
    a.next_bonus, a.status = _ptr(out.next_bonus), _ptr(out.status)
    st = _stream_of(stream, dev)
    with torch.cuda.device(dev):
        rc = lib().cadd_verify_tree_sampled(C.byref(a), st.cuda_stream)
    if rc != OK:
        raise CaddError(rc)
    return out


def cadd_fit_cost_tables(y: torch.Tensor, *, stream: Optional[torch.cuda.Stream] = None):
    """Offline cost fitting (Eq. 12): the convex, non-decreasing least-squares fit of every row of y [n_tables, N]
    (fp64, CUDA).  Returns (fit [n_tables, N] fp64, n_breaks [n_tables] int32, status [n_tables] int32)."""
    if not y.is_cuda:
        raise ValueError("y must be a CUDA tensor (there is no CPU path)")
    if y.dtype != torch.float64 or y.dim() != 2 or not y.is_contiguous():
        raise ValueError("y must be a contiguous float64 tensor [n_tables, N]")
    a = FitArgs()
    a.struct_size = C.sizeof(FitArgs)
    a.n_tables, a.N = y.shape
    fit = torch.empty_like(y)
    nb = torch.empty(y.shape[0], dtype=torch.int32, device=y.device)
    st = torch.empty(y.shape[0], dtype=torch.int32, device=y.device)
    a.y, a.fit, a.n_breaks, a.status = y.data_ptr(), fit.data_ptr(), nb.data_ptr(), st.data_ptr()
    with torch.cuda.device(y.device):
        rc = lib().cadd_fit_cost_tables(C.byref(a), _stream_of(stream, y.device).cuda_stream)
    if rc != OK:
        raise CaddError(rc)
    return fit, nb, st


def cadd_build_tree_static_scratch(draft_logits: torch.Tensor, K: int, B_max: int, R: Optional[int] = None, *,
                                   l_eff=None, bonus_token=None, ctx_len=None,
                                   cost_kind: int = COST_QUADRATIC, cost_coef=None, cost_table=None,
                                   table_idx=None, t_draft=None, ctx_grid=None, flags: int = 0, out: Tree = None,
                                   stream: Optional[torch.cuda.Stream] = None) -> Tree:
    """cadd_build_tree without a workspace argument: the library uses its built-in scratch array.

    For callers that may not allocate device memory (for instance code running inside a host
    application that owns the memory pool): pass every input on the device already and a preallocated
    `out`; the call then allocates nothing.  (If `out` is omitted it is allocated here with torch, which
    is a convenience for tests.)  Shapes whose scratch need exceeds STATIC_SCRATCH_BYTES raise CaddError
    with code ERR_STATIC_SCRATCH.  Calls on one device share the scratch: do not let two of them overlap
    on the GPU.  The first call per device performs a one-time address look-up and belongs outside any
    stream capture."""
    x = draft_logits
    if not x.is_cuda:
        raise ValueError("draft_logits must be a CUDA tensor (there is no CPU path)")
    if x.dim() != 3 or x.stride(2) != 1:
        raise ValueError("draft_logits must be [batch, L, V] with a contiguous vocabulary axis")
    dev = x.device
    batch, L, V = x.shape
    R = B_max + 1 if R is None else R
    a = _build_args(x, K, B_max, R, flags, cost_kind)
    a.draft_logits = x.data_ptr()
    a.stride_b, a.stride_l = x.stride(0), x.stride(1)
    keep = [_dev(l_eff, dev, torch.int32), _dev(bonus_token, dev, torch.int32), _dev(ctx_len, dev, torch.int32),
            _dev(cost_coef, dev, torch.float64), _dev(cost_table, dev, torch.float64),
            _dev(table_idx, dev, torch.int32), _dev(t_draft, dev, torch.float64), _dev(ctx_grid, dev, torch.int32)]
    a.l_eff, a.bonus_token, a.ctx_len = _ptr(keep[0]), _ptr(keep[1]), _ptr(keep[2])
    a.cost_coef, a.cost_table, a.table_idx, a.t_draft = _ptr(keep[3]), _ptr(keep[4]), _ptr(keep[5]), _ptr(keep[6])
    a.ctx_grid = _ptr(keep[7])
    a.n_tables = 0 if keep[4] is None else keep[4].shape[0]
    if out is None:
        W = (R + 31) // 32
        i32 = lambda *s: torch.empty(*s, dtype=torch.int32, device=dev)
        f64 = lambda *s: torch.empty(*s, dtype=torch.float64, device=dev)
        out = Tree(n_nodes=i32(batch), token_ids=i32(batch, R), parent_idx=i32(batch, R), depth=i32(batch, R),
                   position_ids=i32(batch, R), node_logprob=f64(batch, R), phi=f64(batch), theta=f64(batch),
                   mask_bits=i32(batch, R, W),
                   mask_dense=torch.empty(batch, R, R, dtype=torch.uint8, device=dev) if flags & FLAG_EMIT_DENSE_MASK else None,
                   topk_token=i32(batch, L, K) if flags & FLAG_EMIT_TOPK else None,
                   topk_logprob=f64(batch, L, K) if flags & FLAG_EMIT_TOPK else None,
                   status=i32(batch))
    a.n_nodes, a.token_ids, a.parent_idx, a.depth = _ptr(out.n_nodes), _ptr(out.token_ids), _ptr(out.parent_idx), _ptr(out.depth)
    a.position_ids, a.node_logprob, a.phi, a.theta = _ptr(out.position_ids), _ptr(out.node_logprob), _ptr(out.phi), _ptr(out.theta)
    a.mask_bits, a.mask_dense = _ptr(out.mask_bits), _ptr(out.mask_dense)
    a.topk_token, a.topk_logprob, a.status = _ptr(out.topk_token), _ptr(out.topk_logprob), _ptr(out.status)
    st = _stream_of(stream, dev)
    with torch.cuda.device(dev):
        rc = lib().cadd_build_tree_static_scratch(C.byref(a), st.cuda_stream)
    if rc != OK:
        raise CaddError(rc)
    for t in keep:
        if t is not None:
            t.record_stream(st)
    return out
