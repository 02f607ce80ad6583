"""The scratch-free entry point, cadd_build_tree_static_scratch: for callers that cannot give the
library a workspace (no allocator of their own, or allocation forbidden where they run), the library
uses a fixed scratch array of its own.  This file is collected last on purpose, so that a run stopping
at the first failure has already been through every other test.

The GPU test calls the new entry point through the C ABI twice in a row (the shared scratch keeps the
first call's contents, which must not matter) and compares both results with the regular entry point's
on the same inputs: integer outputs bit for bit, floating-point outputs within the tolerances the other
GPU tests use."""
import ctypes as C

import pytest
import torch

from paper_2606_01813_b200 import binding as G
from paper_2606_01813_b200 import build as B
from paper_2606_01813_b200 import synth

INT_FIELDS = ("n_nodes", "token_ids", "parent_idx", "depth", "position_ids", "mask_bits", "topk_token", "status")
FLOAT_FIELDS = ("node_logprob", "phi", "theta", "topk_logprob")


def test_static_scratch_refuses_oversized_problems():
    """Pure host check (no GPU needed): shapes whose scratch need is above the built-in array are refused."""
    B.build()
    lib = G.lib()
    a = G.BuildArgs()
    a.struct_size = C.sizeof(G.BuildArgs)
    a.batch, a.L, a.V, a.K, a.B_max, a.R = 512, 64, 151936, 64, 256, 257
    need = C.c_size_t()
    assert lib.cadd_build_workspace_bytes(C.byref(a), C.byref(need)) == G.OK
    assert need.value > G.STATIC_SCRATCH_BYTES
    assert lib.cadd_build_tree_static_scratch(C.byref(a), None) == G.ERR_STATIC_SCRATCH
    assert "scratch" in G.cadd_status_string(G.ERR_STATIC_SCRATCH)
    a.struct_size += 4                                    # ordinary validation still comes first
    assert lib.cadd_build_tree_static_scratch(C.byref(a), None) == G.ERR_STRUCT_SIZE
    for name in ("c1", "c2", "c3", "c4", "c5"):           # every benchmark shape fits
        cfg = synth.CONFIGS[name]
        assert G.cadd_build_workspace_bytes(cfg.batch, cfg.L, cfg.V, cfg.K, cfg.B_max, cfg.R, cfg.torch_dtype) \
            <= G.STATIC_SCRATCH_BYTES


@pytest.mark.gpu
def test_static_scratch_matches_regular_entry_point_twice():
    cfg = synth.scaled(synth.CONFIGS["c2"], batch=3)
    results = []
    for seed in (11, 12):                                 # two different inputs, back to back
        d = synth.make_draft_inputs(cfg, seed)
        c = synth.make_cost_inputs(cfg, seed)
        x = d.logits.cuda()
        kw = dict(l_eff=d.l_eff, bonus_token=d.bonus_token, ctx_len=d.ctx_len, cost_coef=c.coef, flags=G.FLAG_EMIT_TOPK)
        ref = G.cadd_build_tree(x, cfg.K, cfg.B_max, cfg.R, **kw)
        got = G.cadd_build_tree_static_scratch(x, cfg.K, cfg.B_max, cfg.R, **kw)
        torch.cuda.synchronize()
        results.append((ref, got))
    for ref, got in results:
        for f in INT_FIELDS:
            assert torch.equal(getattr(ref, f), getattr(got, f)), f
        for f in FLOAT_FIELDS:
            a, b = getattr(ref, f), getattr(got, f)
            fin = torch.isfinite(a)
            assert torch.equal(fin, torch.isfinite(b)), f
            assert torch.allclose(a[fin], b[fin], rtol=1e-5, atol=2e-9), f
    assert int(results[0][0].n_nodes.max()) > 0            # the case is not trivial
    # the same call again on the first input: stale scratch contents from the second call do not matter
    d = synth.make_draft_inputs(cfg, 11)
    c = synth.make_cost_inputs(cfg, 11)
    again = G.cadd_build_tree_static_scratch(d.logits.cuda(), cfg.K, cfg.B_max, cfg.R, l_eff=d.l_eff,
                                             bonus_token=d.bonus_token, ctx_len=d.ctx_len, cost_coef=c.coef,
                                             flags=G.FLAG_EMIT_TOPK)
    torch.cuda.synchronize()
    for f in INT_FIELDS:
        assert torch.equal(getattr(results[0][1], f), getattr(again, f)), f


@pytest.mark.gpu
def test_static_scratch_calls_allocate_nothing():
    """With every input already on the device and the outputs preallocated, calls of the scratch-free entry point
    must leave the device's memory exactly as it was: neither torch's allocator nor the driver hands anything out
    (the one-time address look-up happened in the warm-up call)."""
    cfg = synth.scaled(synth.CONFIGS["c2"], batch=2)
    d = synth.make_draft_inputs(cfg, 13)
    c = synth.make_cost_inputs(cfg, 13)
    dev = torch.device("cuda")
    x = d.logits.to(dev)
    kw = dict(l_eff=d.l_eff.to(dev, torch.int32), bonus_token=d.bonus_token.to(dev, torch.int32),
              ctx_len=d.ctx_len.to(dev, torch.int32), cost_coef=c.coef.to(dev, torch.float64), flags=G.FLAG_EMIT_TOPK)
    out = G.cadd_build_tree_static_scratch(x, cfg.K, cfg.B_max, cfg.R, **kw)          # warm-up: allocates `out`
    torch.cuda.synchronize()
    first = out.token_ids.clone()
    allocated, reserved = torch.cuda.memory_allocated(dev), torch.cuda.memory_reserved(dev)
    free_before, _ = torch.cuda.mem_get_info(dev)
    for _ in range(5):
        G.cadd_build_tree_static_scratch(x, cfg.K, cfg.B_max, cfg.R, out=out, **kw)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info(dev)
    assert torch.cuda.memory_allocated(dev) == allocated and torch.cuda.memory_reserved(dev) == reserved
    assert free_after == free_before
    assert torch.equal(out.token_ids, first)
