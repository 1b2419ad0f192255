"""The allocation-free attention entry point against the ordinary one.

litevggt_global_attn_static exists for callers that may not call cudaMalloc (code under a
device-owning memory manager, plug-ins entered after the memory map is frozen, loops that
cannot take an allocation's device-wide synchronisation).  It keeps its intermediates in a
fixed array inside the library, shared by all calls, so the test calls it twice in a row
with different inputs and sizes: the second call must not be disturbed by what the first
left behind.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import oracle as O
from synthdata import WORKLOADS, make_attention_weights, make_images, make_tokens
from helpers import LAYER_NOISE, bf16_bound, check_bf16, rel_err, to_f64

pytestmark = pytest.mark.gpu


def test_static_attention_matches_context_attention_twice():
    import paper_2512_04939_b200 as pkg

    wl = WORKLOADS["C1"]
    ctx = pkg.LiteVGGT(wl.frames, wl.grid_h, wl.grid_w, wl.merge_ratio)  # the ordinary path (allocates)
    m_full = ctx.n_merged  # 543 rows: several key tiles and a ragged tail
    w_qkv, b_qkv, w_o, b_o = [t.cuda() for t in make_attention_weights(wl, 0)]
    gen = torch.Generator().manual_seed(77)
    flag = torch.full((1,), 7, dtype=torch.int32, device="cuda")
    for call, scale in enumerate((1.0, 2.5)):
        xm = (scale * torch.randn(m_full, 1024, generator=gen)).to(torch.bfloat16).cuda()
        want = ctx.global_attn(xm, w_qkv, b_qkv, w_o, b_o)
        ctx.poll()
        out = torch.empty_like(xm)
        got = pkg.global_attn_static(xm, w_qkv, b_qkv, w_o, b_o, out=out, device_status=flag)
        torch.cuda.synchronize()
        assert int(flag.item()) == 0, f"call {call}: a kernel flagged a bounded wait"
        ref = to_f64(want)
        # same kernels on the same inputs: the bf16 tolerance of the other parity tests, and in
        # fact identical bits
        assert rel_err(to_f64(got), ref) <= bf16_bound(ref), f"call {call}"
        assert torch.equal(got, want), f"call {call}"
    # a shorter sequence right after a longer one: rows left in the array must not leak in, so the
    # result is judged against the CPU oracle on the 200 rows alone
    # (rows of the token generator, as in the other end-to-end checks: independent Gaussian rows
    # average to an output far smaller than the values it is made of, which magnifies every per-key
    # rounding in relative terms)
    xs = make_tokens(wl, make_images(wl))[:200].contiguous().cuda()
    got = pkg.global_attn_static(xs, w_qkv, None, w_o, None)
    torch.cuda.synchronize()
    ref_y = O.global_attention(to_f64(xs), to_f64(w_qkv), None, to_f64(w_o), None, heads=16)
    check_bf16("static entry point, 200 rows after 543", to_f64(got), ref_y, noise=LAYER_NOISE)
    # and the call allocates nothing: with the output given, neither the driver's free memory nor
    # the caching allocator's books move across a call
    out = torch.empty_like(xs)
    pkg.global_attn_static(xs, w_qkv, None, w_o, None, out=out)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    booked_before = torch.cuda.memory_allocated()
    reserved_before = torch.cuda.memory_reserved()
    pkg.global_attn_static(xs, w_qkv, None, w_o, None, out=out)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    assert torch.cuda.memory_allocated() == booked_before and torch.cuda.memory_reserved() == reserved_before
    assert torch.equal(out, got)
    ctx.close()


def test_static_attention_rejects_sizes_beyond_its_array():
    import paper_2512_04939_b200 as pkg

    lib = pkg.load_library()
    x = torch.zeros(16, 1024, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(3072, 1024, dtype=torch.bfloat16, device="cuda")
    for m in (0, pkg.STATIC_ATTN_MAX_ROWS + 1, -3):
        rc = lib.litevggt_global_attn_static(x.data_ptr(), m, w.data_ptr(), None, w.data_ptr(), None, x.data_ptr(),
                                             None, None)
        assert rc == 3, f"m={m} must be refused as a shape error, got {rc}"
    assert lib.litevggt_global_attn_static(None, 16, w.data_ptr(), None, w.data_ptr(), None, x.data_ptr(), None,
                                           None) == 1
