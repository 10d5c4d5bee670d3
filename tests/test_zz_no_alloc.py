"""mx_quantize_host_static: the host-buffer quantize for callers that may not allocate device
memory (a plug-in whose host application owns every free byte of the GPU, a loop that must never
enter the CUDA allocator).  Its staging area is a fixed array inside the library, so the test
checks the two things that could go wrong with a shared, never-cleared scratch area: the result
must equal that of the existing mx_quantize_host (which stages in a caller-supplied workspace)
and that of the CPU oracle byte for byte, and a second call right after the first -- with a
different shape, format and scale layout, so that stale bytes of the first call sit where the
second one works -- must be just as exact.  The promise itself is checked too: the free device
memory the driver reports is the same before and after a call, on the first call of the process
and on a later one.  Collected last on purpose: a failure here cannot hide another test's result."""
import ctypes

import numpy as np
import pytest
import torch

import oracle as O
import paper_2310_10537_b200 as mx
import workloads as inputs
from gpu_util import to_oracle_input

pytestmark = pytest.mark.gpu


def _host_outputs(shape, axis, fmt, layout):
    e = torch.empty(mx.mx_elems_bytes(shape, axis, fmt), dtype=torch.uint8).pin_memory()
    s = torch.empty(mx.mx_scales_bytes(shape, axis, layout), dtype=torch.uint8).pin_memory()
    e.fill_(0xA5)
    s.fill_(0xA5)
    return e, s


def _both_ways(x, axis, fmt, rounding, layout):
    shape = list(x.shape)
    # existing entry point: caller-allocated device workspace
    ref_e, ref_s = _host_outputs(shape, axis, fmt, layout)
    ws = torch.empty(mx.mx_quantize_host_workspace_bytes(shape, axis, fmt, x.dtype, layout),
                     dtype=torch.uint8, device="cuda")
    mx.mx_quantize_host(x, ref_e, ref_s, axis, fmt, rounding, ws, layout)
    # new entry point: no workspace, nothing allocated by the call
    got_e, got_s = _host_outputs(shape, axis, fmt, layout)
    mx.mx_quantize_host_static(x, got_e, got_s, axis, fmt, rounding, layout)
    assert torch.equal(got_e, ref_e), "element codes differ from mx_quantize_host"
    assert torch.equal(got_s, ref_s), "scale bytes differ from mx_quantize_host"
    # and against the definition itself: the oracle on the same input bytes
    want_e, want_s = O.quantize(to_oracle_input(x), axis, fmt, rounding, layout)
    assert np.array_equal(got_e.numpy(), want_e), "element codes differ from the oracle"
    assert np.array_equal(got_s.numpy(), want_s), "scale bytes differ from the oracle"


def _free_bytes():
    torch.cuda.synchronize()
    return torch.cuda.mem_get_info()[0]


def test_static_scratch_call_allocates_no_device_memory():
    """Free device memory as the driver reports it must not move across a call.  The first call of
    a process is let through unmeasured: that is when the driver loads the library's device code
    and, with it, claims the built-in array (the header says so) -- module loading, not an
    allocation by the call.  Every later call is held to a difference of exactly zero, also one
    with another shape that leaves stale bytes behind.  Host outputs are pinned beforehand, so
    nothing else in the measured window can allocate."""
    x = inputs.adversarial("cpu", rows=256, cols=512, dtype=torch.bfloat16, seed=33).pin_memory()
    y = inputs.adversarial("cpu", rows=128, cols=320, dtype=torch.bfloat16, seed=35)[:, :300].contiguous().pin_memory()
    ex, sx = _host_outputs(list(x.shape), 1, mx.MX_E4M3, mx.MX_SCALES_SWIZZLED)
    ey, sy = _host_outputs(list(y.shape), 1, mx.MX_E4M3, mx.MX_SCALES_SWIZZLED)
    torch.zeros(1, device="cuda")            # the CUDA context and torch's pool exist before measuring
    # first calls: set-up (address look-up, device code of both kernels used below loaded)
    mx.mx_quantize_host_static(x, ex, sx, 1, mx.MX_E4M3, mx.MX_RNE, mx.MX_SCALES_SWIZZLED)
    mx.mx_quantize_host_static(y, ey, sy, 1, mx.MX_E4M3, mx.MX_RNE, mx.MX_SCALES_SWIZZLED)
    for call, (t, e, s) in enumerate(((x, ex, sx), (y, ey, sy), (x, ex, sx))):
        before = _free_bytes()
        mx.mx_quantize_host_static(t, e, s, 1, mx.MX_E4M3, mx.MX_RNE, mx.MX_SCALES_SWIZZLED)
        after = _free_bytes()
        assert after == before, f"later call {call}: free device memory moved by {before - after} bytes"
        want_e, want_s = O.quantize(to_oracle_input(t), 1, mx.MX_E4M3, O.RNE, O.SWIZZLED)
        assert np.array_equal(e.numpy(), want_e) and np.array_equal(s.numpy(), want_s)


def test_static_scratch_matches_workspace_variant_twice_in_a_row():
    # call 1: BF16, blocks along the last axis, swizzled scales with padding (200 rows, 9 K-blocks)
    x1 = inputs.adversarial("cpu", rows=200, cols=288, dtype=torch.bfloat16, seed=31).pin_memory()
    _both_ways(x1, 1, mx.MX_E4M3, mx.MX_RNE, mx.MX_SCALES_SWIZZLED)
    # call 2, immediately after: FP32, strided axis, 6-bit codes, linear scales, smaller tensor
    x2 = inputs.adversarial("cpu", rows=96, cols=160, dtype=torch.float32, seed=32).t().contiguous().pin_memory()
    _both_ways(x2, 0, mx.MX_E3M2, mx.MX_RHAZ, mx.MX_SCALES_LINEAR)
    # and the first request again: its padding must be clean although call 2 wrote there
    _both_ways(x1, 1, mx.MX_E2M1, mx.MX_RNE, mx.MX_SCALES_SWIZZLED)
    # a row length that is not a whole number of blocks, after larger calls: the zero codes that pad
    # the partial last block and the padding of the scale tensor sit on stale bytes of the calls above
    x3 = inputs.adversarial("cpu", rows=100, cols=320, dtype=torch.bfloat16, seed=34)[:, :300].contiguous().pin_memory()
    _both_ways(x3, 1, mx.MX_E3M2, mx.MX_RNE, mx.MX_SCALES_SWIZZLED)
    _both_ways(x3, 0, mx.MX_E4M3, mx.MX_RHAZ, mx.MX_SCALES_LINEAR)


def test_static_scratch_rejects_oversized_request():
    # 4096 x 4096 FP32 needs 64 MiB of staging for the input alone: beyond the fixed array
    shape = (ctypes.c_int64 * 2)(4096, 4096)
    need = mx.mx_quantize_host_workspace_bytes([4096, 4096], 1, mx.MX_E4M3, torch.float32)
    assert need > mx.binding.MX_STATIC_SCRATCH_BYTES
    dummy = torch.zeros(64, dtype=torch.uint8).pin_memory()
    rc = mx.lib().mx_quantize_host_static(dummy.data_ptr(), dummy.data_ptr(), dummy.data_ptr(),
                                          shape, 2, 1, mx.MX_E4M3, mx.MX_RNE, None)
    assert rc == mx.MX_ERR_WORKSPACE
    # the largest tensors that fit still work: 2048 x 2048 BF16 -> 8 MiB + 4 MiB + scales
    x = torch.randn(2048, 2048).to(torch.bfloat16).pin_memory()
    _both_ways(x, 1, mx.MX_E5M2, mx.MX_RNE, mx.MX_SCALES_SWIZZLED)
