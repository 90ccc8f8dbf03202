"""The allocation-free Stage-2 entry point against the handle-based one.

Some callers may not allocate device memory (stream-ordered or captured regions
of a framework, a memory pool that owns the device, plug-ins that only get raw
buffers).  prox_stage2_ffn_noalloc serves them: it keeps its two intermediates
in a fixed array inside the library instead of in allocated scratch.  This test
calls it through the C ABI twice in a row, on different tokens and masks, and
checks each result against prox_stage2_ffn on the same inputs.  The two paths
run the same kernels, so they may differ only by the order of fp32 atomic adds;
the file sorts last so that a failure here cannot hide any other test.
"""
import numpy as np
import pytest
import torch

import __graft_entry__ as entry
from paper_2607_27591_b200 import inputs
from tests.gpu_common import Problem, check_y

pytestmark = pytest.mark.gpu


def test_noalloc_stage2_matches_handle_based_stage2_twice():
    entry.build()
    from paper_2607_27591_b200 import binding as pb
    from oracle import prox_oracle as po
    wl, wg, wu, wd, x = inputs.make_workload("toy", n_tokens=4)
    p = Problem(pb, wg, wu, wd, x, max_batch=1, out_dtype=1)
    try:
        p.quantize(4, 0)                       # the handle-based call needs its channel-major W_down
        w_down_t = p.t_wd.t().contiguous()      # what a no-alloc caller prepares ahead of time
        rng = np.random.default_rng(7)
        for call, (t, k2) in enumerate(((0, 461), (3, 977))):
            sel_np = np.sort(rng.choice(p.F, size=k2, replace=False)).astype(np.int32)
            sel = torch.from_numpy(sel_np).cuda()
            y_ref = p.y_empty()
            pb.prox_stage2_ffn(p.h, p.t_x[t], 1, sel, k2, y_ref)
            y = torch.full((1, p.D), float("nan"), dtype=torch.float32, device="cuda")
            y16 = torch.full((1, p.D), float("nan"), dtype=torch.bfloat16, device="cuda")
            side = torch.cuda.Stream()                 # the second call runs on a stream of its own
            side.wait_stream(torch.cuda.current_stream())
            torch.cuda.synchronize()
            # the driver's own count of free device memory (torch's counter would not see a cudaMalloc inside
            # the library) and torch's counter (which sees what the binding might allocate)
            free_before, _ = torch.cuda.mem_get_info()
            before = torch.cuda.memory_allocated()
            sp = side.cuda_stream if call == 1 else None
            pb.prox_stage2_ffn_noalloc(p.t_x[t], p.t_wg, p.t_wu, w_down_t, p.D, p.F, sel, k2, y, 1, stream=sp)
            pb.prox_stage2_ffn_noalloc(p.t_x[t], p.t_wg, p.t_wu, w_down_t, p.D, p.F, sel, k2, y16, 0, stream=sp)
            torch.cuda.synchronize()
            assert torch.cuda.memory_allocated() == before
            assert torch.cuda.mem_get_info()[0] == free_before, "device memory was allocated during the call"
            # bf16 output: the fp32 result rounded once
            a16 = y16.float().cpu().numpy()[0]
            assert np.all(np.isfinite(a16))
            assert np.max(np.abs(a16 - y.cpu().numpy()[0])) <= 2.0 ** -8 * np.max(np.abs(y.cpu().numpy()[0])) + 1e-30
            a, b = y.cpu().numpy()[0], y_ref.cpu().numpy()[0]
            assert np.all(np.isfinite(a)), f"call {call}"
            # same kernels, same inputs: only the order of the fp32 atomics may differ
            assert np.max(np.abs(a - b)) <= 1e-5 * np.max(np.abs(b)), f"call {call}"
            # and both stay within the tolerance the parity tests use against the oracle
            y_or, _ = po.stage2(p.x[t], sel_np, p.wg, p.wu, p.wd)
            check_y(a, y_or)
        # limits are refused with a clear status, not truncated
        R = pb.raw("prox_stage2_ffn_noalloc")
        args = lambda D, F, k2: (p.t_x.data_ptr(), p.t_wg.data_ptr(), p.t_wu.data_ptr(), w_down_t.data_ptr(),
                                 D, F, sel.data_ptr(), k2, y.data_ptr(), 1, None)
        assert R(*args(32768, 65536, 16)) == 2           # d_model beyond the fixed scratch
        assert R(*args(512, 65536, 40000)) == 2          # k2 beyond the fixed scratch
        assert R(*args(512, 1536, 0)) == 1
        assert R(None, *args(512, 1536, 8)[1:]) == 1
    finally:
        p.close()
