"""GPU parity: libprox (through the C ABI) against the CPU oracle, element by
element on the same seeded inputs.  Tolerances (written here): integer work (quantizer codes, input mask) bit-exact; channel masks
identical outside a 1e-3 relative band around the k2-th oracle score; outputs
within 2e-2 * RMS(y_oracle)."""
import numpy as np
import pytest
import torch

import __graft_entry__ as entry
from oracle import prox_oracle as po
from paper_2607_27591_b200 import inputs
from tests.gpu_common import Problem, check_mask, check_y

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pb():
    entry.build()
    from paper_2607_27591_b200 import binding
    return binding


@pytest.fixture(scope="module")
def toy(pb):
    wl, wg, wu, wd, x = inputs.make_workload("toy")
    p = Problem(pb, wg, wu, wd, x, max_batch=8)
    yield wl, p
    p.close()


# ---------------------------------------------------------------- quantizer
@pytest.mark.parametrize("bits,group", [(4, 0), (4, 128), (8, 0), (8, 128)])
def test_quantizer_bit_exact(pb, toy, bits, group):
    wl, p = toy
    _, _, (qg, sg, qu, su) = p.quantize(bits, group)
    ng = 1 if group == 0 else p.D // group
    for which, (q_ref, s_ref) in enumerate(((qg, sg), (qu, su))):
        q = np.empty((p.F, p.D), dtype=np.int8)
        s = np.empty((p.F, ng), dtype=np.float32)
        pb.prox_proxy_export(p.h, which, q, s)
        assert np.array_equal(s, s_ref.astype(np.float32)), "scales differ"
        assert np.array_equal(q, q_ref), f"{(q != q_ref).sum()} codes differ"


def test_quantizer_zero_rows_and_ragged_shape(pb):
    wg, wu, wd, x = inputs.make_small(384, 320, 2, seed=5)      # F = 320: last strip is ragged
    wg[7, :] = 0
    wu[9, 128:256] = 0
    p = Problem(pb, wg, wu, wd, x)
    try:
        for bits, group in ((4, 0), (4, 128), (8, 128)):
            _, _, (qg, sg, qu, su) = p.quantize(bits, group)
            ng = 1 if group == 0 else p.D // group
            for which, (q_ref, s_ref) in enumerate(((qg, sg), (qu, su))):
                q = np.empty((p.F, p.D), dtype=np.int8)
                s = np.empty((p.F, ng), dtype=np.float32)
                pb.prox_proxy_export(p.h, which, q, s)
                assert np.array_equal(s, s_ref.astype(np.float32)) and np.array_equal(q, q_ref)
    finally:
        p.close()


# --------------------------------------------------------------- input mask
def test_input_topk_exact(pb, toy):
    wl, p = toy
    p.quantize(4, 0)
    for k1 in (1, 2, 31, 461, p.D - 1, p.D):
        idx = torch.empty(8, k1, dtype=torch.int32, device="cuda")
        pb.prox_input_topk(p.h, p.t_x[:8], 8, k1, idx)
        got = idx.cpu().numpy()
        for t in range(8):
            assert np.array_equal(got[t], po.input_topk(p.x[t], k1)), (k1, t)


def test_input_topk_ties(pb, toy):
    """bf16 magnitudes tie often; lower index must win."""
    wl, p = toy
    vals = np.array([1.0, -1.0, 0.5, 2.0, -2.0, 0.0, -0.0, 1.0], dtype=np.float32)
    x = np.tile(vals, p.D // 8)[None, :]
    bits = inputs.f32_to_bf16_bits(x)
    from tests.gpu_common import dev_bf16
    tx = dev_bf16(bits)
    for k1 in (1, 64, 65, 128, 129, 300, p.D - 3):
        idx = torch.empty(1, k1, dtype=torch.int32, device="cuda")
        pb.prox_input_topk(p.h, tx, 1, k1, idx)
        assert np.array_equal(idx.cpu().numpy()[0], po.input_topk(x[0].astype(np.float64), k1)), k1


# ------------------------------------------------------------------ Stage 1
@pytest.mark.parametrize("bits,group", [(4, 0), (4, 128), (8, 0)])
def test_stage1_mask_toy(pb, toy, bits, group):
    wl, p = toy
    p.quantize(bits, group)
    k1, k2 = wl.points[50]
    sel = torch.empty(1, k2, dtype=torch.int32, device="cuda")
    sc = torch.empty(1, p.F, dtype=torch.float32, device="cuda")
    worst = 0.0
    for t in range(p.x.shape[0]):
        pb.prox_stage1_mask(p.h, p.t_x[t], 1, k1, k2, sel, sc)
        torch.cuda.synchronize()
        idx, score, sel_ref, thr = p.oracle_stage1(t, k1, k2)
        check_mask(sel.cpu().numpy()[0].astype(np.int64), score, sel_ref, thr, k2, p.F)
        got = sc.cpu().numpy()[0].astype(np.float64)
        worst = max(worst, float(np.max(np.abs(got - score)) / thr))
    assert worst < 2e-4, worst          # fp32 accumulation + fast exp, relative to the threshold score
    assert pb.prox_last_device_status(p.h) == 0


@pytest.mark.parametrize("k1,k2", [(512, 1536), (1, 1), (512, 1), (17, 1535), (300, 768)])
def test_stage1_edge_budgets(pb, toy, k1, k2):
    wl, p = toy
    p.quantize(4, 0)
    sel = torch.empty(1, k2, dtype=torch.int32, device="cuda")
    for t in (0, 5):
        pb.prox_stage1_mask(p.h, p.t_x[t], 1, k1, k2, sel, None)
        idx, score, sel_ref, thr = p.oracle_stage1(t, k1, k2)
        check_mask(sel.cpu().numpy()[0].astype(np.int64), score, sel_ref, thr, k2, p.F)


# ------------------------------------------------------------------ Stage 2
def test_stage2_given_mask(pb, toy):
    wl, p = toy
    p.quantize(4, 0)
    rng = np.random.default_rng(0)
    for k2 in (1, 7, 461, 1000, p.F):
        for t in (0, 3):
            sel = np.sort(rng.choice(p.F, size=k2, replace=False)).astype(np.int32)
            y = p.y_empty()
            pb.prox_stage2_ffn(p.h, p.t_x[t], 1, torch.from_numpy(sel).cuda(), k2, y)
            torch.cuda.synchronize()
            y_ref, _ = po.stage2(p.x[t], sel, p.wg, p.wu, p.wd)
            rel = check_y(y.cpu().numpy()[0], y_ref)
            assert rel < 1e-4, rel        # fp32 accumulate, fp32 output: far inside the bound
    assert pb.prox_last_device_status(p.h) == 0


def test_stage2_dense_special_case(pb, toy):
    """k2 = d_ff: the path is the dense SwiGLU FFN (Sec. 2.1)."""
    wl, p = toy
    p.quantize(4, 0)
    y = p.y_empty()
    pb.prox_ffn_forward(p.h, p.t_x[1], 1, 100, p.F, y)
    y_ref, _ = po.dense_ffn(p.x[1], p.wg, p.wu, p.wd)
    assert check_y(y.cpu().numpy()[0], y_ref) < 1e-4


def test_stage2_bf16_output(pb):
    wl, wg, wu, wd, x = inputs.make_workload("toy", n_tokens=2)
    p = Problem(pb, wg, wu, wd, x, out_dtype=0)
    try:
        p.quantize(4, 0)
        sel = np.arange(0, p.F, 3, dtype=np.int32)
        y = p.y_empty()
        pb.prox_stage2_ffn(p.h, p.t_x[0], 1, torch.from_numpy(sel).cuda(), len(sel), y)
        y_ref, _ = po.stage2(p.x[0], sel, p.wg, p.wu, p.wd)
        got = y.float().cpu().numpy()[0]
        check_y(got, y_ref)
        # single rounding: equals bf16(oracle) up to one bf16 ulp where fp32 rounding straddles a tie
        want = inputs.bf16_bits_to_f32(po.f64_to_bf16_bits(y_ref))
        assert np.mean(got == want) > 0.99
        assert np.max(np.abs(got - want) / np.maximum(np.abs(want), 1e-30)) <= 2.0 ** -7
    finally:
        p.close()


def test_stage2_out_of_range_channel_is_skipped_and_recorded(pb, toy):
    wl, p = toy
    p.quantize(4, 0)
    sel = np.array([3, 10, p.F + 5, 2 ** 30], dtype=np.int32)
    y = p.y_empty()
    pb.prox_stage2_ffn(p.h, p.t_x[0], 1, torch.from_numpy(sel).cuda(), 4, y)
    assert pb.prox_last_device_status(p.h) & 1
    assert pb.prox_last_device_status(p.h) == 0      # reading clears
    y_ref, _ = po.stage2(p.x[0], sel[:2], p.wg, p.wu, p.wd)
    check_y(y.cpu().numpy()[0], y_ref)


# --------------------------------------------------------------- whole path
def _forward_check(pb, p, t, k1, k2, B=1):
    y = p.y_empty(B)
    sel = torch.empty(B, k2, dtype=torch.int32, device="cuda")
    xb = p.t_x[t:t + B]
    pb.prox_stage1_mask(p.h, xb, B, k1, k2, sel)
    pb.prox_ffn_forward(p.h, xb, B, k1, k2, y)
    used = torch.empty_like(sel)                     # the mask the forward call itself built
    pb.prox_ffn_last_mask(p.h, B, k2, used)
    torch.cuda.synchronize()
    sel_np, used_np, y_np = (sel.cpu().numpy().astype(np.int64), used.cpu().numpy().astype(np.int64),
                             y.float().cpu().numpy())
    nd = 0
    for b in range(B):
        idx, score, sel_ref, thr = p.oracle_stage1(t + b, k1, k2)
        nd += check_mask(sel_np[b], score, sel_ref, thr, k2, p.F)
        nd += check_mask(used_np[b], score, sel_ref, thr, k2, p.F)
        y_ref, _ = po.stage2(p.x[t + b], used_np[b], p.wg, p.wu, p.wd)
        check_y(y_np[b], y_ref)
    return nd


def _check_fused_stage1(pb, p, tx, x64, k1, k2):
    """The persistent kernel's own kept-input list and proxy scores against the oracle."""
    y = p.y_empty()
    pb.prox_ffn_forward(p.h, tx, 1, k1, k2, y)
    idx = torch.empty(k1, dtype=torch.int32, device="cuda")
    sc = torch.empty(p.F, dtype=torch.float32, device="cuda")
    pb.prox_ffn_last_stage1(p.h, k1, idx, sc)
    torch.cuda.synchronize()
    dg, du, _ = p.deq[p.fmt]
    idx_ref = po.input_topk(x64, k1)
    assert np.array_equal(idx.cpu().numpy().astype(np.int64), idx_ref), "kept inputs differ from the oracle"
    score = po.proxy_scores(x64, idx_ref, dg, du)
    _, thr = po.channel_topk(score, k2)
    err = float(np.max(np.abs(sc.cpu().numpy().astype(np.float64) - score)) / thr)
    assert err < 2e-4, err                # relative to the threshold score (fp32 sums, fast exp)
    return err


@pytest.mark.parametrize("bits,group", [(4, 0), (4, 128), (8, 0), (8, 128)])
def test_fused_kernel_own_input_list_and_scores(pb, toy, bits, group):
    wl, p = toy
    p.quantize(bits, group)
    k1, k2 = wl.points[50]
    for t in (0, 7, 19):
        _check_fused_stage1(pb, p, p.t_x[t], p.x[t], k1, k2)
    # hand-made ties among the magnitudes: the lower index must win inside the kernel too
    from tests.gpu_common import dev_bf16
    vals = np.array([1.0, -1.0, 0.5, 2.0, -2.0, 0.0, -0.0, 1.0], dtype=np.float32)
    x = np.tile(vals, p.D // 8)[None, :]
    tx = dev_bf16(inputs.f32_to_bf16_bits(x))
    for k1t in (1, 64, 65, 129, 300, p.D - 3):
        _check_fused_stage1(pb, p, tx, x[0].astype(np.float64), k1t, k2)
    # inputs spread over many binades (the integer form of x drops bits only far below the largest)
    xf = p.x[3].copy()
    xf[::7] *= 2.0 ** -20
    xf[5::11] *= 2.0 ** 9
    bits16 = inputs.f32_to_bf16_bits(xf.astype(np.float32)[None, :])
    _check_fused_stage1(pb, p, dev_bf16(bits16), po.bf16_to_f64(bits16)[0], k1, k2)
    assert pb.prox_last_device_status(p.h) == 0


def test_bounded_wait_runs_out_and_the_handle_recovers(pb, toy):
    """A grid barrier that cannot complete: every block gives up after a few hundred polls and leaves
    (nothing hangs, nothing faults); y is not written, the status says so, and the next call is ordinary."""
    wl, p = toy
    p.quantize(4, 128)
    k1, k2 = wl.points[50]
    y = torch.full((1, p.D), 7.0, dtype=torch.float32, device="cuda")
    pb.prox_debug_set_wait(p.h, 300, 1)
    try:
        pb.prox_ffn_forward(p.h, p.t_x[1], 1, k1, k2, y)
        torch.cuda.synchronize()
        status, code = pb.prox_last_device_status_raw(p.h)
        assert code & 4 and status == 6          # PROX_ERR_TIMEOUT
        assert torch.all(y == 7.0)               # untouched
        # the host-buffer entry point synchronises and reports the expiry itself
        xh = torch.from_numpy(p.bits["x"][1:2].view(np.int16)).view(torch.bfloat16).pin_memory()
        yh = torch.empty(1, p.D, dtype=torch.float32).pin_memory()
        with pytest.raises(pb.ProxError) as ei:
            pb.prox_ffn_forward_host(p.h, xh, 1, k1, k2, yh)
        assert ei.value.status == 6
    finally:
        pb.prox_debug_set_wait(p.h, 0, 0)
    assert pb.prox_last_device_status(p.h) == 0
    _forward_check(pb, p, 1, k1, k2)
    assert pb.prox_last_device_status(p.h) == 0


def test_forward_toy_all_tokens(pb, toy):
    wl, p = toy
    p.quantize(4, 0)
    k1, k2 = wl.points[50]
    for t in range(p.x.shape[0]):
        _forward_check(pb, p, t, k1, k2)
    assert pb.prox_last_device_status(p.h) == 0


@pytest.mark.parametrize("B", [2, 4, 8])
def test_forward_batched_per_token_masks(pb, toy, B):
    wl, p = toy
    p.quantize(4, 128)
    k1, k2 = wl.points[50]
    _forward_check(pb, p, 3, k1, k2, B=B)


@pytest.mark.parametrize("bits,group", [(4, 0), (4, 128), (8, 0)])
def test_union_and_per_token_batch_paths_agree(pb, toy, bits, group):
    """B > 1: one read of the weights for the union of the tokens' masks (on the tensor cores
    or with plain FMAs) must give every token the result of the per-token path (and of the oracle)."""
    wl, p = toy
    p.quantize(bits, group)
    k1, k2 = wl.points[50]
    B, t0 = 8, 8
    res = []
    for union in (2, 1, 0):          # tensor-core union kernels, CUDA-core union kernels, one token at a time
        pb.prox_ffn_set_union(p.h, union)
        y = p.y_empty(B)
        m = torch.empty(B, k2, dtype=torch.int32, device="cuda")
        pb.prox_ffn_forward(p.h, p.t_x[t0:t0 + B], B, k1, k2, y)
        pb.prox_ffn_last_mask(p.h, B, k2, m)
        torch.cuda.synchronize()
        res.append((y.cpu().numpy(), m.cpu().numpy().astype(np.int64)))
    pb.prox_ffn_set_union(p.h, 2)
    for b in range(B):
        idx, score, sel_ref, thr = p.oracle_stage1(t0 + b, k1, k2)
        for yv, mv in res:
            check_mask(mv[b], score, sel_ref, thr, k2, p.F)
            y_ref, _ = po.stage2(p.x[t0 + b], mv[b], p.wg, p.wu, p.wd)
            assert check_y(yv[b], y_ref) < 1e-4
    # stage-wise entry points on the union path, odd batch size
    B = 3
    sel = torch.empty(B, k2, dtype=torch.int32, device="cuda")
    sc = torch.empty(B, p.F, dtype=torch.float32, device="cuda")
    y = p.y_empty(B)
    pb.prox_stage1_mask(p.h, p.t_x[1:1 + B], B, k1, k2, sel, sc)
    pb.prox_stage2_ffn(p.h, p.t_x[1:1 + B], B, sel, k2, y)
    torch.cuda.synchronize()
    for b in range(B):
        idx, score, sel_ref, thr = p.oracle_stage1(1 + b, k1, k2)
        mv = sel.cpu().numpy()[b].astype(np.int64)
        check_mask(mv, score, sel_ref, thr, k2, p.F)
        assert float(np.max(np.abs(sc.cpu().numpy()[b] - score)) / thr) < 2e-4
        y_ref, _ = po.stage2(p.x[1 + b], mv, p.wg, p.wu, p.wd)
        assert check_y(y.cpu().numpy()[b], y_ref) < 1e-4
    assert pb.prox_last_device_status(p.h) == 0


@pytest.mark.parametrize("group", [0, 128])
def test_batch_tokens_of_very_different_magnitude(pb, group):
    """B = 8 on the tensor-core path: every token's x is scaled by its own power of two before it
    becomes fp16, so tokens whose magnitudes differ by dozens of binades still get the oracle's masks."""
    D, F, B = 512, 1024, 8
    wg, wu, wd, x = inputs.make_small(D, F, B, seed=77)
    xf = inputs.bf16_bits_to_f32(x).astype(np.float64)
    for b, e in enumerate((-40, -17, -3, 0, 5, 12, 25, 38)):
        xf[b] *= 2.0 ** e                              # exact in bf16: only the exponent moves
    x = inputs.f32_to_bf16_bits(xf.astype(np.float32))
    p = Problem(pb, wg, wu, wd, x, max_batch=B)
    try:
        p.quantize(4, group)
        k1, k2 = 154, 256
        _forward_check(pb, p, 0, k1, k2, B=B)
        sel = torch.empty(B, k2, dtype=torch.int32, device="cuda")
        sc = torch.empty(B, F, dtype=torch.float32, device="cuda")
        pb.prox_stage1_mask(p.h, p.t_x, B, k1, k2, sel, sc)
        torch.cuda.synchronize()
        for b in range(B):
            _, score, _, thr = p.oracle_stage1(b, k1, k2)
            assert float(np.max(np.abs(sc.cpu().numpy()[b] - score)) / thr) < 2e-4
        assert pb.prox_last_device_status(p.h) == 0
    finally:
        p.close()


def test_forward_host_buffers(pb, toy):
    wl, p = toy
    p.quantize(4, 0)
    k1, k2 = wl.points[50]
    xh = torch.from_numpy(p.bits["x"][2:3].view(np.int16)).view(torch.bfloat16).pin_memory()
    yh = torch.empty(1, p.D, dtype=torch.float32).pin_memory()
    pb.prox_ffn_forward_host(p.h, xh, 1, k1, k2, yh)
    y = p.y_empty()
    pb.prox_ffn_forward(p.h, p.t_x[2], 1, k1, k2, y)
    torch.cuda.synchronize()
    # same kernels, same mask; the fp32 atomics of the down projection may add in another order
    assert torch.allclose(yh, y.cpu(), rtol=0, atol=1e-5 * float(y.abs().max()))


def test_calls_are_repeatable(pb, toy):
    """Scratch (tickets, accumulators) is left clean: the same call twice gives the same bits
    for the mask, and outputs that differ only by fp32 atomic ordering."""
    wl, p = toy
    p.quantize(4, 0)
    k1, k2 = wl.points[50]
    s1 = torch.empty(1, k2, dtype=torch.int32, device="cuda")
    s2 = torch.empty_like(s1)
    y1, y2 = p.y_empty(), p.y_empty()
    pb.prox_stage1_mask(p.h, p.t_x[4], 1, k1, k2, s1)
    pb.prox_ffn_forward(p.h, p.t_x[4], 1, k1, k2, y1)
    pb.prox_stage1_mask(p.h, p.t_x[4], 1, k1, k2, s2)
    pb.prox_ffn_forward(p.h, p.t_x[4], 1, k1, k2, y2)
    assert torch.equal(s1, s2)
    assert torch.allclose(y1, y2, rtol=0, atol=1e-5 * float(y1.abs().max()))


@pytest.mark.parametrize("bits,group", [(4, 0), (4, 128), (8, 0), (8, 128)])
def test_fused_and_stepwise_paths_agree(pb, toy, bits, group):
    """B = 1 runs as one persistent kernel by default; the kernel-per-step path
    must give the same mask (up to the band) and the same y (up to fp32 order)."""
    wl, p = toy
    p.quantize(bits, group)
    k1, k2 = wl.points[50]
    for t in (0, 9, 31):
        outs = []
        for fused in (1, 0):
            pb.prox_ffn_set_fused(p.h, fused)
            y = p.y_empty()
            m = torch.empty(1, k2, dtype=torch.int32, device="cuda")
            pb.prox_ffn_forward(p.h, p.t_x[t], 1, k1, k2, y)
            pb.prox_ffn_last_mask(p.h, 1, k2, m)
            torch.cuda.synchronize()
            outs.append((y.cpu().numpy()[0], m.cpu().numpy()[0].astype(np.int64)))
        pb.prox_ffn_set_fused(p.h, 1)
        idx, score, sel_ref, thr = p.oracle_stage1(t, k1, k2)
        for yv, mv in outs:
            check_mask(mv, score, sel_ref, thr, k2, p.F)
            y_ref, _ = po.stage2(p.x[t], mv, p.wg, p.wu, p.wd)
            assert check_y(yv, y_ref) < 1e-4
    assert pb.prox_last_device_status(p.h) == 0


@pytest.mark.parametrize("k1,k2", [(512, 1536), (1, 1), (512, 1), (17, 1535), (300, 768), (16, 148), (33, 149)])
def test_fused_edge_budgets(pb, toy, k1, k2):
    wl, p = toy
    p.quantize(4, 128)
    for t in (2, 7):
        _forward_check(pb, p, t, k1, k2)
    assert pb.prox_last_device_status(p.h) == 0


def test_fused_random_budgets(pb, toy):
    """Seeded random (k1, k2) pairs, group-128 proxies: the persistent kernel against the oracle."""
    wl, p = toy
    p.quantize(4, 128)
    rng = np.random.default_rng(2024)
    for _ in range(16):
        k1 = int(rng.integers(1, p.D + 1))
        k2 = int(rng.integers(1, p.F + 1))
        _forward_check(pb, p, int(rng.integers(0, p.x.shape[0])), k1, k2)
    assert pb.prox_last_device_status(p.h) == 0


def test_batch_random_budgets(pb, toy):
    """Seeded random batch sizes and budgets on the tensor-core union path."""
    wl, p = toy
    p.quantize(4, 0)
    rng = np.random.default_rng(7)
    for _ in range(8):
        B = int(rng.integers(2, 9))
        k1 = int(rng.integers(1, p.D + 1))
        k2 = int(rng.integers(1, p.F + 1))
        _forward_check(pb, p, int(rng.integers(0, p.x.shape[0] - B + 1)), k1, k2, B=B)
    assert pb.prox_last_device_status(p.h) == 0


@pytest.mark.parametrize("bits,group", [(4, 0), (4, 128), (8, 0), (8, 128)])
def test_batch_edge_budgets_and_scores_all_formats(pb, toy, bits, group):
    """The tensor-core Stage 1 of the batch path at the corners of the budget, for every integer format: masks and
    outputs through the forward call, and the scores themselves (asked for explicitly) against the oracle."""
    wl, p = toy
    dg, du, _ = p.quantize(bits, group)
    for B, t0 in ((2, 0), (8, 5)):
        for k1, k2 in ((p.D, p.F), (1, 1), (p.D, 1), (17, p.F - 1), (154, 358)):
            _forward_check(pb, p, t0, k1, k2, B=B)
        k1, k2 = 154, 358
        sel = torch.empty(B, k2, dtype=torch.int32, device="cuda")
        sc = torch.empty(B, p.F, dtype=torch.float32, device="cuda")
        pb.prox_stage1_mask(p.h, p.t_x[t0:t0 + B], B, k1, k2, sel, sc)
        torch.cuda.synchronize()
        for b in range(B):
            idx, score, sel_ref, thr = p.oracle_stage1(t0 + b, k1, k2)
            assert float(np.max(np.abs(sc.cpu().numpy()[b] - score)) / thr) < 2e-4
    assert pb.prox_last_device_status(p.h) == 0


@pytest.mark.parametrize("bits,group,B", [(4, 128, 5), (8, 0, 8), (4, 0, 2)])
def test_batch_stage1_over_several_units_and_items(pb, bits, group, B):
    """A layer wide and deep enough that a block of the batched proxy GEMM takes several items of several units
    each (reuse of ring stages and of the accumulator sets): scores and masks against the oracle."""
    D, F, k1, k2 = 2048, 4096, 614, 942
    wg, wu, wd, x = inputs.make_small(D, F, 9, seed=D + F + bits)
    p = Problem(pb, wg, wu, wd, x, max_batch=8)
    try:
        p.quantize(bits, group)
        sel = torch.empty(B, k2, dtype=torch.int32, device="cuda")
        sc = torch.empty(B, F, dtype=torch.float32, device="cuda")
        for rep in range(2):                        # twice: the accumulator in global memory must come back clean
            pb.prox_stage1_mask(p.h, p.t_x[:B], B, k1, k2, sel, sc)
            torch.cuda.synchronize()
            for b in range(B):
                idx, score, sel_ref, thr = p.oracle_stage1(b, k1, k2)
                assert float(np.max(np.abs(sc.cpu().numpy()[b] - score)) / thr) < 2e-4, (rep, b)
                check_mask(sel.cpu().numpy()[b].astype(np.int64), score, sel_ref, thr, k2, F)
        _forward_check(pb, p, 1, k1, k2, B=B)
        assert pb.prox_last_device_status(p.h) == 0
    finally:
        p.close()


def test_fused_all_zero_input(pb, toy):
    """x = 0: every score ties at 0; the mask must be the first k2 channels and y = 0."""
    wl, p = toy
    p.quantize(4, 0)
    k1, k2 = wl.points[50]
    xz = torch.zeros(1, p.D, dtype=torch.bfloat16, device="cuda")
    y = p.y_empty()
    m = torch.empty(1, k2, dtype=torch.int32, device="cuda")
    pb.prox_ffn_forward(p.h, xz, 1, k1, k2, y)
    pb.prox_ffn_last_mask(p.h, 1, k2, m)
    torch.cuda.synchronize()
    assert np.array_equal(m.cpu().numpy()[0], np.arange(k2))
    assert float(y.abs().max()) == 0.0


@pytest.mark.parametrize("D,F,k1,k2,bits,group", [
    (16384, 1024, 4915, 239, 4, 128),      # widest d_model the library takes (fused kernel not used: step-wise path)
    (128, 65536, 38, 15270, 4, 0),         # narrowest d_model, widest d_ff (scores do not fit in shared memory)
    (128, 65536, 128, 45000, 4, 0),        # ... with more than 256 channels per block (two batches of the ring)
    (128, 40960, 38, 39000, 4, 128),       # scores in shared memory, more than 256 channels per block
    (8192, 320, 2458, 75, 8, 128),         # ragged last strip, 8-bit codes, two down-projection groups
    (384, 448, 115, 104, 4, 128),          # sizes that are no multiple of the strip or chunk steps
    (128, 64, 38, 15, 4, 0),               # the smallest layer the library takes (a proxy row is half a tile wide)
    (256, 64, 77, 15, 8, 128),             # ... with 8-bit codes and two scale groups
])
def test_extreme_shapes(pb, D, F, k1, k2, bits, group):
    wg, wu, wd, x = inputs.make_small(D, F, 3, seed=D + F)
    p = Problem(pb, wg, wu, wd, x, max_batch=2)
    try:
        p.quantize(bits, group)
        for t in range(2):
            _forward_check(pb, p, t, k1, k2)
        _forward_check(pb, p, 1, k1, k2, B=2)
        assert pb.prox_last_device_status(p.h) == 0
    finally:
        p.close()


# --------------------------------------------------------- threshold variant
def test_threshold_variant(pb, toy):
    wl, p = toy
    dg, du, _ = p.quantize(4, 0)
    k1, k2 = wl.points[50]
    t = 6
    idx, score, sel_ref, thr = p.oracle_stage1(t, k1, k2)
    mags = np.sort(np.abs(p.x[t]))[::-1]
    tau_x = float((mags[k1 - 1] + mags[k1]) / 2) if mags[k1 - 1] != mags[k1] else float(mags[k1 - 1])
    idx_t = po.input_threshold(p.x[t], np.float32(tau_x))
    score_t = po.proxy_scores(p.x[t], idx_t, dg, du)
    srt = np.sort(score_t)[::-1]
    tau_s = float(np.float32((srt[k2 - 1] + srt[k2]) / 2))
    sel_t = po.channel_threshold(score_t, tau_s)
    sel = torch.empty(1, p.F, dtype=torch.int32, device="cuda")
    cnt = torch.empty(1, dtype=torch.int32, device="cuda")
    y = p.y_empty()
    pb.prox_runtime_sparsity(p.h, reset=True)
    pb.prox_stage1_mask_threshold(p.h, p.t_x[t], 1, tau_x, tau_s, sel, cnt)
    pb.prox_stage2_ffn_var(p.h, p.t_x[t], 1, sel, cnt, y)
    torch.cuda.synchronize()
    n = int(cnt.item())
    got = sel.cpu().numpy()[0, :n].astype(np.int64)
    near = np.abs(score_t - tau_s) <= 1e-3 * tau_s
    assert np.all(near[np.setxor1d(got, sel_t)])
    y_ref, _ = po.stage2(p.x[t], got, p.wg, p.wu, p.wd)
    check_y(y.cpu().numpy()[0], y_ref)
    tok, s1h, s2h, eh = pb.prox_runtime_sparsity(p.h)
    assert tok == 1 and abs(s1h - (1 - len(idx_t) / p.D)) < 1e-12 and abs(s2h - (1 - n / p.F)) < 1e-12
    assert abs(eh - po.effective_sparsity(s1h, s2h)) < 1e-12
    y2 = p.y_empty()
    pb.prox_ffn_forward_threshold(p.h, p.t_x[t], 1, tau_x, tau_s, y2)
    assert torch.allclose(y, y2, rtol=0, atol=1e-5 * float(y.abs().max()))


@pytest.mark.parametrize("bits,group", [(4, 0), (4, 128), (8, 0)])
def test_threshold_forward_in_one_launch(pb, toy, bits, group):
    """prox_ffn_forward_threshold at batch 1 is the persistent kernel in its threshold form: masks by
    |x| >= tau_x and score >= tau_s (Sec. 4.1 indicators), counts vary per token."""
    wl, p = toy
    dg, du, _ = p.quantize(bits, group)
    k1, k2 = wl.points[50]
    launches = 0
    for t in (0, 3, 11, 20):
        mags = np.sort(np.abs(p.x[t]))[::-1]
        for tau_x, frac in ((float(mags[k1 - 1]), 0.3), (0.0, 0.6), (float(mags[5]), 0.05)):
            idx_t = po.input_threshold(p.x[t], np.float32(tau_x))
            score_t = po.proxy_scores(p.x[t], idx_t, dg, du)
            srt = np.sort(score_t)[::-1]
            kk = max(1, int(frac * p.F))
            tau_s = float(np.float32((srt[kk - 1] + srt[kk]) / 2))
            sel_t = po.channel_threshold(score_t, tau_s)
            y = p.y_empty()
            pb.prox_runtime_sparsity(p.h, reset=True)
            l0 = pb.prox_launch_count(p.h)
            pb.prox_ffn_forward_threshold(p.h, p.t_x[t], 1, tau_x, tau_s, y)
            launches = pb.prox_launch_count(p.h) - l0
            torch.cuda.synchronize()
            tok, s1h, s2h, _ = pb.prox_runtime_sparsity(p.h)
            n_in, n = int(round((1 - s1h) * p.D)), int(round((1 - s2h) * p.F))
            assert tok == 1 and n_in == len(idx_t), (n_in, len(idx_t))
            got = np.empty(0, dtype=np.int64)
            if n > 0:
                used = torch.empty(1, n, dtype=torch.int32, device="cuda")
                pb.prox_ffn_last_mask(p.h, 1, n, used)
                got = used.cpu().numpy()[0].astype(np.int64)
                assert np.all(got[1:] > got[:-1])
            near = np.abs(score_t - tau_s) <= 1e-3 * tau_s
            assert np.all(near[np.setxor1d(got, sel_t)])
            y_ref, _ = po.stage2(p.x[t], got, p.wg, p.wu, p.wd)
            check_y(y.cpu().numpy()[0], y_ref, extra_abs=1e-30)
    assert launches == 1
    # nothing passes tau_x: all scores are 0; with tau_s = 0 every channel passes and y is the dense FFN
    y = p.y_empty()
    pb.prox_ffn_forward_threshold(p.h, p.t_x[2], 1, 1e30, 0.0, y)
    torch.cuda.synchronize()
    y_dense, _ = po.dense_ffn(p.x[2], p.wg, p.wu, p.wd)
    check_y(y.cpu().numpy()[0], y_dense)
    # nothing passes tau_s: y = 0
    pb.prox_ffn_forward_threshold(p.h, p.t_x[2], 1, 0.5, 1e30, y)
    torch.cuda.synchronize()
    assert float(y.abs().max()) == 0.0
    assert pb.prox_last_device_status(p.h) == 0


# ------------------------------------------------------------- pack save/load
# ------------------------------------------------------------ ablation forms
@pytest.mark.parametrize("B", [1, 3, 8])
def test_sixteen_bit_proxy_forward(pb, toy, B):
    """Ablation A1: the original bf16 weights, input-major, as the proxy."""
    wl, p = toy
    p.quantize(16, 0)
    k1, k2 = wl.points[50]
    for t in (0, 9):
        _forward_check(pb, p, t, k1, k2, B=B)
    _forward_check(pb, p, 1, p.D, 300, B=B)          # exact scores: the mask is the top-k of |s|
    assert pb.prox_last_device_status(p.h) == 0
    R = pb.raw
    assert R("prox_quantize_proxy")(p.h, 16, 128, None) == 2
    q = np.empty((p.F, p.D), dtype=np.int8)
    s = np.empty((p.F, 1), dtype=np.float32)
    assert R("prox_proxy_export")(p.h, 0, q.ctypes.data, s.ctypes.data) == 2


@pytest.mark.parametrize("bits,group,B", [(4, 0, 1), (4, 128, 4), (8, 0, 2), (16, 0, 1), (16, 0, 8)])
def test_proxy_values_into_down(pb, toy, bits, group, B):
    """Ablation A3 (with 16-bit proxies: input sparsity on x, then on s): the selected proxy values
    enter the down projection."""
    wl, p = toy
    dg, du, _ = p.quantize(bits, group)
    for k1, k2 in (wl.points[50], (p.D, p.F), (37, 1)):
        t = 5
        y = p.y_empty(B)
        used = torch.empty(B, k2, dtype=torch.int32, device="cuda")
        pb.prox_ffn_forward_proxy_values(p.h, p.t_x[t:t + B], B, k1, k2, y)
        pb.prox_ffn_last_mask(p.h, B, k2, used)
        torch.cuda.synchronize()
        used_np, y_np = used.cpu().numpy().astype(np.int64), y.float().cpu().numpy()
        for b in range(B):
            idx, score, sel_ref, thr = p.oracle_stage1(t + b, k1, k2)
            check_mask(used_np[b], score, sel_ref, thr, k2, p.F)
            vals = po.proxy_values(p.x[t + b], idx, dg, du)
            y_ref = p.wd[:, used_np[b]].astype(np.float64) @ vals[used_np[b]]
            check_y(y_np[b], y_ref)
            if k1 == p.D and k2 == p.F and bits == 16:       # nothing dropped, exact proxy: the dense FFN
                y_dense, _ = po.dense_ffn(p.x[t + b], p.wg, p.wu, p.wd)
                check_y(y_np[b], y_dense)
    assert pb.prox_last_device_status(p.h) == 0


# ------------------------------------------------------- layer sub-block, stacks
def _norm_weight(D, seed):
    rng = np.random.default_rng(seed)
    return inputs.f32_to_bf16_bits((1.0 + 0.1 * rng.standard_normal(D)).astype(np.float32))


def _check_block(p, dg, du, x_in, nw64, eps, k1, k2, x_out, used):
    """One token of one layer: GPU result x_out against the oracle fed with the same residual stream."""
    xn = po.bf16_to_f64(po.f64_to_bf16_bits(po.rmsnorm(x_in, nw64, eps)))
    idx = po.input_topk(xn, k1)
    score = po.proxy_scores(xn, idx, dg, du)
    sel_ref, thr = po.channel_topk(score, k2)
    check_mask(used, score, sel_ref, thr, k2, p.F)
    y_ref, _ = po.stage2(xn, used, p.wg, p.wu, p.wd)
    # x_out = fp32(x_in + y): the add rounds once more, to fp32
    check_y(x_out.astype(np.float64) - x_in, y_ref, extra_abs=float(np.max(np.abs(x_out))) * 2.0 ** -23)


@pytest.mark.parametrize("bits,group,B", [(4, 128, 1), (4, 0, 1), (8, 0, 1), (4, 128, 3), (8, 128, 8), (16, 0, 1)])
def test_ffn_block_forward(pb, toy, bits, group, B):
    wl, p = toy
    dg, du, _ = p.quantize(bits, group)
    k1, k2 = wl.points[50]
    eps = 1e-6
    nw_bits = _norm_weight(p.D, 4)
    nw64 = po.bf16_to_f64(nw_bits)
    from tests.gpu_common import dev_bf16
    t_nw = dev_bf16(nw_bits)
    rng = np.random.default_rng(8)
    x_res = (p.x[2:2 + B] * 3.7 + rng.standard_normal((B, p.D))).astype(np.float32)
    t_x = torch.from_numpy(x_res).cuda()
    out = torch.empty_like(t_x)
    used = torch.empty(B, k2, dtype=torch.int32, device="cuda")
    pb.prox_ffn_block_forward(p.h, t_x, t_nw, eps, B, k1, k2, out)
    pb.prox_ffn_last_mask(p.h, B, k2, used)
    inplace = t_x.clone()
    pb.prox_ffn_block_forward(p.h, inplace, t_nw, eps, B, k1, k2, inplace)
    torch.cuda.synchronize()
    assert torch.equal(t_x.cpu(), torch.from_numpy(x_res)), "the input stream was written"
    out_np, used_np = out.cpu().numpy(), used.cpu().numpy().astype(np.int64)
    for b in range(B):
        _check_block(p, dg, du, x_res[b].astype(np.float64), nw64, eps, k1, k2, out_np[b], used_np[b])
    np.testing.assert_allclose(inplace.cpu().numpy(), out_np, rtol=1e-5, atol=1e-5)
    assert pb.prox_last_device_status(p.h) == 0


@pytest.mark.parametrize("B", [1, 2])
def test_ffn_stack_forward_layer_by_layer(pb, B):
    """Three layers in place on one stream; every layer is checked against the oracle on the stream the
    GPU itself fed into it (the trace), so a mask difference inside the band in one layer does not
    make the next one incomparable."""
    from tests.gpu_common import dev_bf16
    L, D, F = 3, 512, 1536
    probs = []
    try:
        for l in range(L):
            wg, wu, wd, x = inputs.make_small(D, F, 4, seed=40 + l)
            probs.append(Problem(pb, wg, wu, wd, x, max_batch=2))
        deqs = [q.quantize(4, 128) for q in probs]
        nw_bits = np.stack([_norm_weight(D, 50 + l) for l in range(L)])
        t_nw = dev_bf16(nw_bits)
        k1, k2, eps = 154, 358, 1e-6
        x0 = (probs[0].x[:B] * 2.0).astype(np.float32)
        t_x = torch.from_numpy(x0).cuda()
        trace = torch.zeros(L + 1, B, D, dtype=torch.float32, device="cuda")
        pb.prox_ffn_stack_forward([q.h for q in probs], t_nw, eps, t_x, B, k1, k2, trace)
        torch.cuda.synchronize()
        tr = trace.cpu().numpy()
        assert np.array_equal(tr[0], x0) and np.array_equal(tr[L], t_x.cpu().numpy())
        # layer by layer, with the mask each layer used (asked for by re-running the layer on its input)
        for l in range(L):
            out = torch.empty(B, D, dtype=torch.float32, device="cuda")
            used = torch.empty(B, k2, dtype=torch.int32, device="cuda")
            pb.prox_ffn_block_forward(probs[l].h, trace[l], t_nw[l], eps, B, k1, k2, out)
            pb.prox_ffn_last_mask(probs[l].h, B, k2, used)
            torch.cuda.synchronize()
            np.testing.assert_allclose(out.cpu().numpy(), tr[l + 1], rtol=1e-5, atol=1e-5)
            dg, du, _ = deqs[l]
            for b in range(B):
                _check_block(probs[l], dg, du, tr[l, b].astype(np.float64), po.bf16_to_f64(nw_bits[l]), eps, k1, k2,
                             tr[l + 1, b], used.cpu().numpy()[b].astype(np.int64))
        # and the oracle's own stack from the same start stays close while no mask differs
        layers = [(po.bf16_to_f64(nw_bits[l]), deqs[l][0], deqs[l][1], probs[l].wg, probs[l].wu, probs[l].wd)
                  for l in range(L)]
        xs = po.ffn_stack(x0[0].astype(np.float64), layers, eps, k1, k2)
        assert np.sqrt(np.mean((xs[L] - tr[L, 0]) ** 2)) <= 0.05 * np.sqrt(np.mean((xs[L] - xs[0]) ** 2)) + 1e-6
        for q in probs:
            assert pb.prox_last_device_status(q.h) == 0
    finally:
        for q in probs:
            q.close()


@pytest.mark.parametrize("B", [1, 2])
def test_ffn_stack_forward_threshold_layer_by_layer(pb, B):
    """The layer sub-block with thresholded masks (at B = 1 one launch per layer), three layers in place."""
    from tests.gpu_common import dev_bf16
    L, D, F = 3, 512, 1536
    probs = []
    try:
        for l in range(L):
            wg, wu, wd, x = inputs.make_small(D, F, 4, seed=60 + l)
            probs.append(Problem(pb, wg, wu, wd, x, max_batch=2))
        deqs = [q.quantize(4, 128) for q in probs]
        nw_bits = np.stack([_norm_weight(D, 70 + l) for l in range(L)])
        nw64 = [po.bf16_to_f64(nw_bits[l]) for l in range(L)]
        t_nw = dev_bf16(nw_bits)
        eps = 1e-6
        x0 = (probs[0].x[:B] * 2.0).astype(np.float32)
        # thresholds from the oracle's own top-k stack of token 0: between the k-th and the next value
        k1, k2 = 154, 358
        layers = [(nw64[l], deqs[l][0], deqs[l][1], probs[l].wg, probs[l].wu, probs[l].wd) for l in range(L)]
        xs = po.ffn_stack(x0[0].astype(np.float64), layers, eps, k1, k2)
        tau_x, tau_s = [], []
        for l in range(L):
            xn = po.bf16_to_f64(po.f64_to_bf16_bits(po.rmsnorm(xs[l], nw64[l], eps)))
            mags = np.sort(np.abs(xn))[::-1]
            tau_x.append(float(np.float32(mags[k1 - 1])))
            sc = np.sort(po.proxy_scores(xn, po.input_threshold(xn, np.float32(tau_x[-1])), deqs[l][0], deqs[l][1]))[::-1]
            tau_s.append(float(np.float32((sc[k2 - 1] + sc[k2]) / 2)))
        t_x = torch.from_numpy(x0).cuda()
        trace = torch.zeros(L + 1, B, D, dtype=torch.float32, device="cuda")
        l0 = sum(pb.prox_launch_count(q.h) for q in probs)
        pb.prox_ffn_stack_forward_threshold([q.h for q in probs], t_nw, eps, t_x, B, tau_x, tau_s, trace)
        torch.cuda.synchronize()
        if B == 1:
            assert sum(pb.prox_launch_count(q.h) for q in probs) - l0 == L      # one launch per layer
        tr = trace.cpu().numpy()
        assert np.array_equal(tr[0], x0) and np.array_equal(tr[L], t_x.cpu().numpy())
        for l in range(L):
            dg, du, _ = deqs[l]
            for b in range(B):
                x_in = tr[l, b].astype(np.float64)
                xn = po.bf16_to_f64(po.f64_to_bf16_bits(po.rmsnorm(x_in, nw64[l], eps)))
                idx = po.input_threshold(xn, np.float32(tau_x[l]))
                score = po.proxy_scores(xn, idx, dg, du)
                sel_t = po.channel_threshold(score, tau_s[l])
                # y of this layer from the oracle on its own mask; a channel inside the band may differ:
                # bound the difference by the contribution of the band channels
                y_ref, s_sp = po.stage2(xn, sel_t, probs[l].wg, probs[l].wu, probs[l].wd)
                near = np.nonzero(np.abs(score - tau_s[l]) <= 1e-3 * tau_s[l])[0]
                slack = 0.0
                if len(near):
                    _, s_near = po.stage2(xn, near, probs[l].wg, probs[l].wu, probs[l].wd)
                    slack = float(np.sum(np.abs(s_near)) * np.max(np.abs(probs[l].wd)))
                check_y(tr[l + 1, b].astype(np.float64) - x_in, y_ref,
                        extra_abs=slack + float(np.max(np.abs(tr[l + 1, b]))) * 2.0 ** -23)
        for q in probs:
            assert pb.prox_last_device_status(q.h) == 0
    finally:
        for q in probs:
            q.close()


@pytest.mark.parametrize("D,F,bits,group", [(128, 64, 4, 0), (256, 320, 4, 128), (384, 1984, 8, 0), (1024, 4096, 4, 128),
                                            (640, 2112, 8, 128)])
def test_forms_on_odd_shapes(pb, D, F, bits, group):
    """Threshold form, layer sub-block form and both together on shapes with ragged strips and few channels
    per block, seeded random budgets."""
    from tests.gpu_common import dev_bf16
    wg, wu, wd, x = inputs.make_small(D, F, 4, seed=D + F)
    p = Problem(pb, wg, wu, wd, x, max_batch=2)
    try:
        dg, du, _ = p.quantize(bits, group)
        rng = np.random.default_rng(D * 7 + F)
        nw_bits = _norm_weight(D, 3)
        nw64 = po.bf16_to_f64(nw_bits)
        t_nw = dev_bf16(nw_bits)
        for trial in range(4):
            k1 = int(rng.integers(1, D + 1))
            k2 = int(rng.integers(1, F + 1))
            t = trial % 4
            # the persistent kernel's own input list and scores at this shape and budget
            _check_fused_stage1(pb, p, p.t_x[t], p.x[t], k1, k2)
            # layer sub-block, top-k
            x_res = (p.x[t] * 1.3).astype(np.float32)[None, :]
            t_x = torch.from_numpy(x_res).cuda()
            out = torch.empty_like(t_x)
            used = torch.empty(1, k2, dtype=torch.int32, device="cuda")
            pb.prox_ffn_block_forward(p.h, t_x, t_nw, 1e-5, 1, k1, k2, out)
            pb.prox_ffn_last_mask(p.h, 1, k2, used)
            torch.cuda.synchronize()
            _check_block(p, dg, du, x_res[0].astype(np.float64), nw64, 1e-5, k1, k2, out.cpu().numpy()[0],
                         used.cpu().numpy()[0].astype(np.int64))
            # threshold form on the plain input and on the layer sub-block
            mags = np.sort(np.abs(p.x[t]))[::-1]
            tau_x = float(mags[k1 - 1])
            idx_t = po.input_threshold(p.x[t], np.float32(tau_x))
            score_t = po.proxy_scores(p.x[t], idx_t, dg, du)
            srt = np.sort(score_t)[::-1]
            tau_s = float(np.float32(srt[k2 - 1] if k2 == F else (srt[k2 - 1] + srt[k2]) / 2))
            sel_t = po.channel_threshold(score_t, tau_s)
            y = p.y_empty()
            pb.prox_runtime_sparsity(p.h, reset=True)
            pb.prox_ffn_forward_threshold(p.h, p.t_x[t], 1, tau_x, tau_s, y)
            torch.cuda.synchronize()
            tok, s1h, s2h, _ = pb.prox_runtime_sparsity(p.h)
            n_in, n = int(round((1 - s1h) * D)), int(round((1 - s2h) * F))
            assert n_in == len(idx_t)
            got = np.empty(0, dtype=np.int64)
            if n > 0:
                u2 = torch.empty(1, n, dtype=torch.int32, device="cuda")
                pb.prox_ffn_last_mask(p.h, 1, n, u2)
                got = u2.cpu().numpy()[0].astype(np.int64)
            near = np.abs(score_t - tau_s) <= 1e-3 * tau_s
            assert np.all(near[np.setxor1d(got, sel_t)])
            y_ref, _ = po.stage2(p.x[t], got, p.wg, p.wu, p.wd)
            check_y(y.cpu().numpy()[0], y_ref, extra_abs=1e-30)
        assert pb.prox_last_device_status(p.h) == 0
    finally:
        p.close()


def test_dff_shard_over_the_library_with_one_rank(pb, toy):
    """The d_ff-sharded form with a single rank (no process group): the library's scores -> the exchange's global
    top-k2 -> the library's Stage 2 on that list.  Same acceptance rule as the plain forward call."""
    from paper_2607_27591_b200 import sharded
    wl, p = toy
    from tests.gpu_common import dev_bf16
    k1, k2 = wl.points[50]
    sh = sharded.ShardedProxFFN(p.D, p.F, dev_bf16(p.bits["wg"]), dev_bf16(p.bits["wu"]), dev_bf16(p.bits["wd"]), 4, 128)
    try:
        dg, du, _ = p.quantize(4, 128)
        for t in (0, 3):
            sel, y = sh.forward(p.t_x[t], k1, k2)
            torch.cuda.synchronize()
            idx, score, sel_ref, thr = p.oracle_stage1(t, k1, k2)
            sel_np = sel.cpu().numpy().astype(np.int64)
            check_mask(sel_np, score, sel_ref, thr, k2, p.F)
            y_ref, _ = po.stage2(p.x[t], sel_np, p.wg, p.wu, p.wd)
            check_y(y.cpu().numpy(), y_ref)
    finally:
        sh.close()


def test_calibration_state_matches_the_oracle(pb):
    """Reservoir, quantile and histogram of the library (host side, fed from device buffers) against the oracle's,
    value for value: below and above the capacity, bf16 and fp32 samples, in two pieces."""
    rng = np.random.default_rng(12)
    v32 = rng.standard_normal(5000).astype(np.float32) * 3
    bits = po.f64_to_bf16_bits(rng.laplace(size=3000))
    from tests.gpu_common import dev_bf16
    t32, t16 = torch.from_numpy(v32).cuda(), dev_bf16(bits)
    for cap in (100000, 700):
        c = pb.prox_calib_create(cap, 5)
        try:
            pb.prox_calib_add(c, t32[:1234], 1234, 1)
            pb.prox_calib_add(c, t32[1234:], 5000 - 1234, 1)
            pb.prox_calib_add(c, t16, 3000, 0)
            res, seen = po.reservoir(v32, cap, 5)
            res, seen = po.reservoir(po.bf16_to_f64(bits), cap, 5, state=(res, seen))
            assert pb.prox_calib_seen(c) == (8000, min(cap, 8000))
            for s_ in (0.0, 0.1, 0.55, 0.7, 0.767, 1.0):
                assert np.float32(pb.prox_calib_threshold(c, s_)) == po.empirical_quantile(res, s_)
            counts, hi = pb.prox_calib_histogram(c)
            ref_counts, ref_hi = po.histogram_4096(res)
            assert np.float32(hi) == ref_hi and np.array_equal(np.asarray(counts), ref_counts)
        finally:
            pb.prox_calib_destroy(c)
    # error paths: empty reservoir, bad level
    c = pb.prox_calib_create(10, 0)
    try:
        tau = pb._f()
        assert pb.raw("prox_calib_threshold")(c, 0.5, tau) == 2            # UNSUPPORTED: nothing sampled
        pb.prox_calib_add(c, t32, 5, 1)
        assert pb.raw("prox_calib_threshold")(c, 1.5, tau) == 1            # INVALID_ARG
    finally:
        pb.prox_calib_destroy(c)


def test_sequential_threshold_calibration_of_a_stack(pb):
    """Alg. 1 through the library (RMSNorm -> tau_x -> proxy scores -> tau_s -> advance under the finalized
    rule, layer after layer) against the oracle's calibrate_stack on the same tokens.  Layer 0 sees the same
    inputs on both sides; later layers see streams that may differ where a score sits inside the threshold band,
    so their thresholds are compared with a tolerance and through the sparsities they realise on the GPU's stream."""
    from tests.gpu_common import dev_bf16
    L, D, F, N = 3, 512, 1536, 12
    probs = []
    try:
        for l in range(L):
            wg, wu, wd, x = inputs.make_small(D, F, N, seed=80 + l)
            probs.append(Problem(pb, wg, wu, wd, x, max_batch=1))
        deqs = [q.quantize(4, 128) for q in probs]
        nw_bits = np.stack([_norm_weight(D, 90 + l) for l in range(L)])
        nw64 = [po.bf16_to_f64(nw_bits[l]) for l in range(L)]
        t_nw = dev_bf16(nw_bits)
        eps, s1, s2 = 1e-6, 0.55, 0.7
        x0 = (probs[0].x[:N] * 2.0).astype(np.float32)
        t_x = torch.from_numpy(x0).cuda()
        tau_x, tau_s, hists = pb.prox_calibrate_stack([q.h for q in probs], F, t_nw, eps, t_x, s1, s2)
        assert torch.equal(t_x.cpu(), torch.from_numpy(x0))
        layers = [(nw64[l], deqs[l][0], deqs[l][1], probs[l].wg, probs[l].wu, probs[l].wd) for l in range(L)]
        cal = po.calibrate_stack(x0.astype(np.float64), layers, eps, s1, s2)
        # layer 0: the FFN inputs are bf16 values; the fp32 RMSNorm may round a handful of them to the neighbour
        assert abs(tau_x[0] - float(cal[0]["tau_x"])) <= 2.0 ** -7 * float(cal[0]["tau_x"])
        assert abs(tau_s[0] - float(cal[0]["tau_s"])) <= 2e-3 * float(cal[0]["tau_s"])
        for l in range(L):
            assert abs(tau_x[l] - float(cal[l]["tau_x"])) <= 0.02 * float(cal[l]["tau_x"])
            assert abs(tau_s[l] - float(cal[l]["tau_s"])) <= 0.05 * float(cal[l]["tau_s"])
            (cx, hx), (cs, hs) = hists[l]
            assert sum(cx) == N * D and sum(cs) == N * F and hx > 0 and hs > 0
        # the thresholds realise their targets on the calibration tokens when the stack then runs with them
        for q in probs:
            pb.prox_runtime_sparsity(q.h, reset=True)
        for i in range(N):
            xi = t_x[i:i + 1].clone()
            pb.prox_ffn_stack_forward_threshold([q.h for q in probs], t_nw, eps, xi, 1, tau_x, tau_s)
        torch.cuda.synchronize()
        for q in probs:
            tok, s1h, s2h, _ = pb.prox_runtime_sparsity(q.h)
            assert tok == N
            # bf16 inputs: about ten samples share the magnitude at the threshold (spacing 2^-8 of the value)
            assert abs(s1h - s1) <= 24.0 / (N * D) + 1e-9 and abs(s2h - s2) <= 3.0 / (N * F) + 1e-9
            assert pb.prox_last_device_status(q.h) == 0
    finally:
        for q in probs:
            q.close()


@pytest.mark.parametrize("bits,group,B", [(4, 0, 2), (4, 128, 5), (4, 128, 8), (8, 0, 8), (8, 128, 3)])
def test_shared_batch_mask_policy(pb, toy, bits, group, B):
    """One channel mask for the batch, from the summed proxy scores; Stage 2 of every token on that mask."""
    wl, p = toy
    dg, du, _ = p.quantize(bits, group)
    k1, k2 = wl.points[50]
    t0 = 4
    pb.prox_ffn_set_mask_policy(p.h, 1)
    try:
        y = p.y_empty(B)
        sel = torch.empty(B, k2, dtype=torch.int32, device="cuda")
        used = torch.empty(B, k2, dtype=torch.int32, device="cuda")
        xb = p.t_x[t0:t0 + B]
        pb.prox_stage1_mask(p.h, xb, B, k1, k2, sel)
        pb.prox_ffn_forward(p.h, xb, B, k1, k2, y)
        pb.prox_ffn_last_mask(p.h, B, k2, used)
        torch.cuda.synchronize()
        sel_ref, thr, shared, _ = po.forward_batch_shared(p.x[t0:t0 + B], k1, k2, dg, du, p.wg, p.wu, p.wd)
        sel_np, used_np, y_np = sel.cpu().numpy().astype(np.int64), used.cpu().numpy().astype(np.int64), y.cpu().numpy()
        for b in range(B):
            assert np.array_equal(sel_np[b], sel_np[0]) and np.array_equal(used_np[b], used_np[0])
            check_mask(sel_np[b], shared, sel_ref, thr, k2, p.F)
            check_mask(used_np[b], shared, sel_ref, thr, k2, p.F)
            y_ref, _ = po.stage2(p.x[t0 + b], used_np[b], p.wg, p.wu, p.wd)
            check_y(y_np[b], y_ref)
        # one token: the policy changes nothing
        _forward_check(pb, p, 2, k1, k2, B=1)
        assert pb.prox_last_device_status(p.h) == 0
    finally:
        pb.prox_ffn_set_mask_policy(p.h, 0)
    # 16-bit proxies do not have the tensor-core Stage 1: the policy is refused, not ignored
    p.quantize(16, 0)
    pb.prox_ffn_set_mask_policy(p.h, 1)
    try:
        assert pb.raw("prox_ffn_forward")(p.h, p.t_x[:2].data_ptr(), 2, k1, k2, p.y_empty(2).data_ptr(), None) == 2
    finally:
        pb.prox_ffn_set_mask_policy(p.h, 0)


def test_pack_save_load_roundtrip(pb, toy, tmp_path):
    wl, p = toy
    p.quantize(4, 128)
    k1, k2 = wl.points[50]
    path = str(tmp_path / "layer0.proxpack")
    pb.prox_pack_save(p.h, path)
    sel_a = torch.empty(1, k2, dtype=torch.int32, device="cuda")
    pb.prox_stage1_mask(p.h, p.t_x[0], 1, k1, k2, sel_a)
    p2 = Problem(pb, p.bits["wg"], p.bits["wu"], p.bits["wd"], p.bits["x"])
    try:
        with pytest.raises(pb.ProxError):
            pb.prox_stage1_mask(p2.h, p2.t_x[0], 1, k1, k2, sel_a)      # not quantized yet
        pb.prox_pack_load(p2.h, path)
        sel_b = torch.empty_like(sel_a)
        pb.prox_stage1_mask(p2.h, p2.t_x[0], 1, k1, k2, sel_b)
        assert torch.equal(sel_a, sel_b)
        with pytest.raises(pb.ProxError):
            pb.prox_pack_load(p2.h, str(tmp_path / "missing"))
    finally:
        p2.close()


def test_device_argument_validation(pb, toy):
    wl, p = toy
    p.quantize(4, 0)
    y = p.y_empty()
    sel = torch.empty(1, 8, dtype=torch.int32, device="cuda")
    R = pb.raw
    assert R("prox_ffn_forward")(p.h, p.t_x.data_ptr(), 0, 1, 1, y.data_ptr(), None) == 1
    assert R("prox_ffn_forward")(p.h, p.t_x.data_ptr(), 9, 1, 1, y.data_ptr(), None) == 1
    assert R("prox_ffn_forward")(p.h, p.t_x.data_ptr(), 1, 0, 1, y.data_ptr(), None) == 1
    assert R("prox_ffn_forward")(p.h, p.t_x.data_ptr(), 1, p.D + 1, 1, y.data_ptr(), None) == 1
    assert R("prox_ffn_forward")(p.h, p.t_x.data_ptr(), 1, 1, p.F + 1, y.data_ptr(), None) == 1
    assert R("prox_ffn_forward")(p.h, p.t_x.data_ptr() + 2, 1, 1, 1, y.data_ptr(), None) == 1
    assert R("prox_ffn_forward")(p.h, p.t_x.data_ptr(), 1, 1, 1, None, None) == 1
    assert R("prox_stage1_mask")(p.h, p.t_x.data_ptr(), 1, 1, 1, None, None, None) == 1
    assert R("prox_stage2_ffn")(p.h, p.t_x.data_ptr(), 1, sel.data_ptr(), 0, y.data_ptr(), None) == 1
    assert R("prox_quantize_proxy")(p.h, 3, 0, None) == 2
    assert R("prox_quantize_proxy")(p.h, 4, 64, None) == 2
