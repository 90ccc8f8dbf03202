"""GPU parity at the benchmark shapes (full d_model / d_ff of every workload,
the launch configuration bench.py times), on a few tokens each so that the
oracle finishes in seconds."""
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


def _run(pb, name, n_tok, cases, batches=(1,)):
    wl, wg, wu, wd, x = inputs.make_workload(name, n_tokens=n_tok)
    p = Problem(pb, wg, wu, wd, x, max_batch=max(batches))
    try:
        for (bits, group), e in cases:
            p.quantize(bits, group)
            k1, k2 = wl.points[e]
            for B in batches:
                for t0 in range(0, n_tok - B + 1, B):
                    y = p.y_empty(B)
                    sel = torch.empty(B, k2, dtype=torch.int32, device="cuda")
                    xb = p.t_x[t0:t0 + B]
                    pb.prox_stage1_mask(p.h, xb, B, k1, k2, sel)
                    pb.prox_ffn_forward(p.h, xb, B, k1, k2, y)
                    used = torch.empty_like(sel)           # the mask the forward call itself built
                    pb.prox_ffn_last_mask(p.h, B, k2, used)
                    torch.cuda.synchronize()
                    sel_np, used_np, y_np = (sel.cpu().numpy().astype(np.int64),
                                             used.cpu().numpy().astype(np.int64), y.cpu().numpy())
                    for b in range(B):
                        idx, score, sel_ref, thr = p.oracle_stage1(t0 + b, k1, k2)
                        check_mask(sel_np[b], score, sel_ref, thr, k2, p.F)
                        check_mask(used_np[b], score, sel_ref, thr, k2, p.F)
                        y_ref, _ = po.stage2(p.x[t0 + b], used_np[b], p.wg, p.wu, p.wd)
                        check_y(y_np[b], y_ref)
                    if B == 1:
                        # Stage 2 alone, fed the oracle's own mask
                        ys = p.y_empty(1)
                        pb.prox_stage2_ffn(p.h, p.t_x[t0], 1, torch.from_numpy(sel_ref.astype(np.int32)).cuda(), k2, ys)
                        y_ref, _ = po.stage2(p.x[t0], sel_ref, p.wg, p.wu, p.wd)
                        check_y(ys.cpu().numpy()[0], y_ref)
            assert pb.prox_last_device_status(p.h) == 0
    finally:
        p.close()


def test_qwen3_0p6b_all_sparsities(pb):
    _run(pb, "qwen3_0p6b", 6, [((4, 0), 50), ((4, 0), 70), ((4, 0), 90)])


def test_qwen3_8b(pb):
    _run(pb, "qwen3_8b", 4, [((4, 128), 70)])


@pytest.mark.parametrize("name,fmt", [("qwen3_8b", (4, 128)), ("llama3_8b", (8, 0)), ("llama3_70b", (4, 0))])
def test_fused_kernel_own_input_list_and_scores_at_bench_shapes(pb, name, fmt):
    from tests.test_gpu_parity import _check_fused_stage1
    wl, wg, wu, wd, x = inputs.make_workload(name, n_tokens=2)
    p = Problem(pb, wg, wu, wd, x)
    try:
        p.quantize(*fmt)
        k1, k2 = wl.points[70]
        for t in range(2):
            _check_fused_stage1(pb, p, p.t_x[t], p.x[t], k1, k2)
        assert pb.prox_last_device_status(p.h) == 0
    finally:
        p.close()


def test_llama3_8b_formats_and_batches(pb):
    _run(pb, "llama3_8b", 8, [((8, 0), 70), ((4, 128), 70), ((4, 128), 40)], batches=(1, 4, 8))


def test_llama3_70b(pb):
    _run(pb, "llama3_70b", 8, [((4, 0), 70), ((4, 128), 70)], batches=(1, 8))


def test_llama3_70b_s1_sweep(pb):
    wl, wg, wu, wd, x = inputs.make_workload("llama3_70b", n_tokens=1)
    p = Problem(pb, wg, wu, wd, x)
    try:
        p.quantize(4, 0)
        for k1, k2 in wl.extra["s1_sweep"]:
            y = p.y_empty()
            sel = torch.empty(1, k2, dtype=torch.int32, device="cuda")
            pb.prox_ffn_forward(p.h, p.t_x[0], 1, k1, k2, y)
            pb.prox_ffn_last_mask(p.h, 1, k2, sel)
            torch.cuda.synchronize()
            sel_np = sel.cpu().numpy()[0].astype(np.int64)
            idx, score, sel_ref, thr = p.oracle_stage1(0, k1, k2)
            check_mask(sel_np, score, sel_ref, thr, k2, p.F)
            y_ref, _ = po.stage2(p.x[0], sel_np, p.wg, p.wu, p.wd)
            check_y(y.cpu().numpy()[0], y_ref)
    finally:
        p.close()


@pytest.mark.parametrize("name", ["qwen3_8b", "llama3_70b"])
def test_threshold_block_and_ablation_forms_at_bench_shapes(pb, name):
    """The other forms of the persistent kernel and the ablation variants at full shapes (a few tokens)."""
    from tests.gpu_common import dev_bf16
    from tests.test_gpu_parity import _check_block, _norm_weight
    wl, wg, wu, wd, x = inputs.make_workload(name, n_tokens=3)
    p = Problem(pb, wg, wu, wd, x, max_batch=2)
    try:
        fmt = wl.proxies[0]
        dg, du, _ = p.quantize(*fmt)
        k1, k2 = wl.points[70]
        # threshold form: thresholds between the k-th and the next value of token 0, applied to all tokens
        mags = np.sort(np.abs(p.x[0]))[::-1]
        tau_x = float(mags[k1 - 1])
        score0 = po.proxy_scores(p.x[0], po.input_threshold(p.x[0], np.float32(tau_x)), dg, du)
        srt = np.sort(score0)[::-1]
        tau_s = float(np.float32((srt[k2 - 1] + srt[k2]) / 2))
        for t in range(3):
            idx_t = po.input_threshold(p.x[t], np.float32(tau_x))
            score_t = po.proxy_scores(p.x[t], idx_t, dg, du)
            sel_t = po.channel_threshold(score_t, tau_s)
            y = p.y_empty()
            pb.prox_runtime_sparsity(p.h, reset=True)
            pb.prox_ffn_forward_threshold(p.h, p.t_x[t], 1, tau_x, tau_s, y)
            torch.cuda.synchronize()
            tok, s1h, s2h, _ = pb.prox_runtime_sparsity(p.h)
            n_in, n = int(round((1 - s1h) * p.D)), int(round((1 - s2h) * p.F))
            assert n_in == len(idx_t) and n > 0
            used = torch.empty(1, n, dtype=torch.int32, device="cuda")
            pb.prox_ffn_last_mask(p.h, 1, n, used)
            got = used.cpu().numpy()[0].astype(np.int64)
            near = np.abs(score_t - tau_s) <= 1e-3 * tau_s
            assert np.all(near[np.setxor1d(got, sel_t)])
            y_ref, _ = po.stage2(p.x[t], got, p.wg, p.wu, p.wd)
            check_y(y.cpu().numpy()[0], y_ref)
        # layer sub-block form, batch 1 (one launch) and batch 2 (norm kernel + batch path)
        nw_bits = _norm_weight(p.D, 9)
        t_nw = dev_bf16(nw_bits)
        for B in (1, 2):
            x_res = (p.x[:B] * 1.5).astype(np.float32)
            t_x = torch.from_numpy(x_res).cuda()
            out = torch.empty_like(t_x)
            used = torch.empty(B, k2, dtype=torch.int32, device="cuda")
            pb.prox_ffn_block_forward(p.h, t_x, t_nw, 1e-6, B, k1, k2, out)
            pb.prox_ffn_last_mask(p.h, B, k2, used)
            torch.cuda.synchronize()
            for b in range(B):
                _check_block(p, dg, du, x_res[b].astype(np.float64), po.bf16_to_f64(nw_bits), 1e-6, k1, k2,
                             out.cpu().numpy()[b], used.cpu().numpy()[b].astype(np.int64))
        # proxy values into the down projection
        y = p.y_empty()
        used = torch.empty(1, k2, dtype=torch.int32, device="cuda")
        pb.prox_ffn_forward_proxy_values(p.h, p.t_x[1], 1, k1, k2, y)
        pb.prox_ffn_last_mask(p.h, 1, k2, used)
        torch.cuda.synchronize()
        u = used.cpu().numpy()[0].astype(np.int64)
        idx, score, sel_ref, thr = p.oracle_stage1(1, k1, k2)
        check_mask(u, score, sel_ref, thr, k2, p.F)
        vals = po.proxy_values(p.x[1], idx, dg, du)
        check_y(y.cpu().numpy()[0], p.wd[:, u].astype(np.float64) @ vals[u])
        assert pb.prox_last_device_status(p.h) == 0
    finally:
        p.close()
