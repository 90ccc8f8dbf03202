"""Shared set-up for the GPU parity tests: one synthetic problem held both as
device tensors behind a libprox handle and as float arrays for the oracle."""
from __future__ import annotations

import numpy as np
import torch

from oracle import prox_oracle as po
from paper_2607_27591_b200 import inputs

MASK_BAND = 1e-3      # channels whose oracle score is within 1e-3 (relative) of the k2-th score may differ
Y_TOL = 2e-2          # max |y_gpu - y_oracle| <= 2e-2 * RMS(y_oracle), fp32 accumulation on the GPU


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


class Problem:
    def __init__(self, pb, wg, wu, wd, x, max_batch=1, out_dtype=1):
        self.pb = pb
        self.bits = {"wg": wg, "wu": wu, "wd": wd, "x": x}
        self.F, self.D = wg.shape
        self.t_wg, self.t_wu, self.t_wd, self.t_x = dev_bf16(wg), dev_bf16(wu), dev_bf16(wd), dev_bf16(x)
        # oracle-side copies: float32 holds bf16 exactly; the oracle widens to float64 itself
        self.wg = inputs.bf16_bits_to_f32(wg)
        self.wu = inputs.bf16_bits_to_f32(wu)
        self.wd = inputs.bf16_bits_to_f32(wd)
        self.x = po.bf16_to_f64(x)
        self.out_dtype = out_dtype
        self.max_batch = max_batch
        self.h = pb.prox_ffn_create(self.D, self.F, max_batch, out_dtype, self.t_wg, self.t_wu, self.t_wd)
        self.fmt = None
        self.deq = {}

    def quantize(self, bits, group):
        self.pb.prox_quantize_proxy(self.h, bits, group)
        torch.cuda.synchronize()
        self.fmt = (bits, group)
        if bits == 16 and self.fmt not in self.deq:
            self.deq[self.fmt] = (self.wg, self.wu, None)      # 16-bit proxy: the original weights
        if self.fmt not in self.deq:
            qg, sg = po.quantize_proxy(self.wg, bits, group)
            qu, su = po.quantize_proxy(self.wu, bits, group)
            self.deq[self.fmt] = (po.dequantize(qg, sg, group, np.float32), po.dequantize(qu, su, group, np.float32),
                                  (qg, sg, qu, su))
        return self.deq[self.fmt]

    def oracle_stage1(self, t, k1, k2):
        dg, du, _ = self.deq[self.fmt]
        idx = po.input_topk(self.x[t], k1)
        score = po.proxy_scores(self.x[t], idx, dg, du)
        sel, thr = po.channel_topk(score, k2)
        return idx, score, sel, thr

    def y_empty(self, B=1):
        return torch.empty(B, self.D, dtype=torch.float32 if self.out_dtype else torch.bfloat16, device="cuda")

    def close(self):
        if self.h:
            self.pb.prox_ffn_destroy(self.h)
            self.h = None


def check_mask(sel_gpu: np.ndarray, score: np.ndarray, sel_ref: np.ndarray, thr: float, k2: int, F: int):
    """Acceptance rule for masks: exactly k2 unique ascending ids in range, and
    membership equal to the oracle's except inside the threshold band."""
    assert sel_gpu.shape == (k2,)
    assert np.all(sel_gpu[1:] > sel_gpu[:-1]), "not strictly ascending"
    assert sel_gpu[0] >= 0 and sel_gpu[-1] < F
    diff = np.setxor1d(sel_gpu, sel_ref)
    near = np.abs(score - thr) <= MASK_BAND * thr
    assert np.all(near[diff]), f"{(~near[diff]).sum()} channels differ outside the band"
    return len(diff)


def check_y(y_gpu: np.ndarray, y_ref: np.ndarray, extra_abs: float = 0.0):
    rms = float(np.sqrt(np.mean(y_ref ** 2)))
    err = float(np.max(np.abs(y_gpu.astype(np.float64) - y_ref)))
    assert err <= Y_TOL * rms + extra_abs, (err, rms)
    return err / max(rms, 1e-300)
