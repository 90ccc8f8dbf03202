"""A few calls of the fused Prox FFN on one small synthetic problem.

Meant as the target of profiler captures (a couple of weight replicas, a handful
of launches, < 2 GB on the device) and as a minimal usage example:

    python -m paper_2607_27591_b200.run_small_case [workload] [calls] [batch] [form]

workload is a name from inputs.WORKLOADS (shape and budgets only; weights are
drawn on the device with the workload's standard deviation).  form is "topk"
(default), "threshold" (thresholds set to the k-th values of the first token) or
"block" (RMSNorm + FFN + residual on an fp32 stream); the last two at batch 1.
"""
from __future__ import annotations

import sys

import torch

from . import binding as pb
from . import inputs


def main(argv=None) -> int:
    argv = sys.argv[1:] if argv is None else argv
    name = argv[0] if len(argv) > 0 else "qwen3_8b"
    ncalls = int(argv[1]) if len(argv) > 1 else 6
    batch = int(argv[2]) if len(argv) > 2 else 1
    form = argv[3] if len(argv) > 3 else "topk"
    wl = inputs.WORKLOADS[name]
    D, F = wl.d_model, wl.d_ff
    k1, k2 = wl.points[70] if 70 in wl.points else next(iter(wl.points.values()))
    bits, group = wl.proxies[0]
    torch.manual_seed(0)
    replicas, handles = [], []
    for _ in range(2):
        w = [(torch.randn(s, device="cuda") * wl.w_std).to(torch.bfloat16) for s in ((F, D), (F, D), (D, F))]
        replicas.append(w)
        h = pb.prox_ffn_create(D, F, max(1, batch), 0, *w)
        pb.prox_quantize_proxy(h, bits, group)
        handles.append(h)
    x = torch.randn(8, batch, D, device="cuda").to(torch.bfloat16)
    y = torch.zeros(8, batch, D, dtype=torch.bfloat16, device="cuda")
    if form == "threshold":
        # thresholds: the k1-th largest |x| of the first token, and the k2-th largest of its proxy scores
        tau_x = float(x[0, 0].float().abs().topk(k1).values[-1])
        sel = torch.empty(1, F, dtype=torch.int32, device="cuda")
        cnt = torch.empty(1, dtype=torch.int32, device="cuda")
        sc = torch.empty(1, F, dtype=torch.float32, device="cuda")
        taus = []
        for h in handles:
            pb.prox_stage1_mask_threshold(h, x[0], 1, tau_x, 0.0, sel, cnt, sc)
            taus.append(float(sc[0].topk(k2).values[-1]))
        for t in range(ncalls):
            pb.prox_ffn_forward_threshold(handles[t % 2], x[t % 8], 1, tau_x, taus[t % 2], y[t % 8])
    elif form == "block":
        nw = torch.ones(D, dtype=torch.bfloat16, device="cuda")
        xr = x[:, 0, :].float().contiguous()
        for t in range(ncalls):
            pb.prox_ffn_block_forward(handles[t % 2], xr[t % 8:t % 8 + 1], nw, 1e-6, 1, k1, k2, xr[t % 8:t % 8 + 1])
        y = xr
    else:
        for t in range(ncalls):
            pb.prox_ffn_forward(handles[t % 2], x[t % 8], batch, k1, k2, y[t % 8])
    torch.cuda.synchronize()
    status = [pb.prox_last_device_status(h) for h in handles]
    print(f"{name}: {ncalls} calls ({form}), batch {batch}, k1={k1} k2={k2}, device status {status}, "
          f"|y| sum {float(y.float().abs().sum()):.4f}")
    for h in handles:
        pb.prox_ffn_destroy(h)
    return 0 if not any(status) else 1


if __name__ == "__main__":
    sys.exit(main())
