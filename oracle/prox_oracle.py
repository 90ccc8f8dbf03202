"""CPU oracle for the Prox decode-time sparse SwiGLU FFN.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the
CUDA library is checked against.  It may be imported by the tests, by the
smoke check and by the benchmark's CPU-baseline leg, and by nothing else; the
product path never calls it, and it shares no code with the CUDA library.

Everything is written out step by step in the paper's order and notation
(Sec. 2.1 "SwiGLU Feed-Forward Networks", Sec. 2.2 "Activation Sparsity",
Sec. 4.1 "Two-Stage Sparse Inference", Sec. 4.2 "Sparsity Allocation between
Two Stages", Sec. 4.3 "Hardware-Aware Implementation", appendix "Threshold-
Based Selection and Token-Adaptive Computation").  All sums are accumulated in
float64; inputs are bf16 values widened exactly.

Storage convention of the arguments (the `nn.Linear` one): W_gate and W_up are
[d_ff, d_model] arrays whose row j is the weight vector of intermediate
channel j (column j of the paper's W in R^{d_model x d_ff}); W_down is
[d_model, d_ff], whose column j is row j of the paper's W_down.

Pins (tests/test_oracle_*.py): dense special case against library matmul and
library SiLU; Stage 2 against the dense FFN with unselected channels zeroed;
exact-score mask against a full sort; the allocation tables printed in the
paper; the paper's closed forms q_Lap, q_G, eta, Corr; the residual bound
||xW - x_sp W|| <= ||r|| ||W||; the order-preservation condition; quantizer
invariants; a hand-worked 4x4 example; the ablation forms against the dense FFN
(all inputs and channels kept, original weights as proxy) and against Stage 2 on
the exact top-k of |s|; RMSNorm against the library's rms_norm and the layer
block against its parts; the calibration helpers: the counter-based generator
against the published splitmix64 outputs, the quantile against the library's
quantile routine and an arithmetic progression, the reservoir against its size /
membership / uniformity properties, Alg. 1 against the realised sparsities of
the calibration stream and its one-layer special case.  The mask and output *values* on random
inputs have no worked example in the paper: parity unpinned for those beyond
the properties above.
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "bf16_to_f64", "f64_to_bf16_bits", "silu", "dense_ffn", "quantize_proxy",
    "dequantize", "input_topk", "input_threshold", "input_sparse_projection", "proxy_scores", "channel_topk",
    "channel_threshold", "stage2", "forward", "forward_batch", "allocate_budget",
    "sparsity_to_k", "effective_sparsity", "proxy_values", "forward_proxy_values",
    "rmsnorm", "ffn_block", "ffn_stack", "forward_batch_shared",
    "splitmix64_at", "reservoir", "empirical_quantile", "histogram_4096", "calibrate_stack",
]


# ---------------------------------------------------------------- dtype glue
def bf16_to_f64(bits) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float64, exact."""
    b = np.asarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def f64_to_bf16_bits(v) -> np.ndarray:
    """float64 -> nearest bf16 (ties to even) bit pattern; via float32 only when
    that does not introduce a double rounding (checked by construction: the
    float32 step is exact for values that are already float32)."""
    v = np.asarray(v, dtype=np.float64)
    f = v.astype(np.float32)
    u = f.view(np.uint32)
    # Repair double rounding: if the f32 rounding moved the value onto a bf16
    # tie, decide the tie by the sign of the f32 rounding error instead.
    low = u & np.uint32(0xFFFF)
    tie = low == np.uint32(0x8000)
    err = v - f.astype(np.float64)            # >0: true value is above f
    up = u + np.uint32(0x8000)                # round half up (in magnitude)
    down = u                                  # truncate (in magnitude)
    rne = u + (((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF))
    mag_up = (err > 0) == (f >= 0)            # true magnitude is above |f|
    res = np.where(tie & (err != 0), np.where(mag_up, up, down), rne)
    return (res >> np.uint32(16)).astype(np.uint16)


def silu(z: np.ndarray) -> np.ndarray:
    """SiLU(z) = z * sigmoid(z) = z / (1 + exp(-z))  (Sec. 2.1; the paper uses
    SiLU without restating it, this is its standard definition)."""
    z = np.asarray(z, dtype=np.float64)
    with np.errstate(over="ignore"):
        return z / (1.0 + np.exp(-z))


# ------------------------------------------------------------ dense SwiGLU
def dense_ffn(x, w_gate, w_up, w_down):
    """FFN(x) = (x W_up  (.)  SiLU(x W_gate)) W_down      (Sec. 2.1, first equation)
    with u = x W_up, h = SiLU(x W_gate), s = u (.) h.  Returns (y, s)."""
    x = np.asarray(x, dtype=np.float64)
    u = np.asarray(w_up, dtype=np.float64) @ x
    h = silu(np.asarray(w_gate, dtype=np.float64) @ x)
    s = u * h
    y = np.asarray(w_down, dtype=np.float64) @ s
    return y, s


# --------------------------------------------------------- proxy quantizer
def quantize_proxy(w, bits: int, group_size: int):
    """Symmetric integer proxy of a projection matrix (Sec. 4.3: "symmetric
    per-row INT4 quantization" of W_up and W_gate).

    One scale per intermediate channel j ("row" of the [d_ff, d_model] storage)
    and per group of `group_size` consecutive input indices (0 = whole row):
        a      = max |w|  over the group
        scale  = fp16( fp32(a) / fp32(qmax) ),     qmax = 2^(bits-1) - 1
        q      = clamp( rint( fp32(w) / fp32(scale) ), -qmax, +qmax )
    rint rounds halves to even.  A group whose scale is zero gets q = 0.  These
    few steps are done in IEEE float32 / float16 (not float64) so that a second
    implementation can reproduce q and scale bit for bit.

    Returns q int8 [d_ff, d_model] and scale float16 [d_ff, d_model/group]."""
    if bits not in (4, 8):
        raise ValueError("bits must be 4 or 8")
    w = np.asarray(w, dtype=np.float32)
    d_ff, d_model = w.shape
    g = d_model if group_size == 0 else group_size
    if d_model % g:
        raise ValueError("group_size must divide d_model")
    qmax = np.float32((1 << (bits - 1)) - 1)
    wg = w.reshape(d_ff, d_model // g, g)
    a = np.abs(wg).max(axis=2)
    scale = (a / qmax).astype(np.float16)
    s32 = scale.astype(np.float32)
    with np.errstate(divide="ignore", invalid="ignore"):
        r = wg / s32[:, :, None]
    q = np.clip(np.rint(r), -qmax, qmax)
    q = np.where(s32[:, :, None] == 0, np.float32(0), q)
    return q.reshape(d_ff, d_model).astype(np.int8), scale


def dequantize(q, scale, group_size: int, dtype=np.float64) -> np.ndarray:
    """deq[j, i] = q[j, i] * scale[j, i // group].  The product of an 8-bit
    integer and an fp16 value has at most 19 significant bits, so it is exact in
    float32 as well as in float64 (`dtype` only chooses the storage)."""
    q = np.asarray(q)
    d_ff, d_model = q.shape
    g = d_model if group_size == 0 else group_size
    s = np.asarray(scale).astype(dtype).reshape(d_ff, d_model // g)
    return (q.astype(dtype).reshape(d_ff, d_model // g, g) * s[:, :, None]).reshape(d_ff, d_model)


# ------------------------------------------------------------ Stage 1 masks
def input_topk(x, k1: int) -> np.ndarray:
    """Input mask m_x (Sec. 4.1, first indicator) under the per-token top-k rule
    of the appendix (m_i = 1[i in TopKIndices(|z|, k)]): the k1 indices of
    largest |x_i|; equal magnitudes are taken in order of increasing index.
    Returns the kept indices in increasing order."""
    mag = np.abs(np.asarray(x, dtype=np.float64))
    order = np.argsort(-mag, kind="stable")
    return np.sort(order[:k1]).astype(np.int64)


def input_threshold(x, tau_x: float) -> np.ndarray:
    """Input mask m_x with a fixed layer threshold: [m_x]_i = 1[|x_i| >= tau_x]
    (Sec. 4.1, first indicator).  Returns kept indices in increasing order."""
    mag = np.abs(np.asarray(x, dtype=np.float64))
    return np.nonzero(mag >= tau_x)[0].astype(np.int64)


def input_sparse_projection(x, idx, w) -> np.ndarray:
    """Pi_in(x, W, m) = x_[I(m)] W_[I(m), :]   (Sec. 2.2): only the retained
    input coordinates contribute.  `w` is stored [d_out, d_in]."""
    x = np.asarray(x, dtype=np.float64)
    idx = np.asarray(idx, dtype=np.int64)
    return np.asarray(w)[:, idx].astype(np.float64) @ x[idx]


def proxy_scores(x, idx_x, deq_gate, deq_up) -> np.ndarray:
    """u~ = Pi_in(x, W~_up, m_x),  h~ = SiLU(Pi_in(x, W~_gate, m_x)),
    s~ = u~ (.) h~    (Sec. 4.1, proxy equations).  Returns |s~| per channel."""
    u_t = input_sparse_projection(x, idx_x, deq_up)
    h_t = silu(input_sparse_projection(x, idx_x, deq_gate))
    return np.abs(u_t * h_t)


def channel_topk(score, k2: int):
    """Channel mask m_s (Sec. 4.1, second indicator) under the per-token top-k
    rule: the k2 channels of largest score, equal scores in order of increasing
    index.  Returns (selected channels in increasing order, score of the k2-th
    ranked channel)."""
    score = np.asarray(score, dtype=np.float64)
    order = np.argsort(-score, kind="stable")
    keep = order[:k2]
    return np.sort(keep).astype(np.int64), float(score[keep[-1]])


def channel_threshold(score, tau_s: float) -> np.ndarray:
    """[m_s]_j = 1[|s~_j| >= tau_s]  (Sec. 4.1, second indicator)."""
    return np.nonzero(np.asarray(score, dtype=np.float64) >= tau_s)[0].astype(np.int64)


# ------------------------------------------------------------------ Stage 2
def stage2(x, sel, w_gate, w_up, w_down):
    """u_sp = Pi_out(x, W_up, m_s), h_sp = SiLU(Pi_out(x, W_gate, m_s)),
    s_sp = u_sp (.) h_sp, y = Pi_in(s_sp, W_down, m_s)   (Sec. 4.1, Stage 2).
    The dense x and the original weights are used.  Returns (y, s_sp)."""
    x = np.asarray(x, dtype=np.float64)
    sel = np.asarray(sel, dtype=np.int64)
    u_sp = np.asarray(w_up)[sel, :].astype(np.float64) @ x
    h_sp = silu(np.asarray(w_gate)[sel, :].astype(np.float64) @ x)
    s_sp = u_sp * h_sp
    y = np.asarray(w_down)[:, sel].astype(np.float64) @ s_sp
    return y, s_sp


# ------------------------------------------------------------- whole path
def forward(x, k1: int, k2: int, deq_gate, deq_up, w_gate, w_up, w_down):
    """One token through Stage 1 then Stage 2.  Returns a dict with idx_x,
    score, sel, threshold (score of the k2-th channel), y."""
    idx_x = input_topk(x, k1)
    score = proxy_scores(x, idx_x, deq_gate, deq_up)
    sel, thr = channel_topk(score, k2)
    y, s_sp = stage2(x, sel, w_gate, w_up, w_down)
    return {"idx_x": idx_x, "score": score, "sel": sel, "threshold": thr, "y": y, "s_sp": s_sp}


# ------------------------------------------------------------ ablation forms
def proxy_values(x, idx_x, deq_gate, deq_up) -> np.ndarray:
    """The signed proxy intermediate state s~ = u~ (.) h~ of Sec. 4.1 (its
    magnitude is what `proxy_scores` ranks)."""
    u_t = input_sparse_projection(x, idx_x, deq_up)
    h_t = silu(input_sparse_projection(x, idx_x, deq_gate))
    return u_t * h_t


def forward_proxy_values(x, k1: int, k2: int, deq_gate, deq_up, w_down):
    """Ablation A3 of Sec. "Ablation Studies" (necessity of exact computation):
    everything as in Prox, but Stage 2's exact gate/up is skipped and the
    selected proxy values themselves enter the down projection,
        y = Pi_in(s~, W_down, m_s).
    With the original weights passed as the proxy this is the execution pattern
    the paper attributes to TEAL (Sec. 2.2): input sparsity on x for gate/up,
    then input sparsity on the resulting s for the down projection.  (The
    ablation with 16-bit proxies, A1, needs no function of its own: pass the
    original weights as `deq_gate`, `deq_up` to `forward`.)"""
    idx_x = input_topk(x, k1)
    s_t = proxy_values(x, idx_x, deq_gate, deq_up)
    score = np.abs(s_t)
    sel, thr = channel_topk(score, k2)
    y = np.asarray(w_down)[:, sel].astype(np.float64) @ s_t[sel]
    return {"idx_x": idx_x, "score": score, "sel": sel, "threshold": thr, "y": y, "s_sp": s_t[sel]}


def forward_batch(xs, k1, k2, deq_gate, deq_up, w_gate, w_up, w_down):
    """Tokens are independent: every token gets its own masks (the paper treats
    single-batch decoding only)."""
    return [forward(x, k1, k2, deq_gate, deq_up, w_gate, w_up, w_down) for x in xs]


# ------------------------------------------------ the FFN sub-block of a layer
def rmsnorm(x, w, eps: float) -> np.ndarray:
    """RMSNorm as the models of the paper's evaluation (Qwen3, Llama-3) define
    it: x_i / sqrt(mean(x^2) + eps) * w_i.  The paper only names it (appendix
    "End-to-End Latency Analysis": attention, RMSNorm and residual around the
    FFN); this is the standard definition."""
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    ms = 0.0
    for v in x:                       # plain running sum, one element after the other
        ms += v * v
    inv = 1.0 / np.sqrt(ms / x.shape[0] + eps)
    return x * inv * w


def ffn_block(x_res, norm_w, eps: float, k1: int, k2: int, deq_gate, deq_up, w_gate, w_up, w_down):
    """One layer's FFN sub-block on the residual stream (pre-norm decoder layer):
        x_res' = x_res + ProxFFN(bf16(RMSNorm(x_res) * w)).
    The FFN input is rounded to bf16, the dtype of the FFN's activations and
    weights; the residual stream itself is kept unrounded here.  Returns
    (x_res', dict of the FFN call, FFN input as float64)."""
    xn = bf16_to_f64(f64_to_bf16_bits(rmsnorm(x_res, norm_w, eps)))
    out = forward(xn, k1, k2, deq_gate, deq_up, w_gate, w_up, w_down)
    return np.asarray(x_res, dtype=np.float64) + out["y"], out, xn


def ffn_stack(x_res, layers, eps: float, k1: int, k2: int):
    """`layers` = list of (norm_w, deq_gate, deq_up, w_gate, w_up, w_down): the
    FFN sub-blocks of consecutive layers applied to one residual stream (the
    attention sub-blocks between them are outside the method).  Returns the list
    of residual streams [before layer 0, after layer 0, ...]."""
    xs = [np.asarray(x_res, dtype=np.float64)]
    for (nw, dg, du, wg, wu, wd) in layers:
        xs.append(ffn_block(xs[-1], nw, eps, k1, k2, dg, du, wg, wu, wd)[0])
    return xs


# ------------------------------------------------- a batch with one shared mask
def forward_batch_shared(xs, k1: int, k2: int, deq_gate, deq_up, w_gate, w_up, w_down):
    """A batch policy beyond the paper (it treats single-batch decoding only and
    names batching as future work): every token keeps its own input mask and
    its own proxy scores, the batch keeps ONE channel mask, the k2 channels of
    largest summed score  sum_b |s~_{b,j}|  (ties to the lower channel), and
    Stage 2 of every token runs on that mask.  With one token this is `forward`.
    Returns (sel, threshold, shared score, list of y per token)."""
    scores = []
    for x in xs:
        idx_x = input_topk(x, k1)
        scores.append(proxy_scores(x, idx_x, deq_gate, deq_up))
    shared = np.zeros_like(scores[0])
    for sc in scores:                 # token after token
        shared = shared + sc
    sel, thr = channel_topk(shared, k2)
    ys = [stage2(x, sel, w_gate, w_up, w_down)[0] for x in xs]
    return sel, thr, shared, ys


# ---------------------------------------------------------- budget helper
def effective_sparsity(s1: float, s2: float, alpha: float = 1.0 / 3.0) -> float:
    """e = 1 - C_Prox / C_Dense = s2 - 2 alpha (1 - s1) / 3   (Sec. 4.2)."""
    return s2 - 2.0 * alpha * (1.0 - s1) / 3.0


def allocate_budget(e: float, alpha: float = 1.0 / 3.0, s_ref: float = 0.7,
                    s1_min: float = 0.0, s1_max: float = 0.7):
    """Allocation rule of Sec. 4.2: start from s2 = s_ref and solve the
    effective-sparsity relation for s1; if s1 leaves [s1_min, s1_max], clamp it
    to the nearest bound and re-solve the relation for s2."""
    s2 = s_ref
    s1 = 1.0 - (s2 - e) * 3.0 / (2.0 * alpha)
    if s1 < s1_min or s1 > s1_max:
        s1 = min(max(s1, s1_min), s1_max)
        s2 = e + 2.0 * alpha * (1.0 - s1) / 3.0
    return s1, s2


def sparsity_to_k(s: float, dim: int) -> int:
    """Number of kept coordinates for sparsity s: (1 - s) * dim rounded to the
    nearest integer (halves up), at least 1, at most dim.  The paper says
    "retains the (1 - rho) d_ff coordinates" without a rounding rule."""
    k = int(np.floor((1.0 - s) * dim + 0.5))
    return max(1, min(dim, k))


# ------------------------------------------------ threshold calibration (Alg. 1)
# Appendix "Threshold Calibration and Runtime Sparsity": per layer and per signal a
# reservoir of at most 200,000 activation samples, the threshold "directly from the
# corresponding empirical quantile", a 4,096-bin histogram saved beside it, layers
# calibrated in depth order on the stream that the finalized sparse layers produce.
_M64 = (1 << 64) - 1


def splitmix64_at(seed: int, i: int) -> int:
    """Output number i (0-based) of the splitmix64 sequence started at `seed`: a
    counter-based generator (the state before output i is seed + (i+1)*gamma), so
    that the reservoir's draws are a function of (seed, sample number) alone."""
    z = (seed + (i + 1) * 0x9E3779B97F4A7C15) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def reservoir(values, cap: int, seed: int, state=None):
    """Uniform reservoir sampling (Vitter's algorithm R) of the magnitudes |v|, in
    float32: the first `cap` samples fill the reservoir; sample number i >= cap
    draws j = splitmix64_at(seed, i) mod (i + 1) and replaces slot j if j < cap.
    `state` = (list, samples seen so far) continues an earlier call.
    The paper fixes the capacity (200,000) but not the sampling scheme: this is
    the textbook one.  Returns (list of float32 magnitudes, samples seen)."""
    res, seen = ([], 0) if state is None else (list(state[0]), int(state[1]))
    for v in np.asarray(values, dtype=np.float32).ravel():
        m = np.float32(abs(v))
        if seen < cap:
            res.append(m)
        else:
            j = splitmix64_at(seed, seen) % (seen + 1)
            if j < cap:
                res[j] = m
        seen += 1
    return res, seen


def empirical_quantile(mags, s: float) -> np.float32:
    """Empirical quantile of the samples at level s with linear interpolation
    between order statistics (position s*(n-1); the definition numpy and torch use
    by default; the paper says only "empirical quantile").  Keeping |z| >= tau then
    drops a fraction of about s of the samples.  Computed in float64, returned as
    the float32 the kernels compare with."""
    a = sorted(float(v) for v in mags)
    n = len(a)
    if n == 0:
        raise ValueError("no samples")
    pos = float(s) * (n - 1)
    lo = int(np.floor(pos))
    hi = min(lo + 1, n - 1)
    return np.float32(a[lo] + (pos - lo) * (a[hi] - a[lo]))


def histogram_4096(mags):
    """The saved analysis artifact: 4,096 equal bins over [0, max |v|] of the
    reservoir; a sample equal to the maximum falls into the last bin.  The paper
    fixes the bin count only; range and binning are this reading.
    Returns (int64 counts [4096], upper edge as float32)."""
    a = np.asarray(list(mags), dtype=np.float32)
    hi = np.float32(a.max()) if a.size else np.float32(0.0)
    counts = np.zeros(4096, dtype=np.int64)
    for v in a:
        b = 4095 if hi == 0 else min(4095, int(np.floor(float(v) / float(hi) * 4096.0)))
        counts[b] += 1
    return counts, hi


def calibrate_stack(x_res_tokens, layers, eps: float, s1: float, s2: float, cap: int = 200000, seed: int = 0):
    """Alg. 1 (sequential threshold calibration) on a stack of FFN sub-blocks:
    for layer l = 1..L: the calibration tokens arrive through layers 1..l-1 under
    their finalized threshold rules; collect the layer's FFN inputs x_l; choose
    tau_x as the s1-quantile of |x_l| and build m_x; compute the proxy state
    s~_l = u~ * SiLU(g~) with m_x and the quantized proxies; choose tau_s as the
    s2-quantile of |s~_l|; the layer's rule is final.  Because the stream that
    reaches layer l+1 is the one the finalized rules of layers 1..l produce, it
    is advanced layer by layer instead of being recomputed from the start.
    `layers` = list of (norm_w, deq_gate, deq_up, w_gate, w_up, w_down) as in
    `ffn_stack`; the FFN input is bf16(RMSNorm(x_res) * w).
    Returns a list of dicts per layer: tau_x, tau_s, s1_hat, s2_hat (realised on
    the calibration tokens), hist_x, hist_s."""
    xs = [np.asarray(x, dtype=np.float64) for x in x_res_tokens]
    out = []
    for li, (nw, dg, du, wg, wu, wd) in enumerate(layers):
        xn = [bf16_to_f64(f64_to_bf16_bits(rmsnorm(x, nw, eps))) for x in xs]
        rx, _ = reservoir(np.concatenate(xn), cap, seed + 2 * li)
        tau_x = empirical_quantile(rx, s1)
        idx = [input_threshold(x, tau_x) for x in xn]
        sc = [proxy_scores(x, i, dg, du) for x, i in zip(xn, idx)]
        rs, _ = reservoir(np.concatenate(sc), cap, seed + 2 * li + 1)
        tau_s = empirical_quantile(rs, s2)
        kept_in = sum(len(i) for i in idx)
        kept_ch = 0
        nxt = []
        for x_res, x, s_l in zip(xs, xn, sc):
            sel = channel_threshold(s_l, tau_s)
            kept_ch += len(sel)
            nxt.append(x_res + stage2(x, sel, wg, wu, wd)[0])
        out.append({"tau_x": tau_x, "tau_s": tau_s,
                    "s1_hat": 1.0 - kept_in / (len(xs) * len(xs[0])),
                    "s2_hat": 1.0 - kept_ch / (len(xs) * len(sc[0])),
                    "hist_x": histogram_4096(rx), "hist_s": histogram_4096(rs)})
        xs = nxt
    return out
