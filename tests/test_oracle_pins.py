"""Pins for the CPU oracle: what the paper and the mathematics fix.

Every test here checks oracle/prox_oracle.py against something that is not the
oracle itself: library routines (torch float64 matmul / SiLU, numpy sorts),
values printed in the paper (tests/golden/*.txt), closed forms, invariants, a
hand-worked example, or brute force on tiny inputs.  CPU only.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import prox_oracle as po
from paper_2607_27591_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _problem(d_model=256, d_ff=384, n_tok=3, seed=3):
    wg, wu, wd, x = inputs.make_small(d_model, d_ff, n_tok, seed)
    return po.bf16_to_f64(wg), po.bf16_to_f64(wu), po.bf16_to_f64(wd), po.bf16_to_f64(x)


# ------------------------------------------------------------------ dense pin
def test_dense_ffn_matches_library_swiglu():
    """Sec. 2.1 definition, evaluated by torch float64 library ops."""
    wg, wu, wd, x = _problem()
    for t in range(x.shape[0]):
        y, s = po.dense_ffn(x[t], wg, wu, wd)
        xt = torch.from_numpy(x[t])
        s_ref = (torch.from_numpy(wu) @ xt) * torch.nn.functional.silu(torch.from_numpy(wg) @ xt)
        y_ref = torch.from_numpy(wd) @ s_ref
        np.testing.assert_allclose(s, s_ref.numpy(), rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(y, y_ref.numpy(), rtol=1e-11, atol=1e-14)


def test_k2_equal_dff_is_dense():
    """At 0% channel sparsity the whole path equals the dense FFN, whatever the
    proxy says (proxy values never propagate, Sec. 3.2 / 4.1)."""
    wg, wu, wd, x = _problem()
    qg, sg = po.quantize_proxy(wg, 4, 0)
    qu, su = po.quantize_proxy(wu, 4, 0)
    dg, du = po.dequantize(qg, sg, 0), po.dequantize(qu, su, 0)
    d_ff = wg.shape[0]
    for t in range(x.shape[0]):
        out = po.forward(x[t], 40, d_ff, dg, du, wg, wu, wd)
        xt = torch.from_numpy(x[t])
        y_ref = torch.from_numpy(wd) @ ((torch.from_numpy(wu) @ xt) *
                                        torch.nn.functional.silu(torch.from_numpy(wg) @ xt))
        assert np.array_equal(out["sel"], np.arange(d_ff))
        np.testing.assert_allclose(out["y"], y_ref.numpy(), rtol=1e-11, atol=1e-14)


def test_stage2_is_dense_with_unselected_channels_zeroed():
    """y = Pi_in(s_sp, W_down, m_s) = sum_{j in mask} s_j W_down[j,:]  (Sec. 3.1
    weighted-sum view, Sec. 4.1 Stage 2)."""
    wg, wu, wd, x = _problem(seed=5)
    rng = np.random.default_rng(0)
    d_ff = wg.shape[0]
    for t in range(x.shape[0]):
        sel = np.sort(rng.choice(d_ff, size=97, replace=False))
        y, s_sp = po.stage2(x[t], sel, wg, wu, wd)
        xt = torch.from_numpy(x[t])
        s_full = (torch.from_numpy(wu) @ xt) * torch.nn.functional.silu(torch.from_numpy(wg) @ xt)
        m = torch.zeros(d_ff, dtype=torch.float64)
        m[torch.from_numpy(sel)] = 1.0
        y_ref = torch.from_numpy(wd) @ (s_full * m)
        np.testing.assert_allclose(y, y_ref.numpy(), rtol=1e-10, atol=1e-13)
        np.testing.assert_allclose(s_sp, s_full.numpy()[sel], rtol=1e-12, atol=1e-15)
        # weighted-sum form, one row of W_down per channel, summed one by one
        y_rows = np.zeros_like(y)
        for c, j in enumerate(sel):
            y_rows += s_sp[c] * wd[:, j]
        np.testing.assert_allclose(y, y_rows, rtol=1e-10, atol=1e-13)


def test_output_depends_on_proxy_only_through_mask():
    """Two different proxies that give the same mask give bit-identical y."""
    wg, wu, wd, x = _problem(seed=7)
    dg4 = po.dequantize(*po.quantize_proxy(wg, 4, 0), 0)
    du4 = po.dequantize(*po.quantize_proxy(wu, 4, 0), 0)
    out = po.forward(x[0], 77, 120, dg4, du4, wg, wu, wd)
    y_again, _ = po.stage2(x[0], out["sel"], wg, wu, wd)
    assert np.array_equal(out["y"], y_again)


# ------------------------------------------------------------ selection pins
def test_exact_scores_mask_is_full_sort_topk():
    """oracle-s selection (Sec. 3.1): with exact scores (unquantized weights,
    all inputs kept) the mask is the (1-rho) d_ff largest |s|."""
    wg, wu, wd, x = _problem(seed=11)
    d_model, d_ff = wg.shape[1], wg.shape[0]
    for t in range(x.shape[0]):
        for k2 in (1, 13, 128, d_ff - 1, d_ff):
            out = po.forward(x[t], d_model, k2, wg, wu, wg, wu, wd)
            _, s = po.dense_ffn(x[t], wg, wu, wd)
            # brute force: python sort of (magnitude desc, index asc) pairs
            ranked = sorted(range(d_ff), key=lambda j: (-abs(s[j]), j))[:k2]
            assert sorted(ranked) == out["sel"].tolist()
            assert len(out["sel"]) == k2 == len(set(out["sel"].tolist()))
            assert out["threshold"] == abs(s[ranked[-1]])


def test_topk_tie_rule_on_handmade_ties():
    """Equal magnitudes: lower index wins; exactly k are kept."""
    z = np.array([1.0, -2.0, 2.0, 0.5, -2.0, 1.0, 0.0, -0.0, 2.0, 1.0])
    assert po.input_topk(z, 1).tolist() == [1]
    assert po.input_topk(z, 2).tolist() == [1, 2]
    assert po.input_topk(z, 3).tolist() == [1, 2, 4]
    assert po.input_topk(z, 5).tolist() == [0, 1, 2, 4, 8]
    assert po.input_topk(z, 6).tolist() == [0, 1, 2, 4, 5, 8]
    assert po.input_topk(z, 9).tolist() == [0, 1, 2, 3, 4, 5, 6, 8, 9]
    sel, thr = po.channel_topk(np.abs(z), 5)
    assert sel.tolist() == [0, 1, 2, 4, 8] and thr == 1.0
    # brute force over every k on random tied data
    rng = np.random.default_rng(1)
    v = rng.integers(0, 4, size=16).astype(np.float64)
    for k in range(1, 17):
        want = sorted(sorted(range(16), key=lambda i: (-v[i], i))[:k])
        assert po.channel_topk(v, k)[0].tolist() == want
        assert po.input_topk(-v, k).tolist() == want


def test_threshold_rule_keeps_all_at_or_above_tau():
    z = np.array([0.5, -1.0, 1.0, 0.99, -3.0])
    assert po.input_threshold(z, 1.0).tolist() == [1, 2, 4]
    assert po.channel_threshold(np.abs(z), 0.99).tolist() == [1, 2, 3, 4]


def test_topk_minimises_residual_energy_bruteforce():
    """Sec. 3.2: keeping the largest magnitudes minimises ||r||_2 over all
    coordinate-sparse approximations of the same density (all subsets, tiny d)."""
    import itertools
    rng = np.random.default_rng(2)
    x = rng.laplace(size=9)
    for k in (1, 3, 5, 8):
        kept = po.input_topk(x, k)
        best = min(itertools.combinations(range(9), k),
                   key=lambda c: np.sum(np.delete(x, list(c)) ** 2))
        assert sorted(best) == kept.tolist()


# ----------------------------------------------------------- hand-worked pin
def _read_hand():
    rows = {}
    for line in open(os.path.join(GOLDEN, "hand_worked_4x4.txt")):
        line = line.split("#")[0].strip()
        if line:
            k, *v = line.split()
            rows[k] = [float(t) for t in v]
    return rows


def test_hand_worked_example():
    g = _read_hand()
    x = np.array(g["x"])
    wg = np.array([g[f"w_gate{j}"] for j in range(4)])
    wu = np.array([g[f"w_up{j}"] for j in range(4)])
    wd = np.array([g[f"w_down{d}"] for d in range(4)])
    qg, sg = po.quantize_proxy(wg, 4, 0)
    qu, su = po.quantize_proxy(wu, 4, 0)
    assert np.array_equal(qg, np.array([g[f"q_gate{j}"] for j in range(4)], dtype=np.int8))
    assert np.all(sg.astype(np.float64) == 0.125) and np.all(su.astype(np.float64) == 0.125)
    dg, du = po.dequantize(qg, sg, 0), po.dequantize(qu, su, 0)
    assert np.array_equal(dg, wg) and np.array_equal(du, wu)
    idx = po.input_topk(x, 2)
    assert idx.tolist() == [int(v) for v in g["idx_x"]]
    gp = po.input_sparse_projection(x, idx, dg)
    up = po.input_sparse_projection(x, idx, du)
    assert gp.tolist() == g["g_proxy"] and up.tolist() == g["u_proxy"]
    score = po.proxy_scores(x, idx, dg, du)
    want = [abs(u * z / (1.0 + math.exp(-z))) for u, z in zip(g["u_proxy"], g["g_proxy"])]
    np.testing.assert_allclose(score, want, rtol=1e-15)
    np.testing.assert_allclose(score, [4.4506, 0.3557, 0.4216, 1.1182], atol=5e-5)
    sel, thr = po.channel_topk(score, 2)
    assert sel.tolist() == [int(v) for v in g["sel"]]
    y, s_sp = po.stage2(x, sel, wg, wu, wd)
    s_want = [u * z / (1.0 + math.exp(-z)) for u, z in zip(g["u_exact"], g["g_exact"])]
    np.testing.assert_allclose(s_sp, s_want, rtol=1e-15)
    y_want = [sum(s_want[c] * g[f"w_down{d}"][j] for c, j in enumerate(sel)) for d in range(4)]
    np.testing.assert_allclose(y, y_want, rtol=1e-14)
    np.testing.assert_allclose(y, [-1.227494, -3.502545, -0.523779, 3.764435], atol=2e-6)
    full = po.forward(x, 2, 2, dg, du, wg, wu, wd)
    assert np.array_equal(full["y"], y) and full["sel"].tolist() == sel.tolist()


# ------------------------------------------------------------ quantizer pins
@pytest.mark.parametrize("bits,group", [(4, 0), (4, 128), (8, 0), (8, 128)])
def test_quantizer_invariants(bits, group):
    wg, _, _, _ = _problem(d_model=256, d_ff=96, seed=13)
    wg[5, :] = 0.0                       # an all-zero row
    wg[6, 128:] = 0.0                    # an all-zero group
    q, scale = po.quantize_proxy(wg, bits, group)
    qmax = 2 ** (bits - 1) - 1
    g = wg.shape[1] if group == 0 else group
    assert q.dtype == np.int8 and scale.dtype == np.float16
    assert scale.shape == (wg.shape[0], wg.shape[1] // g)
    assert np.abs(q).max() <= qmax
    deq = po.dequantize(q, scale, group)
    s_full = np.repeat(scale.astype(np.float64), g, axis=1)
    assert np.all(np.abs(wg - deq) <= 0.5 * s_full * (1 + 1e-6) + 1e-30)
    qg = np.abs(q).reshape(wg.shape[0], -1, g).max(axis=2)
    nz = scale.astype(np.float64) > 0
    assert np.all(qg[nz] == qmax) and np.all(qg[~nz] == 0)
    assert np.all(q[5] == 0) and np.all(scale[5] == 0)
    if group:
        assert np.all(q[6, 128:] == 0) and scale[6, 1] == 0
    # re-quantizing the dequantized matrix is the identity on q
    q2, scale2 = po.quantize_proxy(deq, bits, group)
    assert np.array_equal(q2, q) and np.array_equal(scale2, scale)
    # sign symmetry
    qn, sn = po.quantize_proxy(-wg, bits, group)
    assert np.array_equal(qn, -q) and np.array_equal(sn, scale)


def test_quantizer_exact_rational_check():
    """Brute-force check of rint(w / scale) with exact rationals on a small
    matrix: the float32 division must round to the integer nearest to the exact
    quotient (ties to even), which a float32 quotient guarantees for |q| <= 127."""
    rng = np.random.default_rng(17)
    w = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(
        (rng.standard_normal((8, 64)) * 0.02).astype(np.float32))).astype(np.float64)
    for bits in (4, 8):
        q, scale = po.quantize_proxy(w, bits, 0)
        qmax = 2 ** (bits - 1) - 1
        for j in range(8):
            sc = Fraction(float(scale[j, 0]))
            # scale itself: fp16 nearest to fp32(a)/fp32(qmax)
            a32 = np.float32(np.abs(w[j]).max())
            assert scale[j, 0] == np.float16(np.float32(a32 / np.float32(qmax)))
            for i in range(64):
                exact = Fraction(float(w[j, i])) / sc
                near = round(exact)          # python rounds halves to even
                # float32 quotient can only differ from `exact` by < 2^-24 rel;
                # exclude the measure-zero case of straddling a half
                if abs(exact - near) < Fraction(1, 2) - Fraction(1, 10 ** 5):
                    assert q[j, i] == max(-qmax, min(qmax, near))


def test_int8_proxy_ranks_closer_to_exact_than_int4():
    wg, wu, wd, x = _problem(d_model=512, d_ff=1024, n_tok=4, seed=19)
    d_model, d_ff = 512, 1024
    ov = {}
    for bits in (4, 8):
        dg = po.dequantize(*po.quantize_proxy(wg, bits, 0), 0)
        du = po.dequantize(*po.quantize_proxy(wu, bits, 0), 0)
        tot = 0
        for t in range(x.shape[0]):
            a = po.forward(x[t], d_model, 256, dg, du, wg, wu, wd)["sel"]
            b = po.forward(x[t], d_model, 256, wg, wu, wg, wu, wd)["sel"]
            tot += len(set(a.tolist()) & set(b.tolist()))
        ov[bits] = tot
    assert ov[8] > ov[4] > 0.8 * 4 * 256


def test_proxy_storage_is_one_sixth_of_ffn_bytes():
    """Sec. 6 (limitations): INT4 proxies add about 12% weight storage.  Two
    INT4 matrices against three bf16 ones: 2*(1/2) / (3*2) = 1/6 of the FFN;
    with FFNs at roughly 70-75% of model parameters that is 12%."""
    d_model, d_ff = 4096, 12288
    proxy = 2 * d_model * d_ff * 4 // 8
    ffn = 3 * d_model * d_ff * 2
    assert Fraction(proxy, ffn) == Fraction(1, 6)
    assert 0.11 < (1 / 6) * 0.72 < 0.13


# ------------------------------------------------------------- budget pins
def _alloc_rows():
    for line in open(os.path.join(GOLDEN, "stagewise_allocation.txt")):
        line = line.split("#")[0].strip()
        if line:
            src, e, cap, s1, s2 = line.split()
            yield src, float(e) / 100, float(cap) / 100, (None if s1 == "-" else float(s1) / 100), float(s2)


def test_allocation_tables_printed_in_paper():
    n = 0
    for src, e, cap, s1_want, s2_want in _alloc_rows():
        s1, s2 = po.allocate_budget(e, alpha=1 / 3, s_ref=0.7, s1_min=0.0, s1_max=cap)
        assert f"{100 * s2:.1f}" == f"{s2_want:.1f}", (src, e, cap)
        if s1_want is not None:
            assert abs(s1 - s1_want) < 1e-9
        assert abs(po.effective_sparsity(s1, s2) - e) < 1e-12      # Sec. 4.2 relation
        n += 1
    assert n == 10


def test_cost_model_relation():
    """e = 1 - C_Prox / C_Dense with C_Prox = 2 alpha (1 - s1) + 3 (1 - s2), C_Dense = 3."""
    for s1, s2, a in ((0.7, 0.7667, 1 / 3), (0.0, 0.622, 1 / 3), (0.3, 0.8, 0.285)):
        c = 2 * a * (1 - s1) + 3 * (1 - s2)
        assert abs(po.effective_sparsity(s1, s2, a) - (1 - c / 3)) < 1e-15


def test_workload_budgets_follow_allocation_rule():
    for wl in inputs.WORKLOADS.values():
        for e, (k1, k2) in wl.points.items():
            s1, s2 = po.allocate_budget(e / 100)
            assert po.sparsity_to_k(s1, wl.d_model) == k1, (wl.name, e)
            assert po.sparsity_to_k(s2, wl.d_ff) == k2, (wl.name, e)
            # realised sparsity equals the target up to rounding of k
            e_hat = po.effective_sparsity(1 - k1 / wl.d_model, 1 - k2 / wl.d_ff)
            assert abs(e_hat - e / 100) < 1.0 / wl.d_model + 1.0 / wl.d_ff
    sweep = inputs.WORKLOADS["llama3_70b"].extra["s1_sweep"]
    for n, (k1, k2) in enumerate(sweep):
        s1 = n / 10
        s2 = 0.7 + 2 * (1 / 3) * (1 - s1) / 3
        assert (po.sparsity_to_k(s1, 8192), po.sparsity_to_k(s2, 28672)) == (k1, k2)


def test_sparsity_to_k_edges():
    assert po.sparsity_to_k(0.0, 100) == 100
    assert po.sparsity_to_k(1.0, 100) == 1
    assert po.sparsity_to_k(0.995, 100) == 1       # 0.5 rounds up
    assert po.sparsity_to_k(0.985, 100) == 2
    assert po.sparsity_to_k(-0.5, 100) == 100


# -------------------------------------------------------- closed-form pins
def _closed():
    out = {}
    for line in open(os.path.join(GOLDEN, "closed_forms.txt")):
        line = line.split("#")[0].strip()
        if line:
            name, p, v, _ = line.split()
            out[name] = (float(p), float(v))
    return out


def test_laplace_energy_kept_by_magnitude_topk():
    """q_Lap(0.7) ~ 0.879: top-30% magnitudes of Laplace samples keep ~87.9% of
    the energy.  Pins the magnitude top-k rule statistically."""
    p, want = _closed()["q_lap"]
    a = -math.log(1 - p)
    assert abs((1 - p) / 2 * (a * a + 2 * a + 2) - want) < 5e-4
    rng = np.random.default_rng(23)
    z = rng.laplace(0, 1.7, size=200_000)
    kept = po.input_topk(z, po.sparsity_to_k(p, z.size))
    frac = np.sum(z[kept] ** 2) / np.sum(z ** 2)
    assert abs(frac - want) < 6e-3
    # the complement rule (keep the smallest) would keep ~12% - far outside
    assert frac > 0.85


def test_gaussian_input_sparse_projection_error_and_correlation():
    """q_G(0.7) ~ 0.783, eta ~ 0.465, Corr ~ 0.885 for Gaussian x and iid
    Gaussian weights.  Pins Pi_in together with the kept-largest rule."""
    c = _closed()
    p = c["q_g"][0]
    rng = np.random.default_rng(29)
    d_in, d_out = 4096, 1536
    w = rng.standard_normal((d_out, d_in))
    q_acc, eta_acc, corr_acc, n = 0.0, 0.0, 0.0, 6
    for _ in range(n):
        x = rng.standard_normal(d_in) * 0.8
        idx = po.input_topk(x, po.sparsity_to_k(p, d_in))
        dense = w @ x
        sp = po.input_sparse_projection(x, idx, w)
        q_acc += np.sum(x[idx] ** 2) / np.sum(x ** 2)
        eta_acc += np.linalg.norm(dense - sp) / np.linalg.norm(dense)
        corr_acc += np.corrcoef(dense, sp)[0, 1]
    assert abs(q_acc / n - c["q_g"][1]) < 0.01
    assert abs(eta_acc / n - c["eta"][1]) < 0.015
    assert abs(corr_acc / n - c["corr"][1]) < 0.012


def test_residual_bound():
    """||x W - x_sp W||_2 <= ||r||_2 ||W||_2   (Sec. 3.2)."""
    wg, wu, wd, x = _problem(d_model=256, d_ff=384, seed=31)
    spec = np.linalg.norm(wg, 2)
    for t in range(x.shape[0]):
        for k in (1, 26, 77, 255):
            idx = po.input_topk(x[t], k)
            r = x[t].copy()
            r[idx] = 0.0
            lhs = np.linalg.norm(wg @ x[t] - po.input_sparse_projection(x[t], idx, wg))
            assert lhs <= np.linalg.norm(r) * spec * (1 + 1e-12)
            np.testing.assert_allclose(lhs, np.linalg.norm(wg @ r), rtol=1e-9)


def test_order_preserved_when_gap_exceeds_perturbation():
    """If s~_i = s_i + delta_i, the order of |s_i|, |s_j| is kept whenever
    ||s_i| - |s_j|| > |delta_i| + |delta_j|  (appendix, ranking preservation)."""
    wg, wu, wd, x = _problem(d_model=256, d_ff=384, seed=37)
    dg = po.dequantize(*po.quantize_proxy(wg, 4, 0), 0)
    du = po.dequantize(*po.quantize_proxy(wu, 4, 0), 0)
    for t in range(x.shape[0]):
        idx = po.input_topk(x[t], 77)
        s_t = po.input_sparse_projection(x[t], idx, du) * po.silu(po.input_sparse_projection(x[t], idx, dg))
        _, s = po.dense_ffn(x[t], wg, wu, wd)
        delta = np.abs(s_t - s)
        gap = np.abs(np.abs(s)[:, None] - np.abs(s)[None, :])
        safe = gap > delta[:, None] + delta[None, :]
        same = (np.abs(s)[:, None] > np.abs(s)[None, :]) == (np.abs(s_t)[:, None] > np.abs(s_t)[None, :])
        assert safe.sum() > 0 and np.all(same[safe])
        np.testing.assert_array_equal(np.abs(s_t), po.proxy_scores(x[t], idx, dg, du))


# ---------------------------------------------------------------- dtype glue
def test_bf16_round_trip_and_rne():
    bits = np.arange(0, 0x7F80, 7, dtype=np.uint16)          # finite positives
    bits = np.concatenate([bits, bits | np.uint16(0x8000)])
    v = po.bf16_to_f64(bits)
    assert np.array_equal(po.f64_to_bf16_bits(v), bits)
    assert np.array_equal(v.astype(np.float32), inputs.bf16_bits_to_f32(bits))
    # halfway cases go to even; just above half goes up (also through the
    # float32 double-rounding trap)
    one = 1.0
    ulp = 2.0 ** -7
    assert po.f64_to_bf16_bits(one + ulp / 2)[()] == 0x3F80
    assert po.f64_to_bf16_bits(one + 3 * ulp / 2)[()] == 0x3F82
    assert po.f64_to_bf16_bits(one + ulp / 2 + 2.0 ** -40)[()] == 0x3F81
    assert po.f64_to_bf16_bits(-(one + ulp / 2 + 2.0 ** -40))[()] == 0xBF81
    assert po.f64_to_bf16_bits(one + ulp / 2 - 2.0 ** -40)[()] == 0x3F80
    rng = np.random.default_rng(41)
    vals = rng.standard_normal(2000)
    got = po.f64_to_bf16_bits(vals)
    for v_, b_ in zip(vals[:300], got[:300]):
        lo = po.bf16_to_f64(np.uint16(b_ - 1))
        mid = po.bf16_to_f64(np.uint16(b_))
        hi = po.bf16_to_f64(np.uint16(b_ + 1))
        assert abs(v_ - mid) <= min(abs(v_ - lo), abs(v_ - hi))
    assert np.array_equal(inputs.f32_to_bf16_bits(vals.astype(np.float32)),
                          po.f64_to_bf16_bits(vals.astype(np.float32).astype(np.float64)))


def test_batch_tokens_are_independent():
    wg, wu, wd, x = _problem(n_tok=4, seed=43)
    dg = po.dequantize(*po.quantize_proxy(wg, 4, 128), 128)
    du = po.dequantize(*po.quantize_proxy(wu, 4, 128), 128)
    outs = po.forward_batch(x, 77, 100, dg, du, wg, wu, wd)
    for t, o in enumerate(outs):
        single = po.forward(x[t], 77, 100, dg, du, wg, wu, wd)
        assert np.array_equal(o["y"], single["y"]) and np.array_equal(o["sel"], single["sel"])


# ------------------------------------------------------------ ablation forms
def test_proxy_values_into_down_with_exact_proxy_and_nothing_dropped_is_dense():
    """A3 form with the original weights as proxy, k1 = d_model, k2 = d_ff: the
    proxy state is the exact s, so y is the dense FFN (Sec. 2.1) by library ops."""
    wg, wu, wd, x = _problem(seed=11)
    d_model, d_ff = wg.shape[1], wg.shape[0]
    for t in range(x.shape[0]):
        out = po.forward_proxy_values(x[t], d_model, d_ff, wg, wu, wd)
        xt = torch.from_numpy(x[t])
        y_ref = torch.from_numpy(wd) @ ((torch.from_numpy(wu) @ xt) *
                                        torch.nn.functional.silu(torch.from_numpy(wg) @ xt))
        np.testing.assert_allclose(out["y"], y_ref.numpy(), rtol=1e-10, atol=1e-13)


def test_input_then_state_sparsity_pattern_by_library_ops():
    """The pattern the paper attributes to TEAL (Sec. 2.2): zero all but the k1
    largest |x|, run gate/up densely on that x (library matmul), zero all but the
    k2 largest |s|, run the down projection densely.  Written here with masks and
    torch ops, not with the oracle's gathers."""
    wg, wu, wd, x = _problem(seed=12)
    d_model, d_ff = wg.shape[1], wg.shape[0]
    k1, k2 = 90, 130
    for t in range(x.shape[0]):
        out = po.forward_proxy_values(x[t], k1, k2, wg, wu, wd)
        order = np.argsort(-np.abs(x[t]), kind="stable")[:k1]
        mx = np.zeros(d_model)
        mx[order] = 1.0
        xs = torch.from_numpy(x[t] * mx)
        s = (torch.from_numpy(wu) @ xs) * torch.nn.functional.silu(torch.from_numpy(wg) @ xs)
        keep = np.argsort(-np.abs(s.numpy()), kind="stable")[:k2]
        ms = np.zeros(d_ff)
        ms[keep] = 1.0
        y_ref = torch.from_numpy(wd) @ (s * torch.from_numpy(ms))
        assert np.array_equal(out["sel"], np.sort(keep))
        np.testing.assert_allclose(out["y"], y_ref.numpy(), rtol=1e-9, atol=1e-13)


def test_proxy_values_have_the_sign_that_scores_drop():
    wg, wu, wd, x = _problem(seed=13)
    dg = po.dequantize(*po.quantize_proxy(wg, 4, 0), 0)
    du = po.dequantize(*po.quantize_proxy(wu, 4, 0), 0)
    idx = po.input_topk(x[0], 64)
    v = po.proxy_values(x[0], idx, dg, du)
    assert np.array_equal(np.abs(v), po.proxy_scores(x[0], idx, dg, du))
    assert (v < 0).any() and (v > 0).any()
    # on a hand-made case: u~ = -2, g~ = 1  ->  s~ = -2 * SiLU(1)
    w_g = np.array([[1.0, 0.0]])
    w_u = np.array([[-2.0, 5.0]])
    s = po.proxy_values(np.array([1.0, 0.25]), np.array([0]), w_g, w_u)
    assert s[0] == pytest.approx(-2.0 / (1.0 + math.exp(-1.0)), rel=1e-15)


def test_sixteen_bit_proxy_budget_uses_unit_cost_ratio():
    """A1 reallocates the two stages for a 16-bit proxy: alpha = 1 in the cost
    model of Sec. 4.2, e = s2 - 2 alpha (1 - s1) / 3."""
    for e in (0.4, 0.5, 0.6, 0.7):
        s1, s2 = po.allocate_budget(e, alpha=1.0)
        assert 0.0 <= s1 <= 1.0 and 0.0 <= s2 <= 1.0
        assert po.effective_sparsity(s1, s2, alpha=1.0) == pytest.approx(e, abs=1e-12)


# ------------------------------------------------------- layer sub-block pins
def test_rmsnorm_matches_library_rms_norm():
    rng = np.random.default_rng(21)
    for d in (8, 256, 1000):
        x = rng.standard_normal(d) * 3.0
        w = rng.standard_normal(d)
        for eps in (1e-6, 1e-5, 0.5):
            ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (d,), torch.from_numpy(w), eps).numpy()
            np.testing.assert_allclose(po.rmsnorm(x, w, eps), ref, rtol=1e-13, atol=1e-15)
    # unit weight, no eps: the result has mean square 1; scaling the input changes nothing
    x = rng.standard_normal(64)
    y = po.rmsnorm(x, np.ones(64), 0.0)
    assert np.mean(y * y) == pytest.approx(1.0, rel=1e-13)
    np.testing.assert_allclose(po.rmsnorm(7.5 * x, np.ones(64), 0.0), y, rtol=1e-13)


def test_ffn_block_is_residual_plus_ffn_of_the_rounded_norm():
    wg, wu, wd, x = _problem(seed=22)
    d_model, d_ff = wg.shape[1], wg.shape[0]
    rng = np.random.default_rng(5)
    nw = po.bf16_to_f64(inputs.f32_to_bf16_bits((1.0 + 0.1 * rng.standard_normal(d_model)).astype(np.float32)))
    x_res = (x[0] * 2.5).astype(np.float32).astype(np.float64)
    out, call, xn = po.ffn_block(x_res, nw, 1e-6, 60, 100, wg, wu, wg, wu, wd)
    # the FFN input is a bf16 value next to the library's norm
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x_res), (d_model,), torch.from_numpy(nw), 1e-6).numpy()
    assert np.array_equal(po.bf16_to_f64(po.f64_to_bf16_bits(xn)), xn)
    assert np.all(np.abs(xn - ref) <= np.abs(ref) * 2.0 ** -8 + 1e-300)
    # residual: with the down projection zeroed the stream passes unchanged; with everything kept and the
    # original weights as proxy the block is x + dense FFN of the rounded norm (library ops)
    same, _, _ = po.ffn_block(x_res, nw, 1e-6, 60, 100, wg, wu, wg, wu, np.zeros_like(wd))
    assert np.array_equal(same, x_res)
    full, _, xn2 = po.ffn_block(x_res, nw, 1e-6, d_model, d_ff, wg, wu, wg, wu, wd)
    xt = torch.from_numpy(xn2)
    y_ref = torch.from_numpy(wd) @ ((torch.from_numpy(wu) @ xt) * torch.nn.functional.silu(torch.from_numpy(wg) @ xt))
    np.testing.assert_allclose(full, x_res + y_ref.numpy(), rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(out - x_res, call["y"], rtol=0, atol=1e-12)


def test_ffn_stack_chains_blocks():
    wg, wu, wd, x = _problem(seed=23)
    d_model = wg.shape[1]
    nw = np.ones(d_model)
    layers = [(nw, wg, wu, wg, wu, wd), (nw, wu, wg, wu, wg, wd)]
    xs = po.ffn_stack(x[1], layers, 1e-6, 50, 70)
    assert len(xs) == 3 and np.array_equal(xs[0], x[1])
    a, _, _ = po.ffn_block(x[1], nw, 1e-6, 50, 70, wg, wu, wg, wu, wd)
    b, _, _ = po.ffn_block(a, nw, 1e-6, 50, 70, wu, wg, wu, wg, wd)
    assert np.array_equal(xs[1], a) and np.array_equal(xs[2], b)


# ----------------------------------------------------- shared batch mask pins
def test_shared_mask_batch_reduces_to_single_token_and_ignores_token_order():
    wg, wu, wd, x = _problem(seed=31, n_tok=3)
    dg = po.dequantize(*po.quantize_proxy(wg, 4, 0), 0)
    du = po.dequantize(*po.quantize_proxy(wu, 4, 0), 0)
    k1, k2 = 70, 90
    one = po.forward(x[0], k1, k2, dg, du, wg, wu, wd)
    sel, thr, shared, ys = po.forward_batch_shared(x[:1], k1, k2, dg, du, wg, wu, wd)
    assert np.array_equal(sel, one["sel"]) and np.array_equal(ys[0], one["y"]) and thr == one["threshold"]
    # the same token twice: the sums double, the mask stays
    sel2, _, shared2, ys2 = po.forward_batch_shared(np.stack([x[0], x[0]]), k1, k2, dg, du, wg, wu, wd)
    assert np.array_equal(sel2, one["sel"]) and np.array_equal(shared2, 2 * one["score"])
    # three tokens: mask = full sort of the summed scores, unchanged by the order of the tokens,
    # and every token's y is Stage 2 on that mask (dense with the other channels zeroed)
    sel3, thr3, shared3, ys3 = po.forward_batch_shared(x, k1, k2, dg, du, wg, wu, wd)
    ref = sum(po.proxy_scores(x[b], po.input_topk(x[b], k1), dg, du) for b in (2, 0, 1))
    np.testing.assert_allclose(shared3, ref, rtol=1e-14)
    assert np.array_equal(sel3, np.sort(np.argsort(-shared3, kind="stable")[:k2]))
    selp, _, _, ysp = po.forward_batch_shared(x[::-1], k1, k2, dg, du, wg, wu, wd)
    assert np.array_equal(selp, sel3)
    for b in range(3):
        xt = torch.from_numpy(x[b])
        s_full = (torch.from_numpy(wu) @ xt) * torch.nn.functional.silu(torch.from_numpy(wg) @ xt)
        m = torch.zeros(wg.shape[0], dtype=torch.float64)
        m[torch.from_numpy(sel3)] = 1.0
        np.testing.assert_allclose(ys3[b], (torch.from_numpy(wd) @ (s_full * m)).numpy(), rtol=1e-10, atol=1e-13)
        np.testing.assert_allclose(ysp[2 - b], ys3[b], rtol=0, atol=0)


# ------------------------------------------------ threshold calibration (Alg. 1)
def test_counter_based_generator_matches_published_splitmix64_outputs():
    line = [l for l in open(os.path.join(GOLDEN, "splitmix64_reference.txt")) if l.startswith("splitmix64 ")][0].split()
    seed, want = int(line[1]), [int(v) for v in line[2:]]
    assert [po.splitmix64_at(seed, i) for i in range(len(want))] == want


def test_empirical_quantile_against_library_and_closed_form():
    rng = np.random.default_rng(5)
    for n in (1, 2, 7, 100, 1001):
        a = np.abs(rng.standard_normal(n)).astype(np.float32)
        for s in (0.0, 0.1, 0.5, 0.7, 0.767, 1.0):
            got = po.empirical_quantile(a, s)
            assert got.dtype == np.float32
            assert got == np.float32(np.quantile(a.astype(np.float64), s))
    # arithmetic progression 0, 1, ..., n-1: the s-quantile is s * (n - 1)
    assert po.empirical_quantile(np.arange(11, dtype=np.float32), 0.7) == np.float32(7.0)
    assert po.empirical_quantile(np.arange(5, dtype=np.float32), 0.6) == np.float32(2.4)
    # keeping |z| >= tau drops about a fraction s
    a = np.abs(rng.laplace(size=5000)).astype(np.float32)
    for s in (0.1, 0.55, 0.7):
        tau = po.empirical_quantile(a, s)
        assert abs(np.mean(a < tau) - s) <= 1.0 / a.size


def test_reservoir_size_membership_order_and_uniformity():
    v = np.arange(1, 101, dtype=np.float32) * np.where(np.arange(100) % 2 == 0, 1, -1)
    res, seen = po.reservoir(v, cap=200, seed=3)
    assert seen == 100 and res == [np.float32(i) for i in range(1, 101)]       # fewer than cap: all, in order, as magnitudes
    # more than cap: exactly cap kept, every kept value comes from the stream, continuing a call changes nothing
    n, cap = 20000, 500
    stream = np.arange(n, dtype=np.float32)
    res, seen = po.reservoir(stream, cap, seed=11)
    assert seen == n and len(res) == cap and set(res) <= set(stream.tolist())
    part, st = po.reservoir(stream[:7000], cap, seed=11)
    res2, _ = po.reservoir(stream[7000:], cap, seed=11, state=(part, st))
    assert res2 == res
    # hand-checked replacement rule on a tiny case: sample number i >= cap goes to slot u_i mod (i + 1) when that is < cap
    small, _ = po.reservoir(np.arange(6, dtype=np.float32), cap=3, seed=1)
    expect = [0.0, 1.0, 2.0]
    for i in (3, 4, 5):
        j = po.splitmix64_at(1, i) % (i + 1)
        if j < 3:
            expect[j] = float(i)
    assert [float(x) for x in small] == expect
    # uniform: every stream position is kept with probability cap / n (mean of kept positions ~ n / 2; the
    # standard error of that mean is n / sqrt(12 cap) ~ 258)
    assert abs(float(np.mean(res)) - n / 2) < 4 * n / math.sqrt(12 * cap)
    early = sum(1 for x in res if x < n / 4)
    assert abs(early - cap / 4) < 4 * math.sqrt(cap * 0.25 * 0.75)


def test_histogram_4096_counts_everything_once():
    rng = np.random.default_rng(2)
    a = np.abs(rng.standard_normal(3000)).astype(np.float32)
    counts, hi = po.histogram_4096(a)
    assert counts.shape == (4096,) and counts.sum() == a.size and hi == a.max()
    ref, _ = np.histogram(a.astype(np.float64), bins=4096, range=(0.0, float(hi)))
    assert np.abs(counts - ref).sum() <= 4                  # bin edges in float32 vs float64: a few borderline samples
    assert counts[-1] >= 1                                  # the maximum itself lands in the last bin
    z, hz = po.histogram_4096(np.zeros(5, dtype=np.float32))
    assert hz == 0 and z[-1] == 5


def _toy_stack(n_layers=3, d_model=128, d_ff=256, n_tok=12, seed=9):
    layers = []
    for l in range(n_layers):
        wg, wu, wd, x = inputs.make_small(d_model, d_ff, n_tok, seed + l, std=0.05)
        wg, wu, wd = po.bf16_to_f64(wg), po.bf16_to_f64(wu), po.bf16_to_f64(wd)
        qg, sg = po.quantize_proxy(wg, 4, 0)
        qu, su = po.quantize_proxy(wu, 4, 0)
        nw = 1.0 + 0.1 * np.cos(np.arange(d_model) + l)
        layers.append((po.bf16_to_f64(po.f64_to_bf16_bits(nw)), po.dequantize(qg, sg, 0), po.dequantize(qu, su, 0), wg, wu, wd))
    return layers, po.bf16_to_f64(x)


def test_sequential_calibration_realises_its_targets_and_sees_the_sparse_stream():
    """Alg. 1: thresholds are quantiles of the very samples they are then applied to, so on the calibration tokens
    every layer realises (s1, s2) to within one sample; layer l's thresholds come from the stream that the
    finalized rules of layers 1..l-1 produce, not from the dense stream."""
    layers, x0 = _toy_stack()
    s1, s2, eps = 0.55, 0.7, 1e-6
    cal = po.calibrate_stack(x0, layers, eps, s1, s2)
    n_tok, D, F = x0.shape[0], x0.shape[1], layers[0][3].shape[0]
    for c in cal:
        assert abs(c["s1_hat"] - s1) <= 4.0 / (n_tok * D) + 1e-12      # bf16 inputs: a few equal magnitudes at the threshold
        assert abs(c["s2_hat"] - s2) <= 1.5 / (n_tok * F) + 1e-12
        assert c["hist_x"][0].sum() == n_tok * D and c["hist_s"][0].sum() == n_tok * F
    # one layer alone = plain quantiles of that layer's own signals, by library routines
    nw, dg, du = layers[0][0], layers[0][1], layers[0][2]
    xn = np.stack([po.bf16_to_f64(po.f64_to_bf16_bits(po.rmsnorm(x, nw, eps))) for x in x0])
    tx = np.float32(np.quantile(np.abs(xn).astype(np.float32).astype(np.float64), s1))
    assert cal[0]["tau_x"] == tx
    sc = []
    for x in xn:
        xm = np.where(np.abs(x) >= tx, x, 0.0)
        g, u = torch.from_numpy(dg) @ torch.from_numpy(xm), torch.from_numpy(du) @ torch.from_numpy(xm)
        sc.append((u * torch.nn.functional.silu(g)).abs().numpy())
    ts = np.float32(np.quantile(np.concatenate(sc).astype(np.float32).astype(np.float64), s2))
    assert abs(float(cal[0]["tau_s"]) - float(ts)) <= 1e-6 * float(ts)
    # the stream matters: layer 2 calibrated behind a dense layer 1 gets other thresholds
    dense_first = po.calibrate_stack(x0, layers, eps, 0.0, 0.0)
    later = po.calibrate_stack([po.ffn_stack(x, layers[:1], eps, D, F)[-1] for x in x0], layers[1:], eps, s1, s2)
    assert dense_first[0]["s1_hat"] == 0.0 and dense_first[0]["s2_hat"] == 0.0
    assert later[0]["tau_x"] != cal[1]["tau_x"] or later[0]["tau_s"] != cal[1]["tau_s"]
    # ... and equals a calibration started from the sparse stream of layer 1 under its finalized rule
    x1 = []
    for x in x0:
        x_in = po.bf16_to_f64(po.f64_to_bf16_bits(po.rmsnorm(x, nw, eps)))
        sel = po.channel_threshold(po.proxy_scores(x_in, po.input_threshold(x_in, cal[0]["tau_x"]), dg, du), cal[0]["tau_s"])
        x1.append(x + po.stage2(x_in, sel, layers[0][3], layers[0][4], layers[0][5])[0])
    tail = po.calibrate_stack(x1, layers[1:], eps, s1, s2, seed=2)
    assert tail[0]["tau_x"] == cal[1]["tau_x"] and tail[0]["tau_s"] == cal[1]["tau_s"]
