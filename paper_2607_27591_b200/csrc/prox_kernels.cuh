// Device kernels of libprox (sm_100a).  One kernel per step of the path:
//   quantize/pack (offline)  ->  input top-k  ->  proxy GEMV + score
//   ->  channel top-k  ->  gather gate/up + SwiGLU  ->  masked down projection.
// Paper references are to Sec. 4.1 (two-stage inference), Sec. 4.3
// (hardware-aware implementation) and the appendix on top-k selection.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace prox {

constexpr int kMaxBatch = 8;
constexpr int kSelThreads = 1024;      // block size of the two selection kernels
constexpr int kProxyThreads = 256;     // proxy GEMV: 8 warps share one channel strip
constexpr int kProxyWarps = kProxyThreads / 32;

enum DevStatusBits : int { kBadChannel = 1, kBadInput = 2, kWaitExpired = 4 };

// ----------------------------------------------------------------------------
// small helpers
// ----------------------------------------------------------------------------
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may be set up
// while its predecessor on the stream still runs.  Called first thing: lets the NEXT kernel do the same, then
// waits until the predecessor has completed and its writes are visible.  Without the attribute both are no-ops.
__device__ __forceinline__ void pdl_enter() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

__device__ __forceinline__ uint4 ld_stream(const void* p) {   // read-once weights: bypass L1
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

__device__ __forceinline__ float silu_fast(float z) { return z / (1.0f + __expf(-z)); }
__device__ __forceinline__ float silu_exact(float z) { return z / (1.0f + expf(-z)); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Exclusive block scan of a 64-bit value over NT threads (NT multiple of 32,
// <= 1024).  `ws` is shared scratch of 33 entries.  Returns the exclusive
// prefix; *total receives the block sum.  Ends with a barrier, so `ws` can be
// reused right away.
template <int NT>
__device__ __forceinline__ unsigned long long block_scan_excl(unsigned long long v,
                                                              unsigned long long* ws,
                                                              unsigned long long* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned long long inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    unsigned long long t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) ws[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    unsigned long long w = (lane < NT / 32) ? ws[lane] : 0ull;
    unsigned long long winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      unsigned long long t = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += t;
    }
    ws[lane] = winc - w;
    if (lane == 31) ws[32] = winc;
  }
  __syncthreads();
  unsigned long long res = ws[warp] + inc - v;
  *total = ws[32];
  __syncthreads();
  return res;
}

// Given a histogram hist[0..NBINS) in shared memory, find the bin holding the
// k-th largest element (k >= 1, counting from the top bin down) and the number
// of elements in bins above it.  All NT threads call; result via shared out[2].
template <int NT, int NBINS>
__device__ __forceinline__ void find_kth_bin(const unsigned* hist, unsigned k,
                                             unsigned long long* ws, unsigned* out) {
  constexpr int PER = (NBINS + NT - 1) / NT;
  const int t = threadIdx.x;
  unsigned loc[PER];
  unsigned sum = 0;
#pragma unroll
  for (int p = 0; p < PER; ++p) {
    int bin = NBINS - 1 - (t * PER + p);
    loc[p] = (bin >= 0) ? hist[bin] : 0u;
    sum += loc[p];
  }
  unsigned long long tot;
  unsigned ex = (unsigned)block_scan_excl<NT>((unsigned long long)sum, ws, &tot);
  if (ex < k && k <= ex + sum) {
    unsigned run = ex;
#pragma unroll
    for (int p = 0; p < PER; ++p) {
      if (run < k && k <= run + loc[p]) {
        out[0] = (unsigned)(NBINS - 1 - (t * PER + p));
        out[1] = run;
      }
      run += loc[p];
    }
  }
  __syncthreads();
}

// ----------------------------------------------------------------------------
// Offline: scales, proxy packing, W_down transpose          (Sec. 4.3)
// ----------------------------------------------------------------------------
// Packed proxy layout ("input-major"): row i (one input coordinate) holds all
// channels; it is cut into 16-byte chunks, chunk c covering CH consecutive
// channels (CH = 16 for 4-bit, 8 for 8-bit):
//   words 0,1 : gate codes of channels c*CH .. c*CH+CH-1  (lowest bits first)
//   words 2,3 : up   codes of the same channels
// Codes are offset binary: q + 8 (4-bit) or q + 128 (8-bit).
// Scale layout: [group][chunk][2][CH] fp16 (gate scales then up scales).

// One warp per (channel j, group g): scale = fp16(absmax / qmax).
__global__ void proxy_scale_kernel(const __nv_bfloat16* __restrict__ wg,
                                   const __nv_bfloat16* __restrict__ wu, int D, int F, int G,
                                   int bits, __half* __restrict__ S, float* __restrict__ s_plain) {
  const int ngroups = D / G;
  const int CH = (bits == 4) ? 16 : 8;
  const long long warp_id = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const long long total = 2ll * F * ngroups;
  if (warp_id >= total) return;
  const int which = (int)(warp_id / ((long long)F * ngroups));
  const long long rem = warp_id % ((long long)F * ngroups);
  const int j = (int)(rem / ngroups), g = (int)(rem % ngroups);
  const __nv_bfloat16* w = (which ? wu : wg) + (size_t)j * D + (size_t)g * G;
  float a = 0.f;
  for (int i = lane; i < G; i += 32) a = fmaxf(a, fabsf(__bfloat162float(w[i])));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
  if (lane == 0) {
    const float qmax = (float)((1 << (bits - 1)) - 1);
    const __half s = __float2half_rn(__fdiv_rn(a, qmax));
    const int chunk = j / CH, c = j % CH;
    const int nchunks = F / CH;
    S[(((size_t)g * nchunks + chunk) * 2 + which) * CH + c] = s;
    s_plain[((size_t)which * F + j) * ngroups + g] = __half2float(s);
  }
}

// One thread per packed 32-bit word.
__global__ void proxy_pack_kernel(const __nv_bfloat16* __restrict__ wg,
                                  const __nv_bfloat16* __restrict__ wu, int D, int F, int G,
                                  int bits, const float* __restrict__ s_plain,
                                  uint32_t* __restrict__ P) {
  const int CH = (bits == 4) ? 16 : 8;
  const int per_word = (bits == 4) ? 8 : 4;
  const int nchunks = F / CH;
  const int ngroups = D / G;
  const long long words_per_row = (long long)nchunks * 4;
  // consecutive threads take consecutive input coordinates (coalesced reads of W)
  const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long total = words_per_row * D;
  if (tid >= total) return;
  const int i = (int)(tid % D);
  const long long wword = tid / D;                 // word index within the row
  const int chunk = (int)(wword >> 2), word = (int)(wword & 3);
  const int which = word >> 1;                     // 0 gate, 1 up
  const int j0 = chunk * CH + (word & 1) * per_word;
  const __nv_bfloat16* w = which ? wu : wg;
  const float qmax = (float)((1 << (bits - 1)) - 1);
  const int g = i / G;
  uint32_t out = 0;
  for (int m = 0; m < per_word; ++m) {
    const int j = j0 + m;
    const float s = s_plain[((size_t)which * F + j) * ngroups + g];
    const float v = __bfloat162float(w[(size_t)j * D + i]);
    int q = 0;
    if (s != 0.f) {
      float r = rintf(__fdiv_rn(v, s));
      r = fminf(fmaxf(r, -qmax), qmax);
      q = (int)r;
    }
    const uint32_t code = (uint32_t)(q + (bits == 4 ? 8 : 128));
    out |= code << (m * bits);
  }
  P[(size_t)i * words_per_row + wword] = out;
}

// 16-bit "proxies" (ablation A1 of Sec. "Ablation Studies"; also the 16-bit input-sparse GEMV that
// the cost ratio alpha of Sec. 4.2 is measured against): the original bf16 weights in the proxies'
// input-major order.  A 16-byte chunk of row i holds 4 channels: words 0,1 gate, words 2,3 up.
// One thread per 32-bit word (two channels of one matrix).
__global__ void proxy_pack16_kernel(const uint16_t* __restrict__ wg, const uint16_t* __restrict__ wu,
                                    int D, int F, uint32_t* __restrict__ P) {
  const long long words_per_row = (long long)(F / 4) * 4;
  const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (tid >= words_per_row * D) return;
  const int i = (int)(tid % D);                    // consecutive threads: consecutive inputs (coalesced reads)
  const long long wword = tid / D;
  const int chunk = (int)(wword >> 2), word = (int)(wword & 3);
  const uint16_t* w = (word >> 1) ? wu : wg;
  const int j0 = chunk * 4 + (word & 1) * 2;
  P[(size_t)i * words_per_row + wword] =
      (uint32_t)w[(size_t)j0 * D + i] | ((uint32_t)w[(size_t)(j0 + 1) * D + i] << 16);
}

// W_down [D, F] -> channel-major [F, D]  (Sec. 3.1: y = sum_j s_j W_down[j,:]).
__global__ void transpose_bf16_kernel(const uint16_t* __restrict__ in, uint16_t* __restrict__ out,
                                      int rows, int cols) {
  __shared__ uint16_t tile[32][33];
  int c = blockIdx.x * 32 + threadIdx.x;
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    int rr = blockIdx.y * 32 + r;
    if (rr < rows && c < cols) tile[r][threadIdx.x] = in[(size_t)rr * cols + c];
  }
  __syncthreads();
  int oc = blockIdx.y * 32 + threadIdx.x;            // output column = input row
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    int orow = blockIdx.x * 32 + r;                  // output row = input column
    if (orow < cols && oc < rows) out[(size_t)orow * rows + oc] = tile[threadIdx.x][r];
  }
}

// ----------------------------------------------------------------------------
// Input mask m_x: exact top-k1 of |x_i| (ties -> lower index), or |x_i| >= tau.
// One block per token.  bf16 magnitudes compare as 15-bit integers.
// ----------------------------------------------------------------------------
constexpr int kMaxInPer = 16;  // d_model <= 16384

__global__ void __launch_bounds__(kSelThreads)
input_select_kernel(const uint16_t* __restrict__ x, int D, int k1, float tau, int use_tau,
                    int* __restrict__ idx_out, int idx_stride, int* __restrict__ cnt_out) {
  __shared__ unsigned hist[256];
  __shared__ unsigned long long ws[33];
  __shared__ unsigned res[2];
  const int b = blockIdx.x, t = threadIdx.x;
  const uint16_t* xb = x + (size_t)b * D;
  const int per = (D + kSelThreads - 1) / kSelThreads;
  const int base = t * per;
  unsigned key[kMaxInPer];
#pragma unroll
  for (int e = 0; e < kMaxInPer; ++e) {
    const int i = base + e;
    key[e] = (e < per && i < D) ? (unsigned)(xb[i] & 0x7fffu) : 0xffffffffu;  // sentinel: not an element
  }
  unsigned T, quota;
  if (use_tau) {
    T = 0; quota = 0;   // unused
  } else {
    // level 1: bits 14..7
    if (t < 256) hist[t] = 0;
    __syncthreads();
#pragma unroll
    for (int e = 0; e < kMaxInPer; ++e)
      if (key[e] != 0xffffffffu) atomicAdd(&hist[key[e] >> 7], 1u);
    __syncthreads();
    find_kth_bin<kSelThreads, 256>(hist, (unsigned)k1, ws, res);
    const unsigned bin1 = res[0], above1 = res[1];
    __syncthreads();
    // level 2: bits 6..0 among keys in bin1
    if (t < 256) hist[t] = 0;
    __syncthreads();
#pragma unroll
    for (int e = 0; e < kMaxInPer; ++e)
      if (key[e] != 0xffffffffu && (key[e] >> 7) == bin1) atomicAdd(&hist[key[e] & 127u], 1u);
    __syncthreads();
    find_kth_bin<kSelThreads, 128>(hist, (unsigned)k1 - above1, ws, res);
    T = (bin1 << 7) | res[0];
    quota = (unsigned)k1 - above1 - res[1];      // ties at T to accept, lowest index first
    __syncthreads();
  }
  unsigned gt = 0, eq = 0;
#pragma unroll
  for (int e = 0; e < kMaxInPer; ++e) {
    if (key[e] == 0xffffffffu) continue;
    if (use_tau) {
      gt += (__uint_as_float(key[e] << 16) >= tau) ? 1u : 0u;
    } else {
      gt += (key[e] > T) ? 1u : 0u;
      eq += (key[e] == T) ? 1u : 0u;
    }
  }
  unsigned long long tot;
  unsigned long long ex = block_scan_excl<kSelThreads>(((unsigned long long)eq << 32) | gt, ws, &tot);
  unsigned gtb = (unsigned)(ex & 0xffffffffu), eqb = (unsigned)(ex >> 32);
  int* out = idx_out + (size_t)b * idx_stride;
#pragma unroll
  for (int e = 0; e < kMaxInPer; ++e) {
    if (key[e] == 0xffffffffu) continue;
    bool g, q;
    if (use_tau) { g = __uint_as_float(key[e] << 16) >= tau; q = false; }
    else { g = key[e] > T; q = key[e] == T; }
    if (g || (q && eqb < quota)) out[gtb + min(eqb, quota)] = base + e;
    gtb += g ? 1u : 0u;
    eqb += q ? 1u : 0u;
  }
  if (cnt_out && t == 0) {
    unsigned tg = (unsigned)(tot & 0xffffffffu), te = (unsigned)(tot >> 32);
    cnt_out[b] = (int)(tg + (use_tau ? 0u : min(te, quota)));
  }
}

// ----------------------------------------------------------------------------
// Proxy GEMV (fused gate + up), Sec. 4.1 proxy equations / Sec. 4.3 Stage 1.
//   g~_j = sum_{i in I_x} x_i deq(W~_gate)_{j,i},   u~_j likewise,
//   score_j = |u~_j SiLU(g~_j)|.
// grid = (strips, ksplit, B); a strip is 32*CH channels; the 8 warps of a block
// split the block's share of kept rows; partial sums meet in shared memory,
// blocks of the same strip meet through a partial buffer and the last one to
// arrive (ticket counter, nobody waits) finishes the scores.
// 4-bit codes become fp32 without an int->float convert: the code is moved into
// the top mantissa bits of 2.0f, giving f = 2 + code/8 = 3 + q/8, and the
// constant 3 is removed once per group: sum x q = 8 (sum x f - 3 sum x).
// ----------------------------------------------------------------------------
template <int BITS>
struct ProxyFmt {
  static constexpr int CH = (BITS == 4) ? 16 : (BITS == 8 ? 8 : 4);    // channels per 16-byte chunk
  static constexpr int NACC = 2 * CH;
};

template <int BITS>
__device__ __forceinline__ void proxy_accumulate(const uint4& v, float xv, float* acc) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
  if (BITS == 4) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
#pragma unroll
      for (int m = 0; m < 8; ++m) {
        const int sh = 19 - 4 * m;
        const uint32_t t = (sh >= 0) ? (w[q] << sh) : (w[q] >> (-sh));
        uint32_t bits;                                          // (t & mask) | magic as one lop3
        asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(bits) : "r"(t), "r"(0x00780000u), "r"(0x40000000u));
        acc[q * 8 + m] = fmaf(__uint_as_float(bits), xv, acc[q * 8 + m]);
      }
    }
  } else if (BITS == 8) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
#pragma unroll
      for (int m = 0; m < 4; ++m) {
        const uint32_t bits = __byte_perm(w[q], 0x4B000000u, 0x7650u | m);
        const float f = __uint_as_float(bits) - 8388736.0f;     // 2^23 + 128
        acc[q * 4 + m] = fmaf(f, xv, acc[q * 4 + m]);
      }
    }
  } else {
#pragma unroll
    for (int q = 0; q < 4; ++q) {                               // bf16 weights as they are
      acc[q * 2] = fmaf(__uint_as_float(w[q] << 16), xv, acc[q * 2]);
      acc[q * 2 + 1] = fmaf(__uint_as_float(w[q] & 0xffff0000u), xv, acc[q * 2 + 1]);
    }
  }
}

// Variant that forms the exact integer code q = n - 8 with full-rate
// instructions only.  A 4-bit code sitting at bit 4m (m <= 4) of a word, OR-ed
// into the mantissa of 2^(23-4m), is the float 2^(23-4m) + n; one LOP3 isolates
// it, one FADD removes 2^(23-4m) + 8, one FFMA accumulates q * x (exact product,
// nothing to correct later).  The three codes above bit 19 are reached through
// one shift of the word by 12.  On this GPU shifts, byte permutes and packed
// half arithmetic issue at half the rate of LOP3 / FADD / FFMA.
template <int BITS>
__device__ __forceinline__ void proxy_accumulate_exact(const uint4& v, float xv, float* acc) {
  if (BITS == 4) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const uint32_t hi = w[q] >> 12;
#pragma unroll
      for (int m = 0; m < 8; ++m) {
        const int pos = (m < 5) ? m : (m - 3);                  // code position inside w or inside hi
        const uint32_t src = (m < 5) ? w[q] : hi;
        const uint32_t magic = (uint32_t)(150 - 4 * pos) << 23;  // 2^(23 - 4 pos)
        const float off = (float)(1u << (23 - 4 * pos)) + 8.0f;
        // (src & mask) | magic as ONE lop3 (truth table 0xEA), written out: left to the compiler, the
        // unpack took 184 cycles per 16-byte chunk and warp instead of 145
        uint32_t bits;
        asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(bits) : "r"(src), "r"(0xFu << (4 * pos)), "r"(magic));
        const float f = __uint_as_float(bits) - off;
        acc[q * 8 + m] = fmaf(f, xv, acc[q * 8 + m]);
      }
    }
  } else {
    proxy_accumulate<8>(v, xv, acc);
  }
}

template <int BITS>
__global__ void __launch_bounds__(kProxyThreads, BITS == 16 ? 3 : 2)
proxy_gemv_kernel(const uint8_t* __restrict__ P, const __half* __restrict__ S,
                  const uint16_t* __restrict__ x, const int* __restrict__ idx, int idx_stride,
                  const int* __restrict__ cnt, int k1_static, int D, int F, int gshift,
                  float* __restrict__ part, unsigned* __restrict__ ticket,
                  float* __restrict__ scores, float* __restrict__ values, int* __restrict__ status) {
  constexpr int CH = ProxyFmt<BITS>::CH, NACC = ProxyFmt<BITS>::NACC;
  constexpr int U = 8;
  extern __shared__ float red[];                    // [warps][NACC*32]
  __shared__ int s_last;
  const int strip = blockIdx.x, ks = blockIdx.y, b = blockIdx.z;
  const int nstrips = gridDim.x, ksplit = gridDim.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nchunks = F / CH;
  const int chunk = strip * 32 + lane;
  const bool valid = chunk < nchunks;
  const size_t row_bytes = (size_t)nchunks * 16;
  const int n = cnt ? cnt[b] : k1_static;
  const int* idb = idx + (size_t)b * idx_stride;
  const uint16_t* xb = x + (size_t)b * D;

  const int r0 = (int)(((long long)n * ks) / ksplit), r1 = (int)(((long long)n * (ks + 1)) / ksplit);
  const int w0 = r0 + (int)(((long long)(r1 - r0) * warp) / kProxyWarps);
  const int w1 = r0 + (int)(((long long)(r1 - r0) * (warp + 1)) / kProxyWarps);

  float acc[NACC], tot[NACC];
#pragma unroll
  for (int c = 0; c < NACC; ++c) { acc[c] = 0.f; tot[c] = 0.f; }
  float sumx = 0.f;
  int curg = -1;

  auto flush = [&](int g) {
    if (g < 0 || !valid) return;
    if (BITS == 16) {                                 // no scales: the weights themselves
#pragma unroll
      for (int c = 0; c < NACC; ++c) { tot[c] += acc[c]; acc[c] = 0.f; }
      return;
    }
    const uint4* sp = reinterpret_cast<const uint4*>(S + ((size_t)g * nchunks + chunk) * NACC);
#pragma unroll
    for (int v4 = 0; v4 < (NACC >= 8 ? NACC / 8 : 1); ++v4) {
      const uint4 sv = __ldg(sp + v4);
      const uint32_t sw[4] = {sv.x, sv.y, sv.z, sv.w};
#pragma unroll
      for (int h2 = 0; h2 < 4; ++h2) {
        const float2 sc = __half22float2(*reinterpret_cast<const __half2*>(&sw[h2]));
        const int c = v4 * 8 + h2 * 2;
        if (BITS == 4) {
          tot[c] = fmaf(sc.x * 8.0f, fmaf(-3.0f, sumx, acc[c]), tot[c]);
          tot[c + 1] = fmaf(sc.y * 8.0f, fmaf(-3.0f, sumx, acc[c + 1]), tot[c + 1]);
        } else {
          tot[c] = fmaf(sc.x, acc[c], tot[c]);
          tot[c + 1] = fmaf(sc.y, acc[c + 1], tot[c + 1]);
        }
        acc[c] = 0.f; acc[c + 1] = 0.f;
      }
    }
    sumx = 0.f;
  };

  for (int r = w0; r < w1; r += U) {
    int ii[U];
    uint4 v[U];
    float xv[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      ii[u] = (r + u < w1) ? __ldg(idb + r + u) : -1;
      if (ii[u] >= D) { ii[u] = -1; atomicOr(status, kBadInput); }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      v[u] = make_uint4(0, 0, 0, 0);
      xv[u] = 0.f;
      if (ii[u] >= 0) {
        if (valid) v[u] = ld_stream(P + (size_t)ii[u] * row_bytes + (size_t)chunk * 16);
        xv[u] = __uint_as_float(((uint32_t)xb[ii[u]]) << 16);
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      if (ii[u] < 0) continue;
      const int g = ii[u] >> gshift;
      if (g != curg) { flush(curg); curg = g; }
      sumx += xv[u];
      proxy_accumulate<BITS>(v[u], xv[u], acc);
    }
  }
  flush(curg);

  // meet in shared memory: element k = c*32 + lane of this strip
  float* mine = red + warp * (NACC * 32);
#pragma unroll
  for (int c = 0; c < NACC; ++c) mine[c * 32 + lane] = tot[c];
  __syncthreads();
  constexpr int PER_T = NACC * 32 / kProxyThreads;
  float sumv[PER_T];
#pragma unroll
  for (int p = 0; p < PER_T; ++p) {
    const int k = threadIdx.x + p * kProxyThreads;
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < kProxyWarps; ++w) s += red[w * (NACC * 32) + k];
    sumv[p] = s;
  }
  __syncthreads();
  // element k -> (c = k / 32, lane = k % 32): c < CH is gate, else up
  float* fin = red;                                  // reuse: final sums of the strip
  if (ksplit == 1) {
#pragma unroll
    for (int p = 0; p < PER_T; ++p) fin[threadIdx.x + p * kProxyThreads] = sumv[p];
    __syncthreads();
  } else {
    float* pb = part + (((size_t)b * ksplit + ks) * nstrips + strip) * (NACC * 32);
#pragma unroll
    for (int p = 0; p < PER_T; ++p) __stcg(pb + threadIdx.x + p * kProxyThreads, sumv[p]);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
      const unsigned tk = atomicAdd(&ticket[b * nstrips + strip], 1u);
      s_last = (tk == (unsigned)(ksplit - 1));
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
#pragma unroll
    for (int p = 0; p < PER_T; ++p) {
      const int k = threadIdx.x + p * kProxyThreads;
      float s = 0.f;
      for (int q = 0; q < ksplit; ++q)
        s += __ldcg(part + (((size_t)b * ksplit + q) * nstrips + strip) * (NACC * 32) + k);
      fin[k] = s;
    }
    if (threadIdx.x == 0) ticket[b * nstrips + strip] = 0;   // ready for the next call
    __syncthreads();
  }
  // score_j = |u~_j SiLU(g~_j)|   (never stored as separate u~, g~ vectors)
  for (int k = threadIdx.x; k < CH * 32; k += kProxyThreads) {
    const int c = k >> 5, ln = k & 31;
    const int ch = (strip * 32 + ln) * CH + c;
    if (ch < F) {
      const float g = fin[k], u = fin[k + CH * 32];
      const float v = u * silu_fast(g);
      scores[(size_t)b * F + ch] = fabsf(v);
      if (values) values[(size_t)b * F + ch] = v;     // signed s~, for the proxy-values-into-down variant
    }
  }
}

// ----------------------------------------------------------------------------
// Channel mask m_s: exact top-k2 of the scores (ties -> lower index), or
// score >= tau.  One block per token; radix select on the fp32 bit pattern
// (scores are >= 0, so unsigned order = numeric order), 11 + 11 + 9 bits.
// ----------------------------------------------------------------------------
constexpr int kMaxChPer = 64;   // d_ff <= 65536

__global__ void __launch_bounds__(kSelThreads)
channel_select_kernel(const float* __restrict__ scores, int F, int k2, float tau, int use_tau,
                      int* __restrict__ sel_out, int sel_stride, int* __restrict__ cnt_out) {
  __shared__ unsigned hist[2048];
  __shared__ unsigned long long ws[33];
  __shared__ unsigned res[2];
  const int b = blockIdx.x, t = threadIdx.x;
  const unsigned* sb = reinterpret_cast<const unsigned*>(scores) + (size_t)b * F;
  int per = (F + kSelThreads - 1) / kSelThreads;
  per = (per + 3) & ~3;                               // contiguous run per thread, float4 friendly
  const int base = t * per;
  const int lim = min(F, base + per);

  unsigned T = 0, quota = 0;
  if (!use_tau) {
    unsigned prefix = 0, kk = (unsigned)k2;
    const int shifts[3] = {20, 9, 0};
    const int nbits[3] = {11, 11, 9};
#pragma unroll
    for (int lv = 0; lv < 3; ++lv) {
      for (int i = t; i < 2048; i += kSelThreads) hist[i] = 0;
      __syncthreads();
      const int sh = shifts[lv], nb = nbits[lv];
      for (int i = base; i < lim; ++i) {
        const unsigned key = sb[i] & 0x7fffffffu;
        if (lv == 0 || (key >> (sh + nb)) == prefix) atomicAdd(&hist[(key >> sh) & ((1u << nb) - 1u)], 1u);
      }
      __syncthreads();
      if (lv < 2) find_kth_bin<kSelThreads, 2048>(hist, kk, ws, res);
      else        find_kth_bin<kSelThreads, 512>(hist, kk, ws, res);
      prefix = (prefix << nb) | res[0];
      kk -= res[1];
      __syncthreads();
    }
    T = prefix;
    quota = kk;
  }
  unsigned gt = 0, eq = 0;
  for (int i = base; i < lim; ++i) {
    const unsigned key = sb[i] & 0x7fffffffu;
    if (use_tau) gt += (__uint_as_float(key) >= tau) ? 1u : 0u;
    else { gt += (key > T) ? 1u : 0u; eq += (key == T) ? 1u : 0u; }
  }
  unsigned long long tot;
  unsigned long long ex = block_scan_excl<kSelThreads>(((unsigned long long)eq << 32) | gt, ws, &tot);
  unsigned gtb = (unsigned)(ex & 0xffffffffu), eqb = (unsigned)(ex >> 32);
  int* out = sel_out + (size_t)b * sel_stride;
  for (int i = base; i < lim; ++i) {
    const unsigned key = sb[i] & 0x7fffffffu;
    bool g, q;
    if (use_tau) { g = __uint_as_float(key) >= tau; q = false; }
    else { g = key > T; q = key == T; }
    if (g || (q && eqb < quota)) out[gtb + min(eqb, quota)] = i;
    gtb += g ? 1u : 0u;
    eqb += q ? 1u : 0u;
  }
  if (cnt_out && t == 0) {
    unsigned tg = (unsigned)(tot & 0xffffffffu), te = (unsigned)(tot >> 32);
    cnt_out[b] = (int)(tg + (use_tau ? 0u : min(te, quota)));
  }
}

// ----------------------------------------------------------------------------
// Stage 2a: h_j = SiLU(x . W_gate[j,:]) * (x . W_up[j,:]) for j in the mask
// (Sec. 4.1 Stage 2, Pi_out with the original weights and the dense x).
// One warp per kept channel; x staged in shared memory as bf16.
// ----------------------------------------------------------------------------
constexpr int kGateUpThreads = 256;

__global__ void __launch_bounds__(kGateUpThreads)
gateup_kernel(const uint16_t* __restrict__ wg, const uint16_t* __restrict__ wu,
              const uint16_t* __restrict__ x, const int* __restrict__ sel, int sel_stride,
              const int* __restrict__ cnt, int k2_static, int D, int F,
              float* __restrict__ h_out, int h_stride, int* __restrict__ status) {
  extern __shared__ uint4 xs4[];                      // D bf16
  const int b = blockIdx.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n = cnt ? cnt[b] : k2_static;
  if ((int)blockIdx.x * (kGateUpThreads / 32) >= n) return;
  const uint4* xg = reinterpret_cast<const uint4*>(x + (size_t)b * D);
  for (int i = threadIdx.x; i < D / 8; i += kGateUpThreads) xs4[i] = __ldg(xg + i);
  __syncthreads();
  const int r = blockIdx.x * (kGateUpThreads / 32) + warp;
  if (r >= n) return;
  const int j = sel[(size_t)b * sel_stride + r];
  if (j < 0 || j >= F) {
    if (lane == 0) { atomicOr(status, kBadChannel); h_out[(size_t)b * h_stride + r] = 0.f; }
    return;
  }
  const uint4* g4 = reinterpret_cast<const uint4*>(wg + (size_t)j * D);
  const uint4* u4 = reinterpret_cast<const uint4*>(wu + (size_t)j * D);
  const int nv = D / 8;                               // 16-byte vectors per row
  float ag = 0.f, au = 0.f;
  constexpr int UN = 4;
  for (int i0 = lane; i0 < nv; i0 += 32 * UN) {
    uint4 a[UN], c[UN];
#pragma unroll
    for (int u = 0; u < UN; ++u) {
      const int i = i0 + 32 * u;
      if (i < nv) { a[u] = ld_stream(g4 + i); c[u] = ld_stream(u4 + i); }
    }
#pragma unroll
    for (int u = 0; u < UN; ++u) {
      const int i = i0 + 32 * u;
      if (i < nv) {
        const uint4 xv = xs4[i];
        const uint32_t xw[4] = {xv.x, xv.y, xv.z, xv.w};
        const uint32_t aw[4] = {a[u].x, a[u].y, a[u].z, a[u].w};
        const uint32_t cw[4] = {c[u].x, c[u].y, c[u].z, c[u].w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float x0 = bf16_lo(xw[q]), x1 = bf16_hi(xw[q]);
          ag = fmaf(bf16_lo(aw[q]), x0, ag); ag = fmaf(bf16_hi(aw[q]), x1, ag);
          au = fmaf(bf16_lo(cw[q]), x0, au); au = fmaf(bf16_hi(cw[q]), x1, au);
        }
      }
    }
  }
  ag = warp_sum(ag);
  au = warp_sum(au);
  if (lane == 0) h_out[(size_t)b * h_stride + r] = au * silu_exact(ag);
}

// Proxy values into the down projection (ablation A3): h_r = s~[sel[r]].
__global__ void gather_values_kernel(const float* __restrict__ values, const int* __restrict__ sel,
                                     int sel_stride, int k2, int F, float* __restrict__ h_out, int h_stride,
                                     int* __restrict__ status) {
  const int b = blockIdx.y, r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= k2) return;
  const int j = sel[(size_t)b * sel_stride + r];
  if (j < 0 || j >= F) { atomicOr(status, kBadChannel); h_out[(size_t)b * h_stride + r] = 0.f; return; }
  h_out[(size_t)b * h_stride + r] = values[(size_t)b * F + j];
}

// ----------------------------------------------------------------------------
// Stage 2b: y = sum_{j in mask} h_j W_down[j,:]   (Sec. 4.1; Sec. 3.1 weighted
// sum view) over the channel-major copy of W_down.  grid = (D tiles, channel
// splits, B); each thread owns 8 outputs; partial sums are added to an fp32
// accumulator with atomics; a last small kernel rounds once to the output type.
// ----------------------------------------------------------------------------
constexpr int kDownThreads = 256;
constexpr int kDownChunk = 512;     // max channels staged per pass

__global__ void __launch_bounds__(kDownThreads)
down_kernel(const uint16_t* __restrict__ wdt, const float* __restrict__ h, int h_stride,
            const int* __restrict__ sel, int sel_stride, const int* __restrict__ cnt,
            int k2_static, int D, int F, float* __restrict__ yacc) {
  __shared__ float hs[kDownChunk];
  __shared__ int js[kDownChunk];
  const int b = blockIdx.z;
  const int n = cnt ? cnt[b] : k2_static;
  const int nsplit = gridDim.y, sp = blockIdx.y;
  const int c0 = (int)(((long long)n * sp) / nsplit), c1 = (int)(((long long)n * (sp + 1)) / nsplit);
  const int e = (blockIdx.x * kDownThreads + threadIdx.x) * 8;
  float acc[8];
#pragma unroll
  for (int m = 0; m < 8; ++m) acc[m] = 0.f;
  for (int cb = c0; cb < c1; cb += kDownChunk) {
    const int cn = min(kDownChunk, c1 - cb);
    __syncthreads();
    for (int i = threadIdx.x; i < cn; i += kDownThreads) {
      int j = sel[(size_t)b * sel_stride + cb + i];
      float hv = h[(size_t)b * h_stride + cb + i];
      if (j < 0 || j >= F) { j = 0; hv = 0.f; }       // already recorded by the gate/up kernel
      js[i] = j; hs[i] = hv;
    }
    __syncthreads();
    if (e < D) {
      constexpr int UN = 8;
      for (int i0 = 0; i0 < cn; i0 += UN) {
        uint4 w[UN];
#pragma unroll
        for (int u = 0; u < UN; ++u)
          if (i0 + u < cn) w[u] = ld_stream(wdt + (size_t)js[i0 + u] * D + e);
#pragma unroll
        for (int u = 0; u < UN; ++u) {
          if (i0 + u < cn) {
            const float hv = hs[i0 + u];
            const uint32_t ww[4] = {w[u].x, w[u].y, w[u].z, w[u].w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              acc[2 * q] = fmaf(hv, bf16_lo(ww[q]), acc[2 * q]);
              acc[2 * q + 1] = fmaf(hv, bf16_hi(ww[q]), acc[2 * q + 1]);
            }
          }
        }
      }
    }
  }
  if (e < D && c1 > c0) {
    float* yp = yacc + (size_t)b * D + e;
#pragma unroll
    for (int m = 0; m < 8; ++m) atomicAdd(yp + m, acc[m]);
  }
}

// Round the fp32 accumulator once to the output type and clear it for the next call.
// With `resid` (layer sub-block form): y = resid + accumulator, fp32 (y may be resid itself).
__global__ void finalize_kernel(float* __restrict__ yacc, void* y, int n, int out_fp32,
                                const float* resid = nullptr) {
  pdl_enter();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const float v = yacc[i];
  yacc[i] = 0.f;
  if (resid) reinterpret_cast<float*>(y)[i] = resid[i] + v;
  else if (out_fp32) reinterpret_cast<float*>(y)[i] = v;
  else reinterpret_cast<__nv_bfloat16*>(y)[i] = __float2bfloat16_rn(v);
}

// ----------------------------------------------------------------------------
// FFN input of a layer sub-block: bf16(x / sqrt(mean(x^2) + eps) * w).
// The masks depend on this rounding, so it must be the rounding of the exact
// value.  The arithmetic is done on pairs of floats (an unevaluated sum hi + lo,
// about 2^-44 relative) rather than in fp64: the same result for this purpose, no
// fp64 divide / square-root subroutines in the prologue of the persistent kernel,
// and full-rate instructions only.
// ----------------------------------------------------------------------------
__device__ __forceinline__ void two_sum(float a, float b, float& s, float& e) {   // a + b = s + e exactly
  s = __fadd_rn(a, b);
  const float bb = __fsub_rn(s, a);
  e = __fadd_rn(__fsub_rn(a, __fsub_rn(s, bb)), __fsub_rn(b, bb));
}

// (hi, lo) += x * x
__device__ __forceinline__ void f2_add_square(float& hi, float& lo, float x) {
  const float p = __fmul_rn(x, x), pe = __fmaf_rn(x, x, -p);
  float s, e;
  two_sum(hi, p, s, e);
  lo = __fadd_rn(lo, __fadd_rn(e, pe));
  hi = s;
}

__device__ __forceinline__ void f2_warp_sum(float& hi, float& lo) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float oh = __shfl_xor_sync(0xffffffffu, hi, o), ol = __shfl_xor_sync(0xffffffffu, lo, o);
    float s, e;
    two_sum(hi, oh, s, e);
    lo = __fadd_rn(__fadd_rn(lo, ol), e);
    hi = s;
  }
}

// The scalars 1/D and eps as pairs of floats, split on the host.
struct RmsConst { float idh, idl, eh, el; };

// sum of squares (hi + lo) -> 1 / sqrt(sum / D + eps) as a pair of floats: pair product, pair sum,
// then one Newton step on rsqrtf whose residual 1 - m y0^2 is formed exactly enough (about 2^-44
// in the end).
__device__ __forceinline__ void rms_inverse(float hi, float lo, const RmsConst& c, float& ih, float& il) {
  const float ph = __fmul_rn(hi, c.idh), pe = __fmaf_rn(hi, c.idh, -ph);
  const float pl = __fmaf_rn(lo, c.idh, __fmaf_rn(hi, c.idl, pe));
  float s, e;
  two_sum(ph, c.eh, s, e);
  const float l = __fadd_rn(__fadd_rn(e, pl), c.el);
  float mh, ml;
  two_sum(s, l, mh, ml);                                                    // m = mean + eps
  const float y0 = rsqrtf(mh);
  const float a = __fmul_rn(y0, y0), ae = __fmaf_rn(y0, y0, -a);            // y0^2 = a + ae
  const float th = __fmul_rn(mh, a), te = __fmaf_rn(mh, a, -th);            // mh a = th + te
  const float rest = __fadd_rn(te, __fmaf_rn(mh, ae, __fmul_rn(ml, a)));
  const float rho = __fsub_rn(__fsub_rn(1.0f, th), rest);                   // 1 - m y0^2 (1 - th is exact)
  const float corr = __fmul_rn(__fmul_rn(0.5f, y0), rho);
  two_sum(y0, corr, ih, il);
}

// nearest bf16 (ties to even) of x * w * (ih + il)
__device__ __forceinline__ uint16_t rms_scale_to_bf16(float x, float w, float ih, float il) {
  const float p = __fmul_rn(x, w), e = __fmaf_rn(x, w, -p);                 // x w = p + e exactly
  const float q = __fmul_rn(p, ih), qe = __fmaf_rn(p, ih, -q);              // p ih = q + qe exactly
  const float r = __fmaf_rn(p, il, __fmaf_rn(e, ih, qe));                   // the rest, to ~2^-44
  float s, t;
  two_sum(q, r, s, t);                                                      // s = nearest float, t = what is left
  uint32_t u = __float_as_uint(s);
  if ((u & 0xffffu) == 0x8000u && t != 0.f) {
    // s sits exactly between two bf16 values: the remainder decides (towards larger magnitude or not)
    const bool up = (t > 0.f) == (s > 0.f);
    return (uint16_t)((u >> 16) + (up ? 1u : 0u));
  }
  u += 0x7fffu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}

// One block per token (the batch and step-wise paths; the persistent kernel has this in its prologue).
__global__ void __launch_bounds__(256) rmsnorm_kernel(const float* __restrict__ xres, const uint16_t* __restrict__ w,
                                                      RmsConst rc, int D, uint16_t* __restrict__ out) {
  __shared__ float wh[8], wl[8], inv[2];
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* x = xres + (size_t)b * D;
  float hi = 0.f, lo = 0.f;
  for (int i = tid; i < D; i += 256) f2_add_square(hi, lo, x[i]);
  f2_warp_sum(hi, lo);
  if (lane == 0) { wh[warp] = hi; wl[warp] = lo; }
  __syncthreads();
  if (warp == 0) {
    hi = lane < 8 ? wh[lane] : 0.f;
    lo = lane < 8 ? wl[lane] : 0.f;
    f2_warp_sum(hi, lo);
    if (lane == 0) rms_inverse(hi, lo, rc, inv[0], inv[1]);
  }
  __syncthreads();
  const float ih = inv[0], il = inv[1];
  for (int i = tid; i < D; i += 256)
    out[(size_t)b * D + i] = rms_scale_to_bf16(x[i], __uint_as_float((uint32_t)w[i] << 16), ih, il);
}

}  // namespace prox
