// Batch B > 1 with per-token masks (the paper treats batch 1 only; every token
// keeps its own m_x and m_s, Sec. 4.1).  Weights are read ONCE per call for the
// union of the tokens' kept inputs / channels; a token contributes zero outside
// its own masks (adding 0 * w is exact), so each token's result is the one it
// would get alone.
#pragma once

#include "prox_kernels.cuh"

namespace prox {

constexpr int kBT = 8;                  // token slots carried per union row (max batch)

// ----------------------------------------------------------------------------
// Union of the tokens' ascending index lists (kept inputs or kept channels).
// One block.  Outputs the ascending union list, its length, and per union row
// eight values: for inputs the token's x at that coordinate (0 if the token
// dropped it), for channels 1 / 0 membership.
// ----------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
union_kernel(const int* __restrict__ lists, int stride, const int* __restrict__ cnt, int k_static, int B,
             int n, const uint16_t* __restrict__ x, int* __restrict__ ulist, int* __restrict__ nu_out,
             float* __restrict__ val, int* __restrict__ status) {
  extern __shared__ unsigned ubits[];                  // [B][nw] token bit sets, [nw] union, [nw] offsets
  __shared__ unsigned long long ws[33];
  const int nw = (n + 31) / 32;
  const int t = threadIdx.x;
  for (int i = t; i < B * nw; i += 1024) ubits[i] = 0;
  __syncthreads();
  for (int b = 0; b < B; ++b) {
    const int c = cnt ? cnt[b] : k_static;
    for (int r = t; r < c; r += 1024) {
      const int id = lists[(size_t)b * stride + r];
      if (id >= 0 && id < n) atomicOr(&ubits[b * nw + (id >> 5)], 1u << (id & 31));
      else atomicOr(status, kBadChannel);
    }
  }
  __syncthreads();
  // union words, their popcounts, and an exclusive scan of those (nw <= 2048)
  unsigned* uw = ubits + (size_t)B * nw;               // [nw] union words, then [nw] word offsets
  unsigned* woff = uw + nw;
  const int per = (nw + 1023) / 1024;                  // consecutive words per thread
  const int w0 = t * per;
  unsigned c = 0;
  for (int w = w0; w < w0 + per && w < nw; ++w) {
    unsigned u = 0;
    for (int b = 0; b < B; ++b) u |= ubits[b * nw + w];
    uw[w] = u;
    c += __popc(u);
  }
  unsigned long long tot;
  unsigned off = (unsigned)block_scan_excl<1024>((unsigned long long)c, ws, &tot);
  for (int w = w0; w < w0 + per && w < nw; ++w) { woff[w] = off; off += __popc(uw[w]); }
  __syncthreads();
  // one thread per index: members of the union write their row
  for (int id = t; id < n; id += 1024) {
    const int w = id >> 5, bit = id & 31;
    const unsigned u = uw[w];
    if ((u >> bit) & 1u) {
      const unsigned pos = woff[w] + __popc(u & ((1u << bit) - 1u));
      ulist[pos] = id;
      float v[kBT];
#pragma unroll
      for (int b = 0; b < kBT; ++b) {
        const bool in = b < B && ((ubits[b * nw + w] >> bit) & 1u);
        v[b] = !in ? 0.f : (x ? __uint_as_float(((uint32_t)x[(size_t)b * n + id]) << 16) : 1.f);
      }
      float4* dst = reinterpret_cast<float4*>(val + (size_t)pos * kBT);
      dst[0] = make_float4(v[0], v[1], v[2], v[3]);
      dst[1] = make_float4(v[4], v[5], v[6], v[7]);
    }
  }
  if (t == 0) *nu_out = (int)tot;
}

// ----------------------------------------------------------------------------
// Proxy GEMV for all tokens over the union of kept inputs.  grid = (strips of
// 512 channels, row splits).  In a block, 4 warps share a row (128 channels
// each: a lane owns one 32-bit word = 8 codes of gate or of up) and 4 warp
// groups split the rows.  Scales are applied to the unpacked code, so that the
// eight tokens' accumulators are all a lane has to keep.
// ----------------------------------------------------------------------------
constexpr int kPBThreads = 512;

template <int BITS>
__global__ void __launch_bounds__(kPBThreads)
proxy_batch_kernel(const uint8_t* __restrict__ P, const __half* __restrict__ S,
                   const int* __restrict__ ulist, const int* __restrict__ nu_ptr,
                   const float* __restrict__ xu, int B, int D, int F, int gshift,
                   float* __restrict__ part, unsigned* __restrict__ ticket, float* __restrict__ scores) {
  constexpr int CH = ProxyFmt<BITS>::CH;               // channels per 16-byte chunk
  constexpr int CW = CH / 2;                           // codes per 32-bit word: 8 (4-bit) or 4 (8-bit)
  constexpr int SW = 512 / 4;                          // words per row of a strip
  extern __shared__ float red[];                       // [4 row groups][kBT][SW*CW] partial sums
  __shared__ int s_last;
  const int strip = blockIdx.x, ks = blockIdx.y, nstrips = gridDim.x, ksplit = gridDim.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int wn = warp & 3, wk = warp >> 2;             // quarter of the strip, row group
  const int nchunks = F / CH;
  const size_t row_bytes = (size_t)nchunks * 16;
  const int word = wn * 32 + lane;                     // word inside the strip's 512-byte row segment
  const int chunk = strip * 32 + (word >> 2);
  const int wsel = word & 3;                           // 0,1 gate words; 2,3 up words
  const bool valid = chunk < nchunks;
  const int nu = *nu_ptr;
  const int r0 = (int)(((long long)nu * ks) / ksplit), r1 = (int)(((long long)nu * (ks + 1)) / ksplit);
  const int w0 = r0 + (int)(((long long)(r1 - r0) * wk) / 4), w1 = r0 + (int)(((long long)(r1 - r0) * (wk + 1)) / 4);
  float acc[kBT][CW];
#pragma unroll
  for (int b = 0; b < kBT; ++b)
#pragma unroll
    for (int c = 0; c < CW; ++c) acc[b][c] = 0.f;
  const uint8_t* src = P + (size_t)strip * 512 + (size_t)word * 4;
  const __half* sbase = S + ((size_t)chunk * 2 + (wsel >> 1)) * CH + (wsel & 1) * CW;
  constexpr int U = 4;
  int curg = -1;
  float scl[CW];
#pragma unroll
  for (int c = 0; c < CW; ++c) scl[c] = 0.f;
  for (int r = w0; r < w1; r += U) {
    int ii[U];
    uint32_t wv[U];
    float4 xa[U], xb[U];
#pragma unroll
    for (int u = 0; u < U; ++u) ii[u] = (r + u < w1) ? __ldg(ulist + r + u) : -1;
#pragma unroll
    for (int u = 0; u < U; ++u) {
      wv[u] = 0;
      xa[u] = xb[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (ii[u] >= 0) {
        if (valid) wv[u] = __ldg(reinterpret_cast<const uint32_t*>(src + (size_t)ii[u] * row_bytes));
        xa[u] = __ldg(reinterpret_cast<const float4*>(xu + (size_t)(r + u) * kBT));
        xb[u] = __ldg(reinterpret_cast<const float4*>(xu + (size_t)(r + u) * kBT) + 1);
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      if (ii[u] < 0 || !valid) continue;
      const int g = ii[u] >> gshift;
      if (g != curg) {                                 // union rows ascend: a group's scales are loaded once
        curg = g;
        const __half* sp = sbase + (size_t)g * nchunks * 2 * CH;
        uint4 sv = make_uint4(0, 0, 0, 0);
        if (CW == 8) sv = __ldg(reinterpret_cast<const uint4*>(sp));
        else { const uint2 t2 = __ldg(reinterpret_cast<const uint2*>(sp)); sv.x = t2.x; sv.y = t2.y; }
        const uint32_t sw[4] = {sv.x, sv.y, sv.z, sv.w};
#pragma unroll
        for (int c = 0; c < CW; ++c) {
          const __half2 h2 = *reinterpret_cast<const __half2*>(&sw[c >> 1]);
          scl[c] = (c & 1) ? __high2float(h2) : __low2float(h2);
        }
      }
      float q[CW];
#pragma unroll
      for (int c = 0; c < CW; ++c) {
        float code;
        if (BITS == 4) {
          const int pos = (c < 5) ? c : (c - 3);
          const uint32_t s = (c < 5) ? wv[u] : (wv[u] >> 12);
          code = __uint_as_float((s & (0xFu << (4 * pos))) | ((uint32_t)(150 - 4 * pos) << 23)) -
                 ((float)(1u << (23 - 4 * pos)) + 8.0f);
        } else {
          code = __uint_as_float(__byte_perm(wv[u], 0x4B000000u, 0x7650u | c)) - 8388736.0f;
        }
        q[c] = code * scl[c];
      }
      const float xt[kBT] = {xa[u].x, xa[u].y, xa[u].z, xa[u].w, xb[u].x, xb[u].y, xb[u].z, xb[u].w};
#pragma unroll
      for (int b = 0; b < kBT; ++b)
#pragma unroll
        for (int c = 0; c < CW; ++c) acc[b][c] = fmaf(q[c], xt[b], acc[b][c]);
    }
  }
  // meet: red[wk][b][word*CW + c]
  constexpr int NVAL = SW * CW;                        // values per token per strip (1024 / 512)
#pragma unroll
  for (int b = 0; b < kBT; ++b)
#pragma unroll
    for (int c = 0; c < CW; ++c) red[((size_t)wk * kBT + b) * NVAL + c * SW + word] = acc[b][c];
  __syncthreads();
  // element e = c*SW + word  ->  chunk-local channel: word>>2 chunk, (word&1)*CW + c within gate/up half
  float* pb = part + ((size_t)ks * nstrips + strip) * (size_t)(kBT * NVAL);
  for (int e = threadIdx.x; e < B * NVAL; e += kPBThreads) {
    const float s = red[e] + red[(size_t)kBT * NVAL + e] + red[(size_t)2 * kBT * NVAL + e] + red[(size_t)3 * kBT * NVAL + e];
    if (ksplit > 1) __stcg(pb + e, s); else red[e] = s;
  }
  __syncthreads();
  if (ksplit > 1) {
    if (threadIdx.x == 0) {
      __threadfence();
      const unsigned tk = atomicAdd(&ticket[strip], 1u);
      s_last = (tk == (unsigned)(ksplit - 1));
      __threadfence();
    }
    __syncthreads();
    if (!s_last) return;
    for (int e = threadIdx.x; e < B * NVAL; e += kPBThreads) {
      float s = 0.f;
      for (int z = 0; z < ksplit; ++z) s += __ldcg(part + ((size_t)z * nstrips + strip) * (size_t)(kBT * NVAL) + e);
      red[e] = s;
    }
    if (threadIdx.x == 0) ticket[strip] = 0;
    __syncthreads();
  }
  // scores: channel ch = chunk*CH + half*CW + c ; gate value at word (chunk*4 + half), up at word (chunk*4 + 2 + half)
  for (int e = threadIdx.x; e < B * 32 * CH; e += kPBThreads) {
    const int b = e / (32 * CH), j = e % (32 * CH);     // j: channel inside the strip
    const int cl = j / CH, cc = j % CH;                 // chunk inside the strip, channel inside the chunk
    const int half = cc / CW, c = cc % CW;
    const int ch = (strip * 32 + cl) * CH + cc;
    if (ch < F) {
      const float g = red[(size_t)b * NVAL + c * SW + (cl * 4 + half)];
      const float u = red[(size_t)b * NVAL + c * SW + (cl * 4 + 2 + half)];
      scores[(size_t)b * F + ch] = fabsf(u * silu_fast(g));
    }
  }
}

// ----------------------------------------------------------------------------
// Stage 2a for all tokens over the union of kept channels: one warp per union
// channel; x of every token sits in shared memory as bf16.  h[r][b] is written
// already multiplied by the token's membership (0 for a token that did not
// select the channel).
// ----------------------------------------------------------------------------
constexpr int kGBThreads = 256;

__global__ void __launch_bounds__(kGBThreads)
gateup_batch_kernel(const uint16_t* __restrict__ wg, const uint16_t* __restrict__ wu,
                    const uint16_t* __restrict__ x, int B, const int* __restrict__ ulist,
                    const int* __restrict__ nu_ptr, const float* __restrict__ member, int D, int F,
                    float* __restrict__ h_out) {
  extern __shared__ uint4 xs4[];                       // [B][D] bf16
  const int nu = *nu_ptr;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  constexpr int WPB = kGBThreads / 32;
  if ((int)blockIdx.x * WPB >= nu) return;
  const int nv = D / 8;
  const uint4* xg = reinterpret_cast<const uint4*>(x);
  for (int i = threadIdx.x; i < B * nv; i += kGBThreads) xs4[i] = __ldg(xg + i);
  __syncthreads();
  for (int r = blockIdx.x * WPB + warp; r < nu; r += gridDim.x * WPB) {
    const int j = ulist[r];
    const uint4* g4 = reinterpret_cast<const uint4*>(wg + (size_t)j * D);
    const uint4* u4 = reinterpret_cast<const uint4*>(wu + (size_t)j * D);
    float ag[kBT], au[kBT];
#pragma unroll
    for (int b = 0; b < kBT; ++b) { ag[b] = 0.f; au[b] = 0.f; }
    for (int i = lane; i < nv; i += 32) {
      const uint4 a = ld_stream(g4 + i), c = ld_stream(u4 + i);
      const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, cw[4] = {c.x, c.y, c.z, c.w};
      float af[8], cf[8];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        af[2 * q] = bf16_lo(aw[q]); af[2 * q + 1] = bf16_hi(aw[q]);
        cf[2 * q] = bf16_lo(cw[q]); cf[2 * q + 1] = bf16_hi(cw[q]);
      }
#pragma unroll
      for (int b = 0; b < kBT; ++b) {
        if (b < B) {
          const uint4 xv = xs4[b * nv + i];
          const uint32_t xw[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const float x0 = bf16_lo(xw[q]), x1 = bf16_hi(xw[q]);
            ag[b] = fmaf(af[2 * q], x0, ag[b]); ag[b] = fmaf(af[2 * q + 1], x1, ag[b]);
            au[b] = fmaf(cf[2 * q], x0, au[b]); au[b] = fmaf(cf[2 * q + 1], x1, au[b]);
          }
        }
      }
    }
#pragma unroll
    for (int b = 0; b < kBT; ++b) { ag[b] = warp_sum(ag[b]); au[b] = warp_sum(au[b]); }
    if (lane < kBT) {
      float g = 0.f, u = 0.f;
#pragma unroll
      for (int b = 0; b < kBT; ++b) if (lane == b) { g = ag[b]; u = au[b]; }
      const float m = member[(size_t)r * kBT + lane];
      h_out[(size_t)r * kBT + lane] = (lane < B && m != 0.f) ? u * silu_exact(g) : 0.f;
    }
  }
}

// ----------------------------------------------------------------------------
// Stage 2b for all tokens: y[b] = sum over union rows of h[r][b] * W_downT[j_r,:].
// grid = (D tiles of 2048 outputs, row splits); a thread owns 8 outputs of
// every token.
// ----------------------------------------------------------------------------
__global__ void __launch_bounds__(kDownThreads)
down_batch_kernel(const uint16_t* __restrict__ wdt, const float* __restrict__ h,
                  const int* __restrict__ ulist, const int* __restrict__ nu_ptr, int B, int D,
                  float* __restrict__ yacc) {
  __shared__ float hs[64][kBT];
  __shared__ int js[64];
  const int nu = *nu_ptr;
  const int nsplit = gridDim.y, sp = blockIdx.y;
  const int c0 = (int)(((long long)nu * sp) / nsplit), c1 = (int)(((long long)nu * (sp + 1)) / nsplit);
  const int e = (blockIdx.x * kDownThreads + threadIdx.x) * 8;
  float acc[kBT][8];
#pragma unroll
  for (int b = 0; b < kBT; ++b)
#pragma unroll
    for (int m = 0; m < 8; ++m) acc[b][m] = 0.f;
  for (int cb = c0; cb < c1; cb += 64) {
    const int cn = min(64, c1 - cb);
    __syncthreads();
    for (int i = threadIdx.x; i < cn * kBT; i += kDownThreads) hs[i / kBT][i % kBT] = h[(size_t)(cb + i / kBT) * kBT + i % kBT];
    for (int i = threadIdx.x; i < cn; i += kDownThreads) js[i] = ulist[cb + i];
    __syncthreads();
    if (e < D) {
      constexpr int UN = 4;
      for (int i0 = 0; i0 < cn; i0 += UN) {
        uint4 w[UN];
#pragma unroll
        for (int u = 0; u < UN; ++u)
          if (i0 + u < cn) w[u] = ld_stream(wdt + (size_t)js[i0 + u] * D + e);
#pragma unroll
        for (int u = 0; u < UN; ++u) {
          if (i0 + u < cn) {
            const uint32_t ww[4] = {w[u].x, w[u].y, w[u].z, w[u].w};
            float wf[8];
#pragma unroll
            for (int q = 0; q < 4; ++q) { wf[2 * q] = bf16_lo(ww[q]); wf[2 * q + 1] = bf16_hi(ww[q]); }
#pragma unroll
            for (int b = 0; b < kBT; ++b) {
              const float hv = hs[i0 + u][b];
#pragma unroll
              for (int m = 0; m < 8; ++m) acc[b][m] = fmaf(hv, wf[m], acc[b][m]);
            }
          }
        }
      }
    }
  }
  if (e < D && c1 > c0) {
#pragma unroll
    for (int b = 0; b < kBT; ++b) {
      if (b < B) {
        float4* yp = reinterpret_cast<float4*>(yacc + (size_t)b * D + e);
        atomicAdd(yp, make_float4(acc[b][0], acc[b][1], acc[b][2], acc[b][3]));
        atomicAdd(yp + 1, make_float4(acc[b][4], acc[b][5], acc[b][6], acc[b][7]));
      }
    }
  }
}

}  // namespace prox
