// Batch B > 1, Stage 2 on the tensor cores (Sec. 4.1 Stage 2 for several
// tokens at once; the paper treats batch 1 only).  With up to eight tokens the
// union rows of W_gate / W_up / W_downT form real 16 x 8 x 16 tiles, so the
// exact products move to warp-level bf16 MMAs with fp32 accumulation; the
// kernels stay bound by the weight stream.
//
// Work is cut into units of a few KB of weights and every block takes a
// contiguous, equal range of units, whatever the union size: partial results
// of a tile meet in an fp32 accumulator in global memory (vector-free atomics,
// a few hundred per block).
//
// Fragment layout of mma.sync.m16n8k16 (g = lane / 4, t = lane % 4):
//   A (16 x 16, row): a0a1 = (row g, k 2t..2t+1)  a2a3 = (row g+8, same k)
//                     a4a5 = (row g, k 2t+8..+9)  a6a7 = (row g+8, k 2t+8..+9)
//   B (16 x 8, col):  b0b1 = (k 2t..2t+1, col g)  b2b3 = (k 2t+8..+9, col g)
//   C (16 x 8):       c0c1 = (row g, col 2t..2t+1)  c2c3 = (row g+8, same cols)
// A sum over k does not care which physical k sits at which logical k as long as
// A and B agree, so a lane loads 16 contiguous bytes (8 physical k) and feeds
// them to two MMAs: physical k 8t+{0,1 | 2,3} and 8t+{4,5 | 6,7}.
#pragma once

#include "prox_batch.cuh"

namespace prox {

__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

constexpr int kMmaThreads = 512;
constexpr int kMmaWarps = kMmaThreads / 32;
constexpr int kXPad = 64;               // bytes added to a token's row of x in shared memory (bank spread)

// ----------------------------------------------------------------------------
// Stage 2a: gate and up pre-activations of every union channel for all tokens.
// Unit = (tile of 16 union channels, 32 inputs).  A = weight rows (M = channel),
// B = x (N = token).  Results are added to gacc[union row][gate|up][token].
// ----------------------------------------------------------------------------
__global__ void __launch_bounds__(kMmaThreads, 2)
gateup_mma_kernel(const uint16_t* __restrict__ wg, const uint16_t* __restrict__ wu,
                  const uint16_t* __restrict__ x, int B, const int* __restrict__ ulist,
                  const int* __restrict__ nu_ptr, int D, float* __restrict__ gacc) {
  extern __shared__ __align__(16) uint8_t mm_smem[];
  const int pitch = D * 2 + kXPad;
  uint8_t* xs = mm_smem;                                        // [8][pitch] bf16 rows of x (zero beyond B)
  float* red = reinterpret_cast<float*>(mm_smem + (size_t)8 * pitch);   // [warps][256]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const int nu = *nu_ptr;
  if (nu <= 0) return;
  for (int i = tid; i < 8 * (D / 8); i += kMmaThreads) {
    const int b = i / (D / 8), v = i % (D / 8);
    uint4 val = make_uint4(0, 0, 0, 0);
    if (b < B) val = __ldg(reinterpret_cast<const uint4*>(x + (size_t)b * D) + v);
    *reinterpret_cast<uint4*>(xs + (size_t)b * pitch + (size_t)v * 16) = val;
  }
  __syncthreads();
  const int nkb = D / 32, ntile = (nu + 15) / 16;
  const long long total = (long long)ntile * nkb;
  long long u = total * blockIdx.x / gridDim.x;
  const long long u1 = total * (blockIdx.x + 1) / gridDim.x;
  const uint8_t* xrow = xs + (size_t)g * pitch + (size_t)t * 16;
  while (u < u1) {
    const int tile = (int)(u / nkb), a = (int)(u - (long long)tile * nkb);
    const int b = (int)min((long long)nkb, a + (u1 - u));
    const int rlo = ulist[min(tile * 16 + g, nu - 1)], rhi = ulist[min(tile * 16 + g + 8, nu - 1)];
    const uint16_t* pgl = wg + (size_t)rlo * D + t * 8;
    const uint16_t* pgh = wg + (size_t)rhi * D + t * 8;
    const uint16_t* pul = wu + (size_t)rlo * D + t * 8;
    const uint16_t* puh = wu + (size_t)rhi * D + t * 8;
    float ag[4] = {0.f, 0.f, 0.f, 0.f}, au[4] = {0.f, 0.f, 0.f, 0.f};
    for (int kb = a + 2 * warp; kb < b; kb += 2 * kMmaWarps) {   // two neighbouring units: whole 128-byte lines per row
      const int kb2 = kb + 1;
      const bool two = kb2 < b;
      const int kc = two ? kb2 : kb;                            // a valid address for the second set of loads
      const uint4 gl0 = ld_stream(pgl + kb * 32), gh0 = ld_stream(pgh + kb * 32);
      const uint4 ul0 = ld_stream(pul + kb * 32), uh0 = ld_stream(puh + kb * 32);
      const uint4 gl1 = ld_stream(pgl + kc * 32), gh1 = ld_stream(pgh + kc * 32);
      const uint4 ul1 = ld_stream(pul + kc * 32), uh1 = ld_stream(puh + kc * 32);
      const uint4 x0 = *reinterpret_cast<const uint4*>(xrow + (size_t)kb * 64);
      const uint4 x1 = *reinterpret_cast<const uint4*>(xrow + (size_t)kc * 64);
      mma_bf16(ag, gl0.x, gh0.x, gl0.y, gh0.y, x0.x, x0.y);
      mma_bf16(ag, gl0.z, gh0.z, gl0.w, gh0.w, x0.z, x0.w);
      mma_bf16(au, ul0.x, uh0.x, ul0.y, uh0.y, x0.x, x0.y);
      mma_bf16(au, ul0.z, uh0.z, ul0.w, uh0.w, x0.z, x0.w);
      if (two) {
        mma_bf16(ag, gl1.x, gh1.x, gl1.y, gh1.y, x1.x, x1.y);
        mma_bf16(ag, gl1.z, gh1.z, gl1.w, gh1.w, x1.z, x1.w);
        mma_bf16(au, ul1.x, uh1.x, ul1.y, uh1.y, x1.x, x1.y);
        mma_bf16(au, ul1.z, uh1.z, ul1.w, uh1.w, x1.z, x1.w);
      }
    }
    // the warps' partial tiles meet in shared memory: index = row * 16 + (gate 0 | up 8) + token
    float* mine = red + warp * 256;
    mine[g * 16 + 2 * t] = ag[0]; mine[g * 16 + 2 * t + 1] = ag[1];
    mine[(g + 8) * 16 + 2 * t] = ag[2]; mine[(g + 8) * 16 + 2 * t + 1] = ag[3];
    mine[g * 16 + 8 + 2 * t] = au[0]; mine[g * 16 + 8 + 2 * t + 1] = au[1];
    mine[(g + 8) * 16 + 8 + 2 * t] = au[2]; mine[(g + 8) * 16 + 8 + 2 * t + 1] = au[3];
    __syncthreads();
    if (tid < 256) {
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < kMmaWarps; ++w) s += red[w * 256 + tid];
      if (tile * 16 + (tid >> 4) < nu) atomicAdd(gacc + (size_t)tile * 256 + tid, s);
    }
    __syncthreads();
    u += b - a;
  }
}

// h[r][b] = SiLU(gate) * up for the tokens that kept channel r, 0 for the others;
// the accumulator is cleared for the next call.
__global__ void __launch_bounds__(256)
gateup_finish_kernel(float* __restrict__ gacc, const float* __restrict__ member, const int* __restrict__ nu_ptr,
                     int B, float* __restrict__ h_out) {
  const int nu = *nu_ptr;
  for (int i = blockIdx.x * 256 + threadIdx.x; i < nu * kBT; i += gridDim.x * 256) {
    const int r = i / kBT, b = i % kBT;
    const float gate = gacc[(size_t)r * 16 + b], up = gacc[(size_t)r * 16 + 8 + b];
    gacc[(size_t)r * 16 + b] = 0.f; gacc[(size_t)r * 16 + 8 + b] = 0.f;
    h_out[i] = (b < B && member[i] != 0.f) ? up * silu_exact(gate) : 0.f;
  }
}

// ----------------------------------------------------------------------------
// Stage 2b: y[b] += sum over union rows of h[r][b] * W_downT[j_r, :].
// Unit = (64 output columns, 16 union rows).  A = h (M = token, rows 8..15 are
// zero), B = W_downT rows (K = union row, N = output column).  A K-pair of B
// comes from two different rows of W_downT: one byte permute per register.
// h is fed as a bf16 pair hi + lo (two MMAs), which keeps ~16 bits of it.
// A lane loads columns 8g..8g+7, so MMA number i of a unit covers the columns
// {8c + i}: accumulator (i, c0) is column 8 * 2t + i, (i, c1) column 8 * (2t+1) + i.
// ----------------------------------------------------------------------------
__global__ void __launch_bounds__(kMmaThreads, 1)
down_mma_kernel(const uint16_t* __restrict__ wdt, const float* __restrict__ h, const int* __restrict__ ulist,
                const int* __restrict__ nu_ptr, int B, int D, float* __restrict__ yacc) {
  extern __shared__ __align__(16) uint8_t mm_smem[];
  float* red = reinterpret_cast<float*>(mm_smem);               // [warps][8 tokens][64 columns]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const int nu = *nu_ptr;
  if (nu <= 0) return;
  const int nkb = (nu + 15) / 16, ncol = D / 64;
  const long long total = (long long)ncol * nkb;
  long long u = total * blockIdx.x / gridDim.x;
  const long long u1 = total * (blockIdx.x + 1) / gridDim.x;
  while (u < u1) {
    const int ct = (int)(u / nkb), a = (int)(u - (long long)ct * nkb);
    const int b = (int)min((long long)nkb, a + (u1 - u));
    float acc[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    const uint16_t* colp = wdt + (size_t)ct * 64 + g * 8;
    auto load_unit = [&](int kb, uint4 (&w)[4], float (&hv)[4]) {
      const int c0 = kb * 16 + 2 * t;
      const int cr[4] = {c0, c0 + 1, c0 + 8, c0 + 9};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int c = min(cr[q], nu - 1);
        w[q] = ld_stream(colp + (size_t)ulist[c] * D);
        hv[q] = (cr[q] < nu) ? __ldg(h + (size_t)c * kBT + g) : 0.f;
      }
    };
    auto mma_unit = [&](const uint4 (&w)[4], const float (&hv)[4]) {
      uint32_t ahi[2], alo[2];
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const __nv_bfloat16 h0 = __float2bfloat16_rn(hv[2 * q]), h1 = __float2bfloat16_rn(hv[2 * q + 1]);
        const __nv_bfloat16 l0 = __float2bfloat16_rn(hv[2 * q] - __bfloat162float(h0));
        const __nv_bfloat16 l1 = __float2bfloat16_rn(hv[2 * q + 1] - __bfloat162float(h1));
        ahi[q] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
        alo[q] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
      }
      const uint32_t w0[4] = {w[0].x, w[0].y, w[0].z, w[0].w}, w1[4] = {w[1].x, w[1].y, w[1].z, w[1].w};
      const uint32_t w2[4] = {w[2].x, w[2].y, w[2].z, w[2].w}, w3[4] = {w[3].x, w[3].y, w[3].z, w[3].w};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint32_t be0 = __byte_perm(w0[q], w1[q], 0x5410), be1 = __byte_perm(w2[q], w3[q], 0x5410);
        const uint32_t bo0 = __byte_perm(w0[q], w1[q], 0x7632), bo1 = __byte_perm(w2[q], w3[q], 0x7632);
        mma_bf16(acc[2 * q], ahi[0], 0u, ahi[1], 0u, be0, be1);
        mma_bf16(acc[2 * q], alo[0], 0u, alo[1], 0u, be0, be1);
        mma_bf16(acc[2 * q + 1], ahi[0], 0u, ahi[1], 0u, bo0, bo1);
        mma_bf16(acc[2 * q + 1], alo[0], 0u, alo[1], 0u, bo0, bo1);
      }
    };
    for (int kb = a + warp; kb < b; kb += 2 * kMmaWarps) {      // two units in flight per warp
      uint4 wa[4], wb[4];
      float ha[4], hb[4];
      const bool two = kb + kMmaWarps < b;
      load_unit(kb, wa, ha);
      if (two) load_unit(kb + kMmaWarps, wb, hb);
      mma_unit(wa, ha);
      if (two) mma_unit(wb, hb);
    }
    float* mine = red + warp * 512 + g * 64;                    // token g
#pragma unroll
    for (int i = 0; i < 8; ++i) { mine[8 * (2 * t) + i] = acc[i][0]; mine[8 * (2 * t + 1) + i] = acc[i][1]; }
    __syncthreads();
    {
      float s = 0.f;
#pragma unroll
      for (int w2i = 0; w2i < kMmaWarps; ++w2i) s += red[w2i * 512 + tid];
      const int tok = tid >> 6, col = tid & 63;
      if (tok < B) atomicAdd(yacc + (size_t)tok * D + (size_t)ct * 64 + col, s);
    }
    __syncthreads();
    u += b - a;
  }
}

}  // namespace prox
