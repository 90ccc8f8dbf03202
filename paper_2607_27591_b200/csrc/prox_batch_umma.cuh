// Stage 1 for B > 1 on the tcgen05 tensor cores (integer proxies, 4 or 8 bits).
//
// Same formulation as the batch-1 kernel (Sec. 4.1 proxy equations): the packed proxy rows are the u8 A
// operand of an integer MMA as they lie in memory (MN-major, 128-byte swizzle, 128 bytes of 32 rows per
// stage), the inputs enter as signed base-256 digits of an integer form of x.  With up to eight tokens
// the kept inputs of the tokens cover nearly every row, so the GEMM runs over ALL rows (a dropped input
// is a zero digit word) and a block of 32 rows never straddles a 128-input scale group.
//
// Data movement: one producer lane keeps a ring of stages full with TMA: per unit of 128 inputs one tiled
// tensor copy drops the 128 x 128-byte tile of the proxy rows into shared memory already in the swizzled
// operand layout (four blocks of 32 rows), a bulk copy brings the unit's digit rows (stored in operand layout
// by batch_digits_kernel).  For 8-bit codes
// nothing else touches the bytes: a worker warp waits for the stage and issues the MMA.  For 4-bit
// codes the worker first writes the tile with the high nibbles masked off into a second buffer (the
// operand of the second MMA).  B operand of a block: row k = 8 tokens x 4 digits = 32 bytes (N = 32).
// A unit = 128 consecutive inputs (4 blocks): its MMAs accumulate into one of four 64-column sets of
// tensor memory (32 columns for the bytes, 32 for the low nibbles; a unit's first MMA overwrites them); two groups
// of eight read-back warps take turns on the units and apply their scales while the workers already fill
// the other sets.  Items = (128-byte tile of the rows, range of units); an item's partial sums are added to an fp32 accumulator in global memory, a small kernel forms
// the scores.
#pragma once

#include <cuda.h>

#include "prox_batch_mma.cuh"

namespace prox {

constexpr int kBuWorkers = 8;                        // warps 1..8: (mask the low nibbles,) issue the MMAs
constexpr int kBuRb = 16;                            // warps 9..24: read the accumulators back (eight per accumulator set)
constexpr int kBuThreads = (1 + kBuWorkers + kBuRb) * 32;
constexpr int kBuStages4 = 8, kBuStages8 = 10;       // stage = one unit (four blocks); even: a stage always meets the same workers
constexpr int kBuStagesMax = 10;                     // (8-bit codes need no low-nibble buffers: two stages more)
constexpr int kBuTile = 4096, kBuDig = 1024;         // block: 32 rows x 128 bytes | 32 rows x 32 digit bytes
constexpr int kBuSmem4 = 1024 + kBuStages4 * 4 * (kBuTile + kBuDig) + kBuWorkers * kBuTile;
constexpr int kBuSmem8 = 1024 + kBuStages8 * 4 * (kBuTile + kBuDig);

__device__ __forceinline__ void sts128(uint32_t a, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
// tile of a 2-D tensor map (x = byte column, a multiple of 16; y = row) into shared memory
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

// Integer form of a token's masked, scaled fp16 input: X = x_h * 2^16 (|X| < 2^30), as four signed
// base-256 digits; x_h = x * 2^se is what batch_input_mask_kernel writes (max |x_h| in [2^13, 2^14)).
// xd = the digit words in the layout of the MMA's B operand, 1 KB per block of 32 inputs: two planes of
// 32 rows x 16 bytes (tokens 0..3 | tokens 4..7), row = input, 4 bytes per token.
// soff[u][b] = sum of X over the 128 inputs of unit u (as float).  One block per token slot.
__global__ void __launch_bounds__(512)
batch_digits_kernel(const __half* __restrict__ xh, int D, uint32_t* __restrict__ xd, float* __restrict__ soff) {
  __shared__ int sd[128 * 4];
  const int b = blockIdx.x, tid = threadIdx.x;
  const int ng = D >> 7;                              // units of 128 inputs (d_model <= 16384)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the proxy GEMM may set up and start on the weights
  sd[tid] = 0;
  __syncthreads();
  const __half* row = xh + (size_t)b * D;
  for (int i0 = tid * 8; i0 < D; i0 += 512 * 8) {
    const uint4 v = *reinterpret_cast<const uint4*>(row + i0);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    int d0 = 0, d1 = 0, d2 = 0, d3 = 0;
    uint32_t* dst = xd + (size_t)(i0 >> 5) * 256 + (b >> 2) * 128 + (i0 & 31) * 4 + (b & 3);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const __half hv = __ushort_as_half((unsigned short)((w[e >> 1] >> ((e & 1) * 16)) & 0xffffu));
      const int X = __float2int_rn(__half2float(hv) * 65536.f);
      const uint32_t dg = ((uint32_t)X + 0x00808080u) ^ 0x00808080u;
      dst[e * 4] = dg;
      d0 += (int)(int8_t)(dg & 0xffu); d1 += (int)(int8_t)((dg >> 8) & 0xffu);
      d2 += (int)(int8_t)((dg >> 16) & 0xffu); d3 += (int)(int8_t)(dg >> 24);
    }
    int* sdg = sd + 4 * (i0 >> 7);
    if (d0) atomicAdd(sdg, d0);
    if (d1) atomicAdd(sdg + 1, d1);
    if (d2) atomicAdd(sdg + 2, d2);
    if (d3) atomicAdd(sdg + 3, d3);
  }
  __syncthreads();
  if (tid < ng)
    soff[(size_t)tid * kBT + b] = digits_to_float((uint32_t)sd[tid * 4], (uint32_t)sd[tid * 4 + 1], (uint32_t)sd[tid * 4 + 2],
                                                  (uint32_t)sd[tid * 4 + 3]);
}

// sum_d digit_d 256^d of int32 digit sums (|digit sum| < 2^22: 128 rows x 255 x 128), two integer pairs
__device__ __forceinline__ float digits4_to_float(int d0, int d1, int d2, int d3) {
  return fmaf((float)(d2 + d3 * 256), 65536.f, (float)(d0 + d1 * 256));
}

// pacc[(token * 2 + which) * F + channel] += partial proxy sums (gate: which = 0, up: 1), already scaled.
// pmap: the packed proxy as a 2-D byte tensor [D rows][row bytes], box 128 bytes x 128 rows, 128-byte swizzle.
template <int BITS>
__global__ void __launch_bounds__(kBuThreads, 1)
proxy_umma_kernel(const __grid_constant__ CUtensorMap pmap, const __half* __restrict__ S, const uint32_t* __restrict__ xd,
                  const float* __restrict__ soff, const float* __restrict__ tokfac, int D, int F, int gshift, int usplit,
                  float* __restrict__ pacc, int* __restrict__ status) {
  constexpr bool LO = BITS == 4;
  constexpr int CH = LO ? 16 : 8;
  constexpr int kBuStages = LO ? kBuStages4 : kBuStages8;
  extern __shared__ __align__(128) uint8_t bu_smem[];
  __shared__ unsigned long long full[kBuStagesMax], empty[kBuStagesMax], gdone[4];
  __shared__ unsigned drained[kBuRb];                 // per read-back warp: units it has read back and cleared
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool per_row = gshift >= 31;
  const int nchunks = F / CH, row_bytes = nchunks * 16, ntiles = (row_bytes + 127) >> 7;
  const int nunits = D >> 7;                          // units of 128 inputs
  const uint32_t raw0 = (smem_u32(bu_smem) + 1023u) & ~1023u;           // [stages][4][4096] tiles as TMA writes them
  const uint32_t lo0 = raw0 + (uint32_t)(kBuStages * 4 * kBuTile);      // [workers][4096] low-nibble copies
  const uint32_t dig0 = lo0 + (uint32_t)(LO ? kBuWorkers * kBuTile : 0);         // [stages][4][1024] digit rows
  volatile int* abortp = &abort_flag;
  if (tid == 32) asm volatile("prefetch.tensormap [%0];" ::"l"(&pmap) : "memory");
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid < kBuStages) { mbar_init(smem_u32(&full[tid]), 1); mbar_init(smem_u32(&empty[tid]), 1); }
  if (tid < 4) mbar_init(smem_u32(&gdone[tid]), 1);
  if (tid < kBuRb) drained[tid] = 0u;
  if (tid == 0) abort_flag = 0;
  fence_mbar_init();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tbase = tmem_base_s;
  const int rb = warp - 1 - kBuWorkers;               // read-back warp: set rb / 8, tokens 4 * (rb / 4 % 2) .., lanes 32 * (warp % 4) ..
  const int nitems = ntiles * usplit;
  if (tid != 0) asm volatile("griddepcontrol.wait;" ::: "memory");   // thread 0 (the producer) first requests weights
  unsigned gseq = 0;                                  // units this CTA has started (unit number modulo 4 = accumulator set)
  if (warp == 0) {
    // ---- producer: one lane keeps the ring full
    if (lane == 0) {
      // the proxy rows are weights: the first ring-full of tiles is requested before the kernels that
      // produce this call's digits have finished (programmatic dependent launch); the digits follow
      bool early = true;
      int first_u0 = 0;
#pragma unroll 1
      for (int item = blockIdx.x; item < nitems && !*abortp; item += gridDim.x) {
        const int tile = item % ntiles, part = item / ntiles;
        const int u0 = (int)(((long long)nunits * part) / usplit), u1 = (int)(((long long)nunits * (part + 1)) / usplit);
        if (item == (int)blockIdx.x) first_u0 = u0;
#pragma unroll 1
        for (int u = u0; u < u1; ++u, ++gseq) {
          const unsigned s = gseq % kBuStages, use = gseq / kBuStages;
          if (early && (use > 0 || item != (int)blockIdx.x)) {
            // the ring is full (or the first item has ended): now the digits of what was requested
            asm volatile("griddepcontrol.wait;" ::: "memory");
            for (unsigned k = 0; k < gseq; ++k)
              bulk_g2s(dig0 + k * (uint32_t)(4 * kBuDig), xd + (size_t)(first_u0 + (int)k) * 1024, (uint32_t)(4 * kBuDig),
                       smem_u32(&full[k]));
            early = false;
          }
          if (use > 0 && !mbar_wait(smem_u32(&empty[s]), (use - 1u) & 1u, abortp)) break;
          const uint32_t fb = smem_u32(&full[s]);
          mbar_expect_tx(fb, (uint32_t)(4 * (kBuTile + kBuDig)));
          tma_load_2d(raw0 + s * (uint32_t)(4 * kBuTile), &pmap, tile * 128, u << 7, fb);
          if (!early) bulk_g2s(dig0 + s * (uint32_t)(4 * kBuDig), xd + (size_t)u * 1024, (uint32_t)(4 * kBuDig), fb);
        }
      }
      if (early) {                                    // fewer units than stages in all: nothing of the digits requested yet
        asm volatile("griddepcontrol.wait;" ::: "memory");
        for (unsigned k = 0; k < gseq; ++k)
          bulk_g2s(dig0 + k * (uint32_t)(4 * kBuDig), xd + (size_t)(first_u0 + (int)k) * 1024, (uint32_t)(4 * kBuDig), smem_u32(&full[k]));
      }
      if (*abortp) {                                  // no copy may be in flight when the block ends
#pragma unroll 1
        for (unsigned s = 0; s < (unsigned)kBuStages; ++s) {
          const unsigned armed = (gseq + (unsigned)kBuStages - 1u - s) / (unsigned)kBuStages;
          if (armed == 0) continue;
#pragma unroll 1
          for (unsigned it = 0; it < 65536u; ++it) {
            if (mbar_try_wait(smem_u32(&full[s]), (armed - 1u) & 1u)) break;
            __nanosleep(64);
          }
        }
      }
    }
  } else if (rb < 0) {
    // ---- workers: group w / 4 owns the units with number gs % 2 == w / 4 (accumulator sets gs % 4).  4-bit codes:
    // each warp of the group writes the low nibbles of one block of the unit, then the group's first warp
    // issues the unit's MMAs, the first of them overwriting the accumulators.  8-bit codes: only that warp works.
    const int w = warp - 1, wj = w & 3, grp = w >> 2;
    const uint32_t lob = lo0 + (uint32_t)w * (uint32_t)kBuTile;
    const uint32_t lo_group = lo0 + (uint32_t)(grp * 4) * (uint32_t)kBuTile;
    constexpr uint32_t idesc = umma_idesc_u8s8(128, 32);
    unsigned mine = 0, s_prev = 0, use_prev = 0;
    bool bad = false;                                 // a wait of this warp gave up; the group leaves together
    if (LO || wj == 0) {
#pragma unroll 1
      for (int item = blockIdx.x; item < nitems; item += gridDim.x) {
        const int part = item / ntiles;
        const int u0 = (int)(((long long)nunits * part) / usplit), u1 = (int)(((long long)nunits * (part + 1)) / usplit);
        bool dead = false;
#pragma unroll 1
        for (int ul = (int)(((unsigned)grp + gseq) & 1u); ul < u1 - u0; ul += 2) {
          const unsigned gs = gseq + (unsigned)ul, s = gs % kBuStages, use = gs / kBuStages;
          const int set = (int)(gs & 3u);              // four accumulator sets: a group alternates between two of them
          const uint32_t raws = raw0 + s * (uint32_t)(4 * kBuTile);
          bad = bad || !__all_sync(0xffffffffu, mbar_wait(smem_u32(&full[s]), use & 1u, abortp));
          if (LO) {
            // the low-nibble buffers are free once the MMAs of the group's previous unit are done
            if (mine > 0) bad = bad || !__all_sync(0xffffffffu, mbar_wait(smem_u32(&empty[s_prev]), use_prev & 1u, abortp));
            if (!bad) {
              const uint32_t rawb = raws + (uint32_t)(wj * kBuTile);
              uint4 v[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) v[j] = lds128(rawb + (uint32_t)(j * 512 + lane * 16));
#pragma unroll
              for (int j = 0; j < 8; ++j)
                sts128(lob + (uint32_t)(j * 512 + lane * 16), v[j].x & 0x0f0f0f0fu, v[j].y & 0x0f0f0f0fu, v[j].z & 0x0f0f0f0fu,
                       v[j].w & 0x0f0f0f0fu);
              fence_proxy_async();
            }
            uint32_t any_bad;                         // barrier of the group's 128 threads that also ORs the flags
            asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.or.pred p, %2, 128, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(any_bad) : "r"((uint32_t)bad), "r"(2 + grp) : "memory");
            if (any_bad) { dead = true; break; }
          } else if (bad) { dead = true; break; }
          ++mine; s_prev = s; use_prev = use;
          if (wj != 0) continue;
          // the set must have been read back by its read-back warps: counters, not an mbarrier phase; lanes 0..7
          // each watch one read-back warp of the set
          bool set_ok = true;
          if (gs >= 4u) {
            set_ok = false;
#pragma unroll 1
            for (unsigned it = 0; it < kSpinLimit; ++it) {
              unsigned seen = gs;
              if (lane < 8) asm volatile("ld.acquire.cta.shared.u32 %0, [%1];" : "=r"(seen) : "r"(smem_u32(&drained[grp * 8 + lane])) : "memory");
              if (__all_sync(0xffffffffu, (int)(seen - (gs - 3u)) >= 0)) { set_ok = true; break; }   // unit gs - 4 read back
              __nanosleep(20);
              if ((it & 255u) == 255u && *abortp) break;
            }
            if (!set_ok) *abortp = 1;
          }
          if (!set_ok) { bad = true; if (!LO) { dead = true; break; } continue; }   // 4-bit: leave at the group's next barrier
          tc_fence_after();
          // descriptors by the whole warp (a lone thread computing them costs more than the MMAs): block j of
          // the unit is 4 KB (rows), 1 KB (digits) further on, i.e. 256 / 64 in descriptor address units
          const uint64_t adesc = umma_smem_desc(raws, 4096u, 1024u, 2u);
          const uint64_t ldesc = umma_smem_desc(lo_group, 4096u, 1024u, 2u);
          const uint64_t bdesc = umma_smem_desc(dig0 + s * (uint32_t)(4 * kBuDig), 128u, 512u, 0u);
          const uint32_t dall = tbase + (uint32_t)(set * 64), dlo = dall + 32u;
          if (elect_one()) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              umma_i8(dall, adesc + (uint64_t)(j * 256), bdesc + (uint64_t)(j * 64), idesc, j > 0 ? 1u : 0u);
              if (LO) umma_i8(dlo, ldesc + (uint64_t)(j * 256), bdesc + (uint64_t)(j * 64), idesc, j > 0 ? 1u : 0u);
            }
            umma_commit(smem_u32(&empty[s]));         // frees the stage and the group's low-nibble buffers
            umma_commit(smem_u32(&gdone[set]));       // the unit's sums are complete
          }
          __syncwarp();
        }
        if (dead) break;
        gseq += (unsigned)(u1 - u0);
      }
      if (*abortp && mine > 0 && wj == 0 && lane == 0) {   // nothing may be in flight when the block frees the tensor memory
#pragma unroll 1
        for (unsigned it = 0; it < 65536u; ++it) {
          if (mbar_try_wait(smem_u32(&empty[s_prev]), use_prev & 1u)) break;
          __nanosleep(64);
        }
      }
    }
  } else {
    // ---- read-back: thread = byte column of the tile and four of the tokens; per unit 4 x (bytes, low nibbles) x 4 digits
    const int q4 = warp & 3, half = (rb >> 2) & 1, grp = rb >> 3, col = q4 * 32 + lane;
    float tf[4];
#pragma unroll
    for (int b = 0; b < 4; ++b) tf[b] = tokfac[half * 4 + b] * 9.094947017729282e-13f;   // * 2^-40
#pragma unroll 1
    for (int item = blockIdx.x; item < nitems; item += gridDim.x) {
      const int tile = item % ntiles, part = item / ntiles;
      const int u0 = (int)(((long long)nunits * part) / usplit), u1 = (int)(((long long)nunits * (part + 1)) / usplit);
      const int nu = u1 - u0;
      const int chunk = tile * 8 + (col >> 4);
      const bool col_ok = chunk < nchunks;
      float t0[4] = {0.f, 0.f, 0.f, 0.f}, t1[4] = {0.f, 0.f, 0.f, 0.f};
      bool dead = false;
      // scales and digit sums are fetched one unit of this set (two units) ahead: their latency is longer than a unit takes
      auto load_scale = [&](int ul) -> uint32_t {
        if (!col_ok || ul >= nu) return 0u;
        const int g = per_row ? 0 : (u0 + ul);
        if (LO) return __ldg(reinterpret_cast<const uint32_t*>(S + ((size_t)g * nchunks + chunk) * 32) + (col & 15));
        return (uint32_t)__ldg(reinterpret_cast<const uint16_t*>(S + ((size_t)g * nchunks + chunk) * 16) + (col & 15));
      };
      auto load_so = [&](int ul) -> float4 {
        if (ul >= nu) return make_float4(0.f, 0.f, 0.f, 0.f);
        return __ldg(reinterpret_cast<const float4*>(soff + (size_t)(u0 + ul) * kBT) + half);
      };
      const int ul0 = (int)(((unsigned)grp + gseq) & 1u);            // this group's first unit of the item
      uint32_t scw = load_scale(ul0);
      float4 so4 = load_so(ul0);
#pragma unroll 1
      for (int ul = ul0; ul < nu; ul += 2) {
        const unsigned gs = gseq + (unsigned)ul;
        const uint32_t scw2 = load_scale(ul + 2);
        const float4 so42 = load_so(ul + 2);
        const float so[4] = {so4.x, so4.y, so4.z, so4.w};
        const int set = (int)(gs & 3u);
        if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&gdone[set]), (gs >> 2) & 1u, abortp))) { dead = true; break; }
        tc_fence_after();
        const uint32_t ta = tbase + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(set * 64 + half * 16);
        uint32_t a[16], l[16];
        tmem_ld16(ta, a);
        if (LO) tmem_ld16(ta + 32u, l);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) asm volatile("st.release.cta.shared.u32 [%0], %1;" ::"r"(smem_u32(&drained[rb])), "r"(gs + 1u) : "memory");
        float sx, sy;
        if (LO) { const float2 sc = __half22float2(*reinterpret_cast<const __half2*>(&scw)); sx = sc.x; sy = sc.y * 0.0625f; }
        else { sx = __half2float(__ushort_as_half((unsigned short)scw)); sy = 0.f; }
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          const int a0 = (int)a[4 * b], a1 = (int)a[4 * b + 1], a2 = (int)a[4 * b + 2], a3 = (int)a[4 * b + 3];
          if (LO) {
            const int l0 = (int)l[4 * b], l1 = (int)l[4 * b + 1], l2 = (int)l[4 * b + 2], l3 = (int)l[4 * b + 3];
            const float fl = digits4_to_float(l0, l1, l2, l3);
            const float fh = digits4_to_float(a0 - l0, a1 - l1, a2 - l2, a3 - l3);    // 16 x the high-nibble sums
            t0[b] = fmaf(sx, fmaf(-8.f, so[b], fl), t0[b]);
            t1[b] = fmaf(sy, fmaf(-128.f, so[b], fh), t1[b]);
          } else {
            t0[b] = fmaf(sx, fmaf(-128.f, so[b], digits4_to_float(a0, a1, a2, a3)), t0[b]);
          }
        }
        scw = scw2; so4 = so42;
      }
      if (dead) break;
      // bytes 0..7 of a chunk hold gate codes, bytes 8..15 the up codes of the same channels
      if (col_ok) {
        const int which = (col >> 3) & 1;
        const int ch = LO ? chunk * 16 + 2 * (col & 7) : chunk * 8 + (col & 7);
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          float* dst = pacc + ((size_t)(half * 4 + b) * 2 + which) * F + ch;
          atomicAdd(dst, t0[b] * tf[b]);
          if (LO) atomicAdd(dst + 1, t1[b] * tf[b]);
        }
      }
      gseq += (unsigned)nu;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && abort_flag) atomicOr(status, kWaitExpired);
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "r"(256u) : "memory");
}

// score[b][ch] = |up~ * SiLU(gate~)| from the accumulated sums; the accumulator is cleared for the next call.
__global__ void __launch_bounds__(256)
proxy_umma_finish_kernel(float* __restrict__ pacc, int B, int F, float* __restrict__ scores) {
  pdl_enter();
  for (int i = blockIdx.x * 256 + threadIdx.x; i < kBT * F; i += gridDim.x * 256) {
    const int b = i / F, ch = i - b * F;
    float* pg = pacc + (size_t)b * 2 * F + ch;
    const float gate = pg[0], up = pg[F];
    pg[0] = 0.f; pg[F] = 0.f;
    if (b < B) scores[(size_t)b * F + ch] = fabsf(up * silu_fast(gate));
  }
}

}  // namespace prox
