// One persistent kernel for the whole batch-1 path (Sec. 4.1 Stage 1 + Stage 2):
//
//   A  every block: exact top-k1 of |x| (redundantly; x is a few KB)
//   B  proxy GEMV over (channel strip, row split) items; rows arrive in shared
//      memory through bulk async copies (cp.async.bulk + mbarrier); split-K
//      partials meet through a ticket counter; the last block of a strip writes
//      the scores |u~ SiLU(g~)| and adds them to a global 2048-bin histogram
//   -- one grid-wide barrier (bounded spin, self-resetting) --
//   C  every block: exact k2-th score from the histogram + a refinement over the
//      few candidates of the threshold bin; ballot compaction; the block keeps
//      the slice [rank range] of the ascending channel list that is its share
//   D  gate/up rows of its channels stream through a shared-memory ring filled
//      by a producer warp; 16 consumer warps form h_j = SiLU(g_j) u_j
//   E  the matching rows of channel-major W_down follow in the same ring;
//      y partials are added to an fp32 accumulator with vector atomics
//   F  the last block to finish (ticket) rounds y once and clears the scratch.
//
// Launch: cooperative (all blocks co-resident), one block per SM.
#pragma once

#include "prox_kernels.cuh"

namespace prox {

constexpr int kFusedConsumerWarps = 16;
constexpr int kFusedConsumers = kFusedConsumerWarps * 32;       // 512
constexpr int kFusedThreads = kFusedConsumers + 32;             // + producer warp
constexpr int kFusedWarps = kFusedThreads / 32;                 // 17
constexpr int kMaxSlots = 32;
constexpr int kChanBatch = 128;      // channels whose gate/up partials are held at once
constexpr int kMySelCap = 512;       // channels one block may own
constexpr int kCandCap = 2048;       // threshold-bin candidates kept in shared memory
constexpr unsigned kSpinLimit = 1u << 21;

struct FusedParams {
  const uint8_t* P; const __half* S;
  const uint16_t* wg; const uint16_t* wu; const uint16_t* wdt;
  const uint16_t* x; void* y;
  int D, F, k1, k2, gshift, out_fp32;
  int nstrips, ksplit;
  float* part; unsigned* ticket; float* scores; unsigned* ghist; int* sel_out;
  float* yacc; unsigned* bar_count; unsigned* bar_gen; unsigned* done_ticket; int* status;
  int big_bytes;      // bytes of the large shared buffer
  int nslots;         // ring slots of D*2 bytes inside it
};

// ---- PTX wrappers -----------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void consumer_sync() {     // the 512 consumer threads only
  asm volatile("bar.sync 1, %0;" ::"n"(kFusedConsumers) : "memory");
}

// Bounded wait on an mbarrier phase.  Gives up (and raises the block's abort
// flag) after kSpinLimit polls; once the flag is up every wait returns at once.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (*abort_flag) return false;
  for (unsigned it = 0; it < kSpinLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (it > 64) __nanosleep(64);
    if ((it & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

// ---- shared memory map --------------------------------------------------------
struct FusedSmem {
  unsigned hist[2048];
  unsigned long long ws[40];
  unsigned res[8];
  unsigned long long mbar_full[kMaxSlots];
  unsigned long long mbar_empty[kMaxSlots];
  unsigned long long mbar_warp[kFusedConsumerWarps][2];
  int mysel[kMySelCap];
  float hval[kChanBatch];
  float2 gup[kChanBatch][kFusedConsumerWarps];
  unsigned warp_cnt[kFusedWarps][2];
  int abort_flag;
  int s_last;
  unsigned ncand;
  unsigned prod_seq;       // rows the producer has armed so far (for the give-up path)
};

template <int BITS, int XCH>
__global__ void __launch_bounds__(kFusedThreads, 1) prox_fused_kernel(const FusedParams p) {
  constexpr int CH = ProxyFmt<BITS>::CH, NACC = ProxyFmt<BITS>::NACC;
  constexpr int NT = kFusedThreads;
  extern __shared__ __align__(128) uint8_t smem_raw[];
  FusedSmem& sm = *reinterpret_cast<FusedSmem*>(smem_raw);
  const int D = p.D, F = p.F, k1 = p.k1, k2 = p.k2;
  uint16_t* xs = reinterpret_cast<uint16_t*>(smem_raw + ((sizeof(FusedSmem) + 127) & ~size_t(127)));
  uint16_t* idx16 = xs + D;
  uint8_t* big = reinterpret_cast<uint8_t*>(idx16 + D);        // 128-byte aligned: D % 128 == 0
  const uint32_t big_u32 = smem_u32(big);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, cta = blockIdx.x;
  volatile int* abortp = &sm.abort_flag;
  const unsigned lt_mask = (1u << lane) - 1u;

  // ------------------------------------------------------------------ set-up
  if (tid == 0) {
    sm.abort_flag = 0; sm.ncand = 0; sm.prod_seq = 0;
    for (int s = 0; s < kMaxSlots; ++s) {
      mbar_init(smem_u32(&sm.mbar_full[s]), 1);
      mbar_init(smem_u32(&sm.mbar_empty[s]), kFusedConsumerWarps);
    }
    for (int w = 0; w < kFusedConsumerWarps; ++w) {
      mbar_init(smem_u32(&sm.mbar_warp[w][0]), 1);
      mbar_init(smem_u32(&sm.mbar_warp[w][1]), 1);
    }
    fence_mbar_init();
  }
  const unsigned my_gen = (tid == 0) ? ld_acquire(p.bar_gen) : 0u;
  {
    const uint4* xg = reinterpret_cast<const uint4*>(p.x);
    for (int i = tid; i < D / 8; i += NT) reinterpret_cast<uint4*>(xs)[i] = __ldg(xg + i);
  }
  __syncthreads();

  // ------------------------------------------------- A: input mask (top-k1 of |x|)
  {
    const int region = (((D + kFusedWarps - 1) / kFusedWarps) + 31) & ~31;   // per warp, multiple of 32
    const int w0 = min(D, warp * region), w1 = min(D, w0 + region);
    unsigned T = 0, quota = 0;
    if (k1 < D) {
      for (int i = tid; i < 1024; i += NT) sm.hist[i] = 0;
      __syncthreads();
      for (int i = tid; i < D; i += NT) atomicAdd(&sm.hist[(xs[i] & 0x7fffu) >> 5], 1u);
      __syncthreads();
      find_kth_bin<NT, 1024>(sm.hist, (unsigned)k1, sm.ws, sm.res);
      const unsigned bin1 = sm.res[0], above1 = sm.res[1];
      __syncthreads();
      if (tid < 32) sm.hist[tid] = 0;
      __syncthreads();
      for (int i = tid; i < D; i += NT) {
        const unsigned key = xs[i] & 0x7fffu;
        if ((key >> 5) == bin1) atomicAdd(&sm.hist[key & 31u], 1u);
      }
      __syncthreads();
      find_kth_bin<NT, 32>(sm.hist, (unsigned)k1 - above1, sm.ws, sm.res);
      T = (bin1 << 5) | sm.res[0];
      quota = (unsigned)k1 - above1 - sm.res[1];
      __syncthreads();
    }
    // ballot compaction, index order = (warp region, iteration, lane)
    unsigned cg = 0, ce = 0;
    for (int i0 = w0; i0 < w1; i0 += 32) {
      const int i = i0 + lane;
      const unsigned key = (i < w1) ? (unsigned)(xs[i] & 0x7fffu) : 0u;
      const bool gt = (i < w1) && (k1 >= D || key > T);
      const bool eq = (i < w1) && (k1 < D) && key == T;
      cg += __popc(__ballot_sync(0xffffffffu, gt));
      ce += __popc(__ballot_sync(0xffffffffu, eq));
    }
    if (lane == 0) { sm.warp_cnt[warp][0] = cg; sm.warp_cnt[warp][1] = ce; }
    __syncthreads();
    unsigned rg = 0, re = 0;
    for (int w = 0; w < warp; ++w) { rg += sm.warp_cnt[w][0]; re += sm.warp_cnt[w][1]; }
    for (int i0 = w0; i0 < w1; i0 += 32) {
      const int i = i0 + lane;
      const unsigned key = (i < w1) ? (unsigned)(xs[i] & 0x7fffu) : 0u;
      const bool gt = (i < w1) && (k1 >= D || key > T);
      const bool eq = (i < w1) && (k1 < D) && key == T;
      const unsigned bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
      const unsigned mg = rg + __popc(bg & lt_mask), me = re + __popc(be & lt_mask);
      if (gt || (eq && me < quota)) idx16[mg + min(me, quota)] = (uint16_t)i;
      rg += __popc(bg); re += __popc(be);
    }
    __syncthreads();
  }

  // --------------------------------------- B: proxy GEMV, scores, score histogram
  {
    const int nchunks = F / CH;
    const size_t row_bytes = (size_t)nchunks * 16;
    const int nitems = p.nstrips * p.ksplit;
    int RB = p.big_bytes / (kFusedConsumerWarps * 2 * 512);
    if (RB > 32) RB = 32;
    const uint32_t wbuf = big_u32 + (uint32_t)warp * 2u * RB * 512u;       // this warp's two buffers
    unsigned use0 = 0, use1 = 0;                                          // waits done on the 2 barriers
    unsigned iss0 = 0, iss1 = 0;                                          // times each was armed
    for (int item = cta; item < nitems; item += G) {
      const int strip = item % p.nstrips, ks = item / p.nstrips;
      const int r0 = (int)(((long long)k1 * ks) / p.ksplit), r1 = (int)(((long long)k1 * (ks + 1)) / p.ksplit);
      float tot[NACC];
#pragma unroll
      for (int c = 0; c < NACC; ++c) tot[c] = 0.f;
      if (warp < kFusedConsumerWarps) {
        const int w0 = r0 + (int)(((long long)(r1 - r0) * warp) / kFusedConsumerWarps);
        const int w1 = r0 + (int)(((long long)(r1 - r0) * (warp + 1)) / kFusedConsumerWarps);
        const int seg = (int)min((size_t)512, row_bytes - (size_t)strip * 512);
        const bool lane_valid = lane * 16 < seg;
        const int chunk = strip * 32 + lane;
        const int nch = (w1 - w0 + RB - 1) / RB;
        const uint32_t bar0 = smem_u32(&sm.mbar_warp[warp][0]), bar1 = smem_u32(&sm.mbar_warp[warp][1]);
        auto issue = [&](int c) {
          const int buf = c & 1;
          const int n = min(RB, w1 - w0 - c * RB);
          const uint32_t bar = buf ? bar1 : bar0;
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) mbar_expect_tx(bar, (uint32_t)(n * seg));
          if (buf) ++iss1; else ++iss0;
          __syncwarp();
          if (lane < n) {
            const int i = idx16[w0 + c * RB + lane];
            bulk_g2s(wbuf + (uint32_t)(buf * RB + lane) * 512u, p.P + (size_t)i * row_bytes + (size_t)strip * 512,
                     (uint32_t)seg, bar);
          }
        };
        if (nch > 0) issue(0);
        if (nch > 1) issue(1);
        float acc[NACC];
#pragma unroll
        for (int c = 0; c < NACC; ++c) acc[c] = 0.f;
        float sumx = 0.f;
        int curg = -1;
        auto flush = [&](int g) {
          if (g < 0 || !lane_valid) return;
          const uint4* sp = reinterpret_cast<const uint4*>(p.S + ((size_t)g * nchunks + chunk) * NACC);
#pragma unroll
          for (int v4 = 0; v4 < NACC / 8; ++v4) {
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
        for (int c = 0; c < nch; ++c) {
          const int buf = c & 1;
          const int n = min(RB, w1 - w0 - c * RB);
          const unsigned par = (buf ? use1 : use0) & 1u;
          const bool ok = mbar_wait(buf ? bar1 : bar0, par, abortp);
          if (buf) ++use1; else ++use0;
          if (ok) {
            for (int r = 0; r < n; ++r) {
              const int i = idx16[w0 + c * RB + r];
              const float xv = __uint_as_float(((uint32_t)xs[i]) << 16);
              const int g = i >> p.gshift;
              if (g != curg) { flush(curg); curg = g; }
              sumx += xv;
              if (lane_valid) {
                const uint4 v = lds128(wbuf + (uint32_t)(buf * RB + r) * 512u + (uint32_t)lane * 16u);
                proxy_accumulate<BITS>(v, xv, acc);
              }
            }
          }
          __syncwarp();
          if (c + 2 < nch) issue(c + 2);
        }
        flush(curg);
      }
      __syncthreads();                         // every warp is done with its row buffers
      float* red = reinterpret_cast<float*>(big);
      if (warp < kFusedConsumerWarps) {
#pragma unroll
        for (int c = 0; c < NACC; ++c) red[warp * (NACC * 32) + c * 32 + lane] = tot[c];
      }
      __syncthreads();
      constexpr int NV = NACC * 32;            // values per strip: 1024 (4-bit) or 512 (8-bit)
      float sumv[2] = {0.f, 0.f};
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const int k = tid + q * NT;
        if (k < NV) {
          float s = 0.f;
#pragma unroll
          for (int w = 0; w < kFusedConsumerWarps; ++w) s += red[w * NV + k];
          sumv[q] = s;
        }
      }
      __syncthreads();
      float* fin = red;
      bool last = true;
      if (p.ksplit > 1) {
        float* pb = p.part + ((size_t)ks * p.nstrips + strip) * NV;
#pragma unroll
        for (int q = 0; q < 2; ++q) { const int k = tid + q * NT; if (k < NV) __stcg(pb + k, sumv[q]); }
        __threadfence();
        __syncthreads();
        if (tid == 0) {
          const unsigned tk = atomicAdd(&p.ticket[strip], 1u);
          sm.s_last = (tk == (unsigned)(p.ksplit - 1));
        }
        __syncthreads();
        last = sm.s_last != 0;
        if (last) {
          __threadfence();
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            const int k = tid + q * NT;
            if (k < NV) {
              float s = 0.f;
              for (int z = 0; z < p.ksplit; ++z) s += __ldcg(p.part + ((size_t)z * p.nstrips + strip) * NV + k);
              fin[k] = s;
            }
          }
          if (tid == 0) p.ticket[strip] = 0;
        }
      } else {
#pragma unroll
        for (int q = 0; q < 2; ++q) { const int k = tid + q * NT; if (k < NV) fin[k] = sumv[q]; }
      }
      if (last) {
        for (int i = tid; i < 2048; i += NT) sm.hist[i] = 0;
        __syncthreads();
        for (int k = tid; k < CH * 32; k += NT) {
          const int c = k >> 5, ln = k & 31;
          const int ch = (strip * 32 + ln) * CH + c;
          if (ch < F) {
            const float sc = fabsf(fin[k + CH * 32] * silu_fast(fin[k]));
            __stcg(p.scores + ch, sc);
            atomicAdd(&sm.hist[__float_as_uint(sc) >> 20], 1u);
          }
        }
        __syncthreads();
        for (int i = tid; i < 2048; i += NT) { const unsigned v = sm.hist[i]; if (v) atomicAdd(p.ghist + i, v); }
      }
      fence_proxy_async();                     // generic writes above precede the next item's bulk copies
      __syncthreads();
    }
    // Give-up path only: a copy that was armed but never waited for must land
    // (or its wait expire once more) before this block may leave.
    if (*abortp && warp < kFusedConsumerWarps && lane == 0) {
      for (int b = 0; b < 2; ++b) {
        const unsigned iss = b ? iss1 : iss0, use = b ? use1 : use0;
        if (iss > use)
          for (unsigned it = 0; it < 8192u; ++it) {
            if (mbar_try_wait(smem_u32(&sm.mbar_warp[warp][b]), (iss - 1u) & 1u)) break;
            __nanosleep(256);
          }
      }
    }
  }

  // -------------------------------------------------------------- grid barrier
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const unsigned old = atomicAdd(p.bar_count, 1u);
    if (old == (unsigned)(G - 1)) {
      *(volatile unsigned*)p.bar_count = 0u;
      __threadfence();
      atomicAdd(p.bar_gen, 1u);
    } else {
      bool ok = false;
      for (unsigned it = 0; it < kSpinLimit; ++it) {
        if (ld_acquire(p.bar_gen) != my_gen) { ok = true; break; }
        __nanosleep(32);
      }
      if (!ok) { sm.abort_flag = 1; atomicOr(p.status, kWaitExpired); }
    }
    __threadfence();
  }
  __syncthreads();
  const bool alive = sm.abort_flag == 0;      // block-uniform; a dead block skips to the end

  // ---------------------------------------- C: channel mask (top-k2 of the scores)
  const int R0 = (int)(((long long)k2 * cta) / G), R1 = (int)(((long long)k2 * (cta + 1)) / G);
  if (alive) {
    unsigned* skey = reinterpret_cast<unsigned*>(big);
    const bool in_smem = (size_t)F * 4 + (size_t)kCandCap * 8 <= (size_t)p.big_bytes;
    unsigned* cand_key = reinterpret_cast<unsigned*>(big + (in_smem ? (size_t)F * 4 : 0));
    const unsigned* gkey = reinterpret_cast<const unsigned*>(p.scores);
    for (int i = tid; i < 2048; i += NT) sm.hist[i] = __ldcg(p.ghist + i);
    __syncthreads();
    find_kth_bin<NT, 2048>(sm.hist, (unsigned)k2, sm.ws, sm.res);
    const unsigned b1 = sm.res[0];
    unsigned kk = (unsigned)k2 - sm.res[1];
    __syncthreads();
    for (int i = tid; i < F; i += NT) {
      const unsigned key = __ldcg(gkey + i);
      if (in_smem) skey[i] = key;
      if ((key >> 20) == b1) {
        const unsigned slot = atomicAdd(&sm.ncand, 1u);
        if (slot < (unsigned)kCandCap) cand_key[slot] = key;
      }
    }
    __syncthreads();
    const unsigned ncand = sm.ncand;
    const bool cand_ok = ncand <= (unsigned)kCandCap;
    unsigned prefix = b1;
    // two refinement levels (11 then 9 bits) over the candidates only
    for (int lv = 1; lv < 3; ++lv) {
      const int sh = (lv == 1) ? 9 : 0, nb = (lv == 1) ? 11 : 9;
      for (int i = tid; i < 2048; i += NT) sm.hist[i] = 0;
      __syncthreads();
      if (cand_ok) {
        for (unsigned c = tid; c < ncand; c += NT) {
          const unsigned key = cand_key[c];
          if ((key >> (sh + nb)) == prefix) atomicAdd(&sm.hist[(key >> sh) & ((1u << nb) - 1u)], 1u);
        }
      } else {
        for (int i = tid; i < F; i += NT) {
          const unsigned key = in_smem ? skey[i] : __ldcg(gkey + i);
          if ((key >> (sh + nb)) == prefix) atomicAdd(&sm.hist[(key >> sh) & ((1u << nb) - 1u)], 1u);
        }
      }
      __syncthreads();
      if (lv == 1) find_kth_bin<NT, 2048>(sm.hist, kk, sm.ws, sm.res);
      else         find_kth_bin<NT, 512>(sm.hist, kk, sm.ws, sm.res);
      prefix = (prefix << nb) | sm.res[0];
      kk -= sm.res[1];
      __syncthreads();
    }
    const unsigned T = prefix, quota = kk;
    const int region = (((F + kFusedWarps - 1) / kFusedWarps) + 31) & ~31;
    const int w0 = min(F, warp * region), w1 = min(F, w0 + region);
    unsigned cg = 0, ce = 0;
    for (int i0 = w0; i0 < w1; i0 += 32) {
      const int i = i0 + lane;
      const unsigned key = (i < w1) ? (in_smem ? skey[i] : __ldcg(gkey + i)) : 0u;
      cg += __popc(__ballot_sync(0xffffffffu, (i < w1) && key > T));
      ce += __popc(__ballot_sync(0xffffffffu, (i < w1) && key == T));
    }
    if (lane == 0) { sm.warp_cnt[warp][0] = cg; sm.warp_cnt[warp][1] = ce; }
    __syncthreads();
    unsigned rg = 0, re = 0;
    for (int w = 0; w < warp; ++w) { rg += sm.warp_cnt[w][0]; re += sm.warp_cnt[w][1]; }
    for (int i0 = w0; i0 < w1; i0 += 32) {
      const int i = i0 + lane;
      const unsigned key = (i < w1) ? (in_smem ? skey[i] : __ldcg(gkey + i)) : 0u;
      const bool gt = (i < w1) && key > T, eq = (i < w1) && key == T;
      const unsigned bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
      const unsigned mg = rg + __popc(bg & lt_mask), me = re + __popc(be & lt_mask);
      if (gt || (eq && me < quota)) {
        const int pos = (int)(mg + min(me, quota));
        if (pos >= R0 && pos < R1) {
          if (pos - R0 < kMySelCap) sm.mysel[pos - R0] = i;
          if (p.sel_out) p.sel_out[pos] = i;
        }
      }
      rg += __popc(bg); re += __popc(be);
    }
    __syncthreads();
  }
  const int n_mine = alive ? min(R1 - R0, kMySelCap) : 0;

  // -------------------------------- D + E: exact gate/up, SwiGLU, masked down
  fence_proxy_async();                        // the big buffer now becomes a bulk-copy target again
  __syncthreads();
  const int nv = D / 8;                       // 16-byte vectors per row
  const uint32_t row_bytes2 = (uint32_t)D * 2u;
  const int NS = p.nslots;
  float yr[XCH][8];
#pragma unroll
  for (int m = 0; m < XCH; ++m)
#pragma unroll
    for (int j = 0; j < 8; ++j) yr[m][j] = 0.f;

  if (warp == kFusedConsumerWarps) {
    // ---- producer warp: one lane feeds the ring
    if (lane == 0) {
      unsigned seq = 0;
      for (int b0 = 0; b0 < n_mine; b0 += kChanBatch) {
        const int nb = min(kChanBatch, n_mine - b0);
        for (int q = 0; q < 3 * nb; ++q) {
          const int slot = (int)(seq % (unsigned)NS);
          const unsigned use = seq / (unsigned)NS;
          if (use > 0 && !mbar_wait(smem_u32(&sm.mbar_empty[slot]), (use - 1u) & 1u, abortp)) break;
          const uint16_t* src;
          if (q < 2 * nb) {
            const int j = sm.mysel[b0 + (q >> 1)];
            src = ((q & 1) ? p.wu : p.wg) + (size_t)j * D;
          } else {
            src = p.wdt + (size_t)sm.mysel[b0 + q - 2 * nb] * D;
          }
          const uint32_t bar = smem_u32(&sm.mbar_full[slot]);
          mbar_expect_tx(bar, row_bytes2);
          bulk_g2s(big_u32 + (uint32_t)slot * row_bytes2, src, row_bytes2, bar);
          ++seq;
          sm.prod_seq = seq;
        }
        if (*abortp) break;
      }
    }
  } else {
    // ---- consumer warps
    float xr[XCH][8];
#pragma unroll
    for (int m = 0; m < XCH; ++m) {
      const int v = tid + m * kFusedConsumers;
#pragma unroll
      for (int j = 0; j < 8; ++j) xr[m][j] = 0.f;
      if (v < nv) {
        const uint4 xv = reinterpret_cast<const uint4*>(xs)[v];
        const uint32_t xw[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) { xr[m][2 * q] = bf16_lo(xw[q]); xr[m][2 * q + 1] = bf16_hi(xw[q]); }
      }
    }
    unsigned seq = 0;
    for (int b0 = 0; b0 < n_mine; b0 += kChanBatch) {
      const int nb = min(kChanBatch, n_mine - b0);
      for (int c = 0; c < nb; ++c) {
        const int sg = (int)(seq % (unsigned)NS); const unsigned ug = seq / (unsigned)NS; ++seq;
        const int su = (int)(seq % (unsigned)NS); const unsigned uu = seq / (unsigned)NS; ++seq;
        const bool ok1 = mbar_wait(smem_u32(&sm.mbar_full[sg]), ug & 1u, abortp);
        const bool ok2 = mbar_wait(smem_u32(&sm.mbar_full[su]), uu & 1u, abortp);
        float ag = 0.f, au = 0.f;
        if (ok1 && ok2) {
#pragma unroll
          for (int m = 0; m < XCH; ++m) {
            const int v = tid + m * kFusedConsumers;
            if (v < nv) {
              const uint4 a = lds128(big_u32 + (uint32_t)sg * row_bytes2 + (uint32_t)v * 16u);
              const uint4 b = lds128(big_u32 + (uint32_t)su * row_bytes2 + (uint32_t)v * 16u);
              const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                ag = fmaf(bf16_lo(aw[q]), xr[m][2 * q], ag); ag = fmaf(bf16_hi(aw[q]), xr[m][2 * q + 1], ag);
                au = fmaf(bf16_lo(bw[q]), xr[m][2 * q], au); au = fmaf(bf16_hi(bw[q]), xr[m][2 * q + 1], au);
              }
            }
          }
        }
        ag = warp_sum(ag); au = warp_sum(au);
        if (lane == 0) {
          sm.gup[c][warp] = make_float2(ag, au);
          mbar_arrive(smem_u32(&sm.mbar_empty[sg]));
          mbar_arrive(smem_u32(&sm.mbar_empty[su]));
        }
      }
      consumer_sync();
      if (tid < nb) {
        float g = 0.f, u = 0.f;
#pragma unroll
        for (int w = 0; w < kFusedConsumerWarps; ++w) { const float2 t = sm.gup[tid][w]; g += t.x; u += t.y; }
        const int j = sm.mysel[b0 + tid];
        sm.hval[tid] = (j >= 0 && j < F) ? u * silu_exact(g) : 0.f;
      }
      consumer_sync();
      for (int c = 0; c < nb; ++c) {
        const int sd = (int)(seq % (unsigned)NS); const unsigned ud = seq / (unsigned)NS; ++seq;
        const bool ok = mbar_wait(smem_u32(&sm.mbar_full[sd]), ud & 1u, abortp);
        if (ok) {
          const float hv = sm.hval[c];
#pragma unroll
          for (int m = 0; m < XCH; ++m) {
            const int v = tid + m * kFusedConsumers;
            if (v < nv) {
              const uint4 wv = lds128(big_u32 + (uint32_t)sd * row_bytes2 + (uint32_t)v * 16u);
              const uint32_t ww[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                yr[m][2 * q] = fmaf(hv, bf16_lo(ww[q]), yr[m][2 * q]);
                yr[m][2 * q + 1] = fmaf(hv, bf16_hi(ww[q]), yr[m][2 * q + 1]);
              }
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sm.mbar_empty[sd]));
      }
      consumer_sync();                           // hval / gup are reused by the next batch
    }
    if (n_mine > 0) {
#pragma unroll
      for (int m = 0; m < XCH; ++m) {
        const int v = tid + m * kFusedConsumers;
        if (v < nv) {
          float4* yp = reinterpret_cast<float4*>(p.yacc + (size_t)v * 8);
          atomicAdd(yp, make_float4(yr[m][0], yr[m][1], yr[m][2], yr[m][3]));
          atomicAdd(yp + 1, make_float4(yr[m][4], yr[m][5], yr[m][6], yr[m][7]));
        }
      }
    }
  }

  // -------------------------------------- F: last block rounds y and cleans up
  __threadfence();
  __syncthreads();
  if (sm.abort_flag) {
    // A wait expired: every copy this block armed was either consumed or is
    // waited for here (bounded) so that none lands after the block has left.
    if (tid == 0) {
      atomicOr(p.status, kWaitExpired);
      const unsigned issued = sm.prod_seq;
      const unsigned first = issued > (unsigned)NS ? issued - (unsigned)NS : 0u;
      for (unsigned q = first; q < issued; ++q) {        // the latest use of every slot
        const uint32_t bar = smem_u32(&sm.mbar_full[q % (unsigned)NS]);
        for (unsigned it = 0; it < 8192u; ++it) {
          if (mbar_try_wait(bar, (q / (unsigned)NS) & 1u)) break;
          __nanosleep(256);
        }
      }
    }
    __syncthreads();
    return;
  }
  if (tid == 0) {
    const unsigned t = atomicAdd(p.done_ticket, 1u);
    sm.s_last = (t == (unsigned)(G - 1));
  }
  __syncthreads();
  if (sm.s_last) {
    __threadfence();
    for (int i = tid; i < D; i += NT) {
      const float v = __ldcg(p.yacc + i);
      p.yacc[i] = 0.f;
      if (p.out_fp32) reinterpret_cast<float*>(p.y)[i] = v;
      else reinterpret_cast<__nv_bfloat16*>(p.y)[i] = __float2bfloat16_rn(v);
    }
    for (int i = tid; i < 2048; i += NT) p.ghist[i] = 0;
    if (tid == 0) *p.done_ticket = 0;
  }
}

}  // namespace prox
