// One persistent kernel for the whole batch-1 path (Sec. 4.1 Stage 1 + Stage 2):
//
//   A  every block: exact top-k1 of |x| (redundantly; x is a few KB)
//   B  proxy GEMV over (channel strip, row split) items; the kept rows of the
//      packed proxy land in shared memory through 16-byte async copies; split-K
//      partials meet through a ticket counter; the last block of a strip writes
//      the scores |u~ SiLU(g~)| and adds them to a global 2048-bin histogram
//   -- one grid-wide barrier (bounded spin, self-resetting) --
//   C  every block: exact k2-th score from the histogram plus a refinement over
//      the few candidates of the threshold bin; ballot compaction; the block
//      keeps the slice of the ascending channel list that is its share
//   D  gate/up rows of its channels stream through a shared-memory ring filled
//      by bulk async copies (cp.async.bulk + mbarrier, four issuing warps); each
//      consumer warp owns whole channels: h_j = SiLU(x.g_j) (x.u_j)
//   E  the matching rows of channel-major W_down follow in the same ring; warp
//      groups own whole rows; partial y vectors meet in shared memory and are
//      added to an fp32 accumulator with vector atomics
//   F  the last block to finish (ticket) rounds y once and clears the scratch.
//
// Launch: cooperative (all blocks co-resident), one block per SM.
#pragma once

#include "prox_kernels.cuh"

namespace prox {

constexpr int kFusedConsumerWarps = 16;
constexpr int kFusedConsumers = kFusedConsumerWarps * 32;       // 512
constexpr int kFusedProducers = 4;                               // warps whose lane 0 issues bulk copies
constexpr int kFusedThreads = kFusedConsumers + 32 * kFusedProducers;   // 640
constexpr int kFusedWarps = kFusedThreads / 32;                 // 20
constexpr int kMaxSlots = 32;
constexpr int kEmptyCount = 16;      // arrivals that free a ring slot
constexpr int kChanBatch = 256;      // channels whose h values are held at once
constexpr int kMySelCap = 512;       // channels one block may own
constexpr int kCandCap = 4096;       // threshold-bin candidates kept in shared memory
constexpr int kCand2Cap = 256;       // candidates left after the second refinement
constexpr int kScaleGroupsPerWarp = 2;   // scale blocks a warp stages per item
constexpr int kProxyRowsInFlight = 8;    // packed proxy rows a warp keeps in flight
constexpr unsigned kSpinLimit = 1u << 21;

struct FusedParams {
  const uint8_t* P; const __half* S;
  const uint16_t* wg; const uint16_t* wu; const uint16_t* wdt;
  const uint16_t* x; void* y;
  int D, F, k1, k2, gshift, out_fp32;
  int nstrips, ksplit;
  float* part; unsigned* ticket; float* scores; unsigned* ghist; int* sel_out;
  float* yacc; unsigned long long* bar_count; unsigned* done_ticket; int* status;
  int big_bytes;      // bytes of the large shared buffer
  int nslots;         // ring slots of D*2 bytes inside it
  unsigned long long* trace;   // optional [grid][32] phase time stamps (ns), NULL = off
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
__device__ __forceinline__ void mbar_arrive_n(uint32_t bar, uint32_t n) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(n) : "memory");
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
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
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
__device__ __forceinline__ float4 lds128f(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
#define PROX_TRACE(k) do { if (p.trace && tid == 0) p.trace[(size_t)cta * 32 + (k)] = global_ns(); } while (0)
__device__ __forceinline__ void consumer_sync() {     // the 512 consumer threads only
  asm volatile("bar.sync 1, %0;" ::"n"(kFusedConsumers) : "memory");
}

// Bounded wait on an mbarrier phase.  Gives up (and raises the block's abort
// flag) after kSpinLimit polls; once the flag is up every wait returns at once.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  if (*abort_flag) return false;
  for (unsigned it = 0; it < kSpinLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (it > 256) __nanosleep(64);
    if ((it & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

// Wait for use number `use` of a ring slot.  Different warps consume different
// uses of one slot, and a parity wait cannot tell phase u from phase u-2, so a
// warp first waits (bounded) until the consumer of the previous use has seen
// its data complete; from then on the barrier can only be in phase `use`.
__device__ __forceinline__ bool slot_wait(uint32_t bar, volatile unsigned* seen, unsigned use,
                                          volatile int* abort_flag) {
  if (use > 0 && *seen < use) {
    bool ok = false;
    for (unsigned it = 0; it < kSpinLimit; ++it) {
      if (*seen >= use) { ok = true; break; }
      if (it > 256) __nanosleep(32);
      if ((it & 255u) == 255u && *abort_flag) return false;
    }
    if (!ok) { *abort_flag = 1; return false; }
  }
  if (!mbar_wait(bar, use & 1u, abort_flag)) return false;
  *seen = use + 1u;
  return true;
}

// Exclusive prefix over the lanes of a warp of popc(m8), m8 an 8-bit mask per
// lane: eight ballots instead of a five-step shuffle scan (shuffles are slow here).
__device__ __forceinline__ unsigned lane_prefix8(unsigned m8, unsigned lt_mask) {
  unsigned pre = 0;
#pragma unroll
  for (int e = 0; e < 8; ++e) pre += __popc(__ballot_sync(0xffffffffu, (m8 >> e) & 1u) & lt_mask);
  return pre;
}

// k-th largest bin of hist[0..NBINS) counted from the top, with two block
// barriers: warps scan their bins with shuffles, every thread then adds up the
// totals of the warps in front of it.  Result in res[0] (bin), res[1] (above).
template <int NT, int NBINS>
__device__ __forceinline__ void find_kth_fast(const unsigned* hist, unsigned k, unsigned* wsum, unsigned* res) {
  constexpr int PER = (NBINS + NT - 1) / NT;
  constexpr int NW = NT / 32;
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  unsigned loc[PER];
  unsigned sum = 0;
#pragma unroll
  for (int q = 0; q < PER; ++q) {
    const int bin = NBINS - 1 - (t * PER + q);
    loc[q] = (bin >= 0) ? hist[bin] : 0u;
    sum += loc[q];
  }
  unsigned inc = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned v = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += v;
  }
  if (lane == 31) wsum[warp] = inc;
  __syncthreads();
  unsigned pre = 0;
#pragma unroll
  for (int w = 0; w < NW; ++w) { const unsigned v = wsum[w]; pre += (w < warp) ? v : 0u; }
  const unsigned ex = pre + inc - sum;
  if (ex < k && k <= ex + sum) {
    unsigned run = ex;
#pragma unroll
    for (int q = 0; q < PER; ++q) {
      if (run < k && k <= run + loc[q]) { res[0] = (unsigned)(NBINS - 1 - (t * PER + q)); res[1] = run; }
      run += loc[q];
    }
  }
  __syncthreads();
}

// Same for NBINS <= 256, done by one warp alone (every warp may call it with the
// same arguments and gets the same answer; no block barrier).  Returns the bin
// and writes the count above it.
template <int NBINS>
__device__ __forceinline__ unsigned find_kth_warp(const unsigned* hist, unsigned k, unsigned* above) {
  constexpr int PER = NBINS / 32;
  const int lane = threadIdx.x & 31;
  unsigned loc[PER];
  unsigned sum = 0;
#pragma unroll
  for (int q = 0; q < PER; ++q) { loc[q] = hist[NBINS - 1 - (lane * PER + q)]; sum += loc[q]; }
  unsigned inc = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned v = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += v;
  }
  const unsigned ex = inc - sum;
  const bool mine = ex < k && k <= ex + sum;
  unsigned bin = 0, ab = 0;
  if (mine) {
    unsigned run = ex;
#pragma unroll
    for (int q = 0; q < PER; ++q) {
      if (run < k && k <= run + loc[q]) { bin = (unsigned)(NBINS - 1 - (lane * PER + q)); ab = run; }
      run += loc[q];
    }
  }
  const unsigned who = __ballot_sync(0xffffffffu, mine);
  const int src = who ? (__ffs(who) - 1) : 0;
  bin = __shfl_sync(0xffffffffu, bin, src);
  ab = __shfl_sync(0xffffffffu, ab, src);
  *above = ab;
  return bin;
}

// ---- shared memory map --------------------------------------------------------
struct FusedSmem {
  unsigned hist[2048];
  unsigned hist2[256];
  unsigned wsum[32];
  unsigned res[8];
  unsigned long long mbar_full[kMaxSlots];
  unsigned long long mbar_empty[kMaxSlots];
  int mysel[kMySelCap];
  float hval[kChanBatch];
  unsigned warp_cnt[kFusedWarps][2];
  unsigned cand2_key[kCand2Cap];
  int cand2_idx[kCand2Cap];
  int abort_flag;
  int s_last;
  unsigned ncand;
  unsigned ncand2;
  unsigned prod_seq;       // rows the producers have armed so far (for the give-up path)
  unsigned slot_use[kMaxSlots];   // uses of each ring slot whose data has been seen complete
};

// NG = warp groups of the down projection (4: d_model <= 4096, 2: <= 8192, 1: <= 16384)
template <int BITS, int NG>
__global__ void __launch_bounds__(kFusedThreads, 1) prox_fused_kernel(const FusedParams p) {
  constexpr int CH = ProxyFmt<BITS>::CH, NACC = ProxyFmt<BITS>::NACC;
  constexpr int NT = kFusedThreads;
  extern __shared__ __align__(128) uint8_t smem_raw[];
  FusedSmem& sm = *reinterpret_cast<FusedSmem*>(smem_raw);
  const int D = p.D, F = p.F, k1 = p.k1, k2 = p.k2;
  uint16_t* xs = reinterpret_cast<uint16_t*>(smem_raw + ((sizeof(FusedSmem) + 127) & ~size_t(127)));
  uint16_t* idx16 = xs + D;
  float* xf = reinterpret_cast<float*>(idx16 + D);
  uint8_t* big = reinterpret_cast<uint8_t*>(xf + D);           // 128-byte aligned: D % 128 == 0
  const uint32_t big_u32 = smem_u32(big);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, cta = blockIdx.x;
  volatile int* abortp = &sm.abort_flag;
  const unsigned lt_mask = (1u << lane) - 1u;

  // ------------------------------------------------------------------ set-up
  PROX_TRACE(0);
  if (tid < kMaxSlots) {
    mbar_init(smem_u32(&sm.mbar_full[tid]), 1);
    mbar_init(smem_u32(&sm.mbar_empty[tid]), kEmptyCount);
    fence_mbar_init();
  }
  if (tid == 0) { sm.abort_flag = 0; sm.ncand = 0; sm.ncand2 = 0; sm.prod_seq = 0; }
  if (tid < kMaxSlots) sm.slot_use[tid] = 0;
  {
    const uint4* xg = reinterpret_cast<const uint4*>(p.x);
    for (int i = tid; i < D / 8; i += NT) {
      const uint4 v = __ldg(xg + i);
      reinterpret_cast<uint4*>(xs)[i] = v;
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
      reinterpret_cast<float4*>(xf)[2 * i] = make_float4(bf16_lo(w[0]), bf16_hi(w[0]), bf16_lo(w[1]), bf16_hi(w[1]));
      reinterpret_cast<float4*>(xf)[2 * i + 1] = make_float4(bf16_lo(w[2]), bf16_hi(w[2]), bf16_lo(w[3]), bf16_hi(w[3]));
    }
    for (int i = tid; i < 1024 + 32; i += NT) { if (i < 1024) sm.hist[i] = 0; else sm.hist2[i - 1024] = 0; }
  }
  __syncthreads();
  PROX_TRACE(1);

  // ------------------------------------------------- A: input mask (top-k1 of |x|)
  // A warp takes 256 consecutive inputs at a time, 8 per lane (one 16-byte load).
  {
    const int nvec = D / 8;                               // 8-key vectors
    const int nchk = (nvec + 31) / 32;                    // 256-key chunks (<= 64)
    unsigned T = 0, quota = 0;
    if (k1 < D) {
      // level 1: 10 bits (exponent and two mantissa bits), level 2: the other 5
      for (int q = warp; q < nchk; q += kFusedWarps) {
        const int v = q * 32 + lane;
        if (v < nvec) {
          const uint4 kv = reinterpret_cast<const uint4*>(xs)[v];
          const uint32_t w[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            atomicAdd(&sm.hist[(w[e] & 0x7fffu) >> 5], 1u);
            atomicAdd(&sm.hist[(w[e] >> 21) & 0x3ffu], 1u);
          }
        }
      }
      __syncthreads();
      PROX_TRACE(10);
      find_kth_fast<NT, 1024>(sm.hist, (unsigned)k1, sm.wsum, sm.res);
      const unsigned bin1 = sm.res[0], above1 = sm.res[1];
      PROX_TRACE(11);
      for (int q = warp; q < nchk; q += kFusedWarps) {
        const int v = q * 32 + lane;
        if (v < nvec) {
          const uint4 kv = reinterpret_cast<const uint4*>(xs)[v];
          const uint32_t w[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const unsigned k0 = w[e] & 0x7fffu, k1b = (w[e] >> 16) & 0x7fffu;
            if ((k0 >> 5) == bin1) atomicAdd(&sm.hist2[k0 & 31u], 1u);
            if ((k1b >> 5) == bin1) atomicAdd(&sm.hist2[k1b & 31u], 1u);
          }
        }
      }
      __syncthreads();
      PROX_TRACE(12);
      unsigned above2;
      const unsigned bin2 = find_kth_warp<32>(sm.hist2, (unsigned)k1 - above1, &above2);
      T = (bin1 << 5) | bin2;
      quota = (unsigned)k1 - above1 - above2;      // ties at T to accept, lowest index first
      PROX_TRACE(13);
    }
    // Ordered compaction.  A warp keeps the kept/tie masks of its chunks in
    // registers, counts them with one warp reduction and prefixes them with ballots.
    unsigned* ccnt = sm.hist;                              // reuse: [1024 + q] packed counts of chunk q
    constexpr int MAXC = 4;                                // chunks per warp (64 chunks / 20 warps)
    unsigned gmv[MAXC], emv[MAXC], pgv[MAXC], pev[MAXC];
#pragma unroll
    for (int sidx = 0; sidx < MAXC; ++sidx) {
      const int q = warp + sidx * kFusedWarps;
      gmv[sidx] = emv[sidx] = pgv[sidx] = pev[sidx] = 0;
      if (q < nchk) {                                      // warp-uniform
        const int v = q * 32 + lane;
        unsigned gm = 0, em = 0;
        if (v < nvec) {
          const uint4 kv = reinterpret_cast<const uint4*>(xs)[v];
          const uint32_t w[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const unsigned key = (w[e >> 1] >> ((e & 1) * 16)) & 0x7fffu;
            gm |= ((k1 >= D || key > T) ? 1u : 0u) << e;
            em |= ((k1 < D && key == T) ? 1u : 0u) << e;
          }
        }
        gmv[sidx] = gm; emv[sidx] = em;
        pgv[sidx] = lane_prefix8(gm, lt_mask);
        pev[sidx] = lane_prefix8(em, lt_mask);
        const unsigned tot = __reduce_add_sync(0xffffffffu, (unsigned)__popc(gm) | ((unsigned)__popc(em) << 16));
        if (lane == 0) ccnt[1024 + q] = tot;
      }
    }
    __syncthreads();
    PROX_TRACE(14);
#pragma unroll
    for (int sidx = 0; sidx < MAXC; ++sidx) {
      const int q = warp + sidx * kFusedWarps;
      if (q < nchk) {
        unsigned bsum = 0;                                 // counts of the chunks in front (<= 64)
        for (int j = lane; j < q; j += 32) bsum += ccnt[1024 + j];
        bsum = __reduce_add_sync(0xffffffffu, bsum);
        unsigned rg = (bsum & 0xffffu) + pgv[sidx], re = (bsum >> 16) + pev[sidx];
        const int v = q * 32 + lane;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const bool gt = (gmv[sidx] >> e) & 1u, eq = (emv[sidx] >> e) & 1u;
          if (gt || (eq && re < quota)) idx16[rg + min(re, quota)] = (uint16_t)(v * 8 + e);
          rg += gt ? 1u : 0u; re += eq ? 1u : 0u;
        }
      }
    }
    __syncthreads();
  }

  PROX_TRACE(2);
  // --------------------------------------- B: proxy GEMV, scores, score histogram
  {
    const int nchunks = F / CH;
    const size_t row_bytes = (size_t)nchunks * 16;
    const int nitems = p.nstrips * p.ksplit;
    constexpr int SCB = NACC * 2 * 32;          // bytes of one (group, strip) scale block: 2 KB / 1 KB
    constexpr int NBUF = kProxyRowsInFlight;    // 512-byte row buffers per warp, one async-copy group each
    // per warp: [2 scale blocks][NBUF row buffers]
    const uint32_t wscale = big_u32 + (uint32_t)warp * (uint32_t)(kScaleGroupsPerWarp * SCB + NBUF * 512);
    const uint32_t wbuf = wscale + (uint32_t)(kScaleGroupsPerWarp * SCB);
    for (int item = cta; item < nitems; item += G) {
      const int strip = item % p.nstrips, ks = item / p.nstrips;
      // 32-bit arithmetic on purpose (k1 <= 16384, ks < 64): a 64-bit division costs about a microsecond here
      const int r0 = (int)(((unsigned)k1 * (unsigned)ks) / (unsigned)p.ksplit);
      const int r1 = (int)(((unsigned)k1 * (unsigned)(ks + 1)) / (unsigned)p.ksplit);
      float tot[NACC];
#pragma unroll
      for (int c = 0; c < NACC; ++c) tot[c] = 0.f;
      if (warp < kFusedConsumerWarps) {
        const int w0 = r0 + (int)(((unsigned)(r1 - r0) * (unsigned)warp) / (unsigned)kFusedConsumerWarps);
        const int w1 = r0 + (int)(((unsigned)(r1 - r0) * (unsigned)(warp + 1)) / (unsigned)kFusedConsumerWarps);
        const int nrows = w1 - w0;
        const int seg = (int)min((size_t)512, row_bytes - (size_t)strip * 512);
        const bool lane_valid = lane * 16 < seg;
        const int chunk = strip * 32 + lane;
        // Rows (and the scale blocks of the first two groups they touch) land in
        // shared memory through 16-byte async copies, one copy group per row, so
        // that a row can be consumed as soon as it is there.  Every lane later
        // reads back exactly the bytes it copied itself: no barrier is needed.
        const uint8_t* src0 = p.P + (size_t)strip * 512 + (size_t)lane * 16;
        const int g_first = (nrows > 0) ? (idx16[w0] >> p.gshift) : 0;
        const int g_last = (nrows > 0) ? (idx16[w1 - 1] >> p.gshift) : -1;
        if (lane_valid) {
#pragma unroll
          for (int gq = 0; gq < kScaleGroupsPerWarp; ++gq) {
            if (g_first + gq <= g_last) {
              const uint8_t* ssrc = reinterpret_cast<const uint8_t*>(p.S + ((size_t)(g_first + gq) * nchunks + chunk) * NACC);
#pragma unroll
              for (int v4 = 0; v4 < NACC / 8; ++v4)
                cp_async16(wscale + (uint32_t)(gq * SCB + lane * (NACC * 2) + v4 * 16), ssrc + v4 * 16);
            }
          }
        }
        cp_async_commit();
        auto issue_row = [&](int rr) {                    // always commits, so group counting stays uniform
          if (rr < nrows && lane_valid) {
            const int i = idx16[w0 + rr];
            cp_async16(wbuf + (uint32_t)(rr % NBUF) * 512u + (uint32_t)lane * 16u, src0 + (size_t)i * row_bytes);
          }
          cp_async_commit();
        };
#pragma unroll
        for (int rr = 0; rr < NBUF; ++rr) issue_row(rr);
        PROX_TRACE(29);
        float acc[NACC];
#pragma unroll
        for (int c = 0; c < NACC; ++c) acc[c] = 0.f;
        int curg = -1;
        auto flush = [&](int g) {
          if (g < 0 || !lane_valid) return;
          uint4 sv[NACC / 8];
          if (g - g_first < kScaleGroupsPerWarp) {
#pragma unroll
            for (int v4 = 0; v4 < NACC / 8; ++v4)
              sv[v4] = lds128(wscale + (uint32_t)((g - g_first) * SCB + lane * (NACC * 2) + v4 * 16));
          } else {
            const uint4* sp = reinterpret_cast<const uint4*>(p.S + ((size_t)g * nchunks + chunk) * NACC);
#pragma unroll
            for (int v4 = 0; v4 < NACC / 8; ++v4) sv[v4] = __ldg(sp + v4);
          }
#pragma unroll
          for (int v4 = 0; v4 < NACC / 8; ++v4) {
            const uint32_t sw[4] = {sv[v4].x, sv[v4].y, sv[v4].z, sv[v4].w};
#pragma unroll
            for (int h2 = 0; h2 < 4; ++h2) {
              const float2 sc = __half22float2(*reinterpret_cast<const __half2*>(&sw[h2]));
              const int c = v4 * 8 + h2 * 2;
              tot[c] = fmaf(sc.x, acc[c], tot[c]);
              tot[c + 1] = fmaf(sc.y, acc[c + 1], tot[c + 1]);
              acc[c] = 0.f; acc[c + 1] = 0.f;
            }
          }
        };
        for (int rr = 0; rr < nrows; ++rr) {
          cp_async_wait<NBUF - 1>();                      // the group of row rr (and the scales) has landed
          if (rr == 0) PROX_TRACE(27);
          const int i = idx16[w0 + rr];
          const float xv = xf[i];
          const int g = i >> p.gshift;
          if (g != curg) { flush(curg); curg = g; }
          if (lane_valid) {
            const uint4 v = lds128(wbuf + (uint32_t)(rr % NBUF) * 512u + (uint32_t)lane * 16u);
            proxy_accumulate_exact<BITS>(v, xv, acc);
          }
          issue_row(rr + NBUF);
        }
        cp_async_wait<0>();
        flush(curg);
      }
      PROX_TRACE(22);
      __syncthreads();                         // every warp is done with its row buffers
      PROX_TRACE(23);
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
      PROX_TRACE(24);
      float* fin = red;
      bool last = true;
      if (p.ksplit > 1) {
        float* pb = p.part + ((size_t)ks * p.nstrips + strip) * NV;
#pragma unroll
        for (int q = 0; q < 2; ++q) { const int k = tid + q * NT; if (k < NV) __stcg(pb + k, sumv[q]); }
        __syncthreads();
        if (tid == 0) {
          __threadfence();                      // publishes the whole block's partials (seen through the barrier)
          const unsigned tk = atomicAdd(&p.ticket[strip], 1u);
          sm.s_last = (tk == (unsigned)(p.ksplit - 1));
          __threadfence();
        }
        __syncthreads();
        last = sm.s_last != 0;
        PROX_TRACE(25);
        if (last) {
          float s4[2] = {0.f, 0.f};
          for (int z0 = 0; z0 < p.ksplit; z0 += 8) {         // loads of a batch are independent
            float t[8][2];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const float* pz = p.part + ((size_t)(z0 + u) * p.nstrips + strip) * NV;
#pragma unroll
              for (int q = 0; q < 2; ++q) {
                const int k = tid + q * NT;
                t[u][q] = (z0 + u < p.ksplit && k < NV) ? __ldcg(pz + k) : 0.f;
              }
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) { s4[0] += t[u][0]; s4[1] += t[u][1]; }
          }
#pragma unroll
          for (int q = 0; q < 2; ++q) { const int k = tid + q * NT; if (k < NV) fin[k] = s4[q]; }
          if (tid == 0) p.ticket[strip] = 0;
        }
      } else {
#pragma unroll
        for (int q = 0; q < 2; ++q) { const int k = tid + q * NT; if (k < NV) fin[k] = sumv[q]; }
      }
      PROX_TRACE(26);
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
      __syncthreads();
    }
  }

  PROX_TRACE(3);
  // -------------------------------------------------------------- grid barrier
  // One counter that only grows: a block adds 1 and waits until the count
  // reaches the next multiple of the grid size (no reset, no generation word).
  __syncthreads();
  if (tid == 0) {
    __threadfence();                          // cumulative: publishes the block's writes seen through the barrier above
    const unsigned long long old = atomicAdd(p.bar_count, 1ull);
    // the count is reset by the host long before 2^32 calls; the low word is enough for the division
    const unsigned long long target = old - (unsigned long long)((unsigned)old % (unsigned)G) + (unsigned long long)G;
    bool ok = (old + 1ull == target);
    for (unsigned it = 0; !ok && it < kSpinLimit; ++it) {
      unsigned long long cur;
      asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(cur) : "l"(p.bar_count) : "memory");
      ok = cur >= target;
      if (!ok && it > 64) __nanosleep(32);
    }
    if (!ok) { sm.abort_flag = 1; atomicOr(p.status, kWaitExpired); }
    __threadfence();
  }
  __syncthreads();
  const bool alive = sm.abort_flag == 0;      // block-uniform; a dead block skips to the end
  PROX_TRACE(4);

  // ---------------------------------------- C: channel mask (top-k2 of the scores)
  // k2 <= 65536 and cta < 65536 would overflow 32 bits only beyond any real grid (k2 * G < 2^31 is checked on the host)
  const int R0 = (int)(((unsigned)k2 * (unsigned)cta) / (unsigned)G), R1 = (int)(((unsigned)k2 * (unsigned)(cta + 1)) / (unsigned)G);
  if (alive) {
    unsigned* skey = reinterpret_cast<unsigned*>(big);
    const bool in_smem = (size_t)F * 4 + (size_t)kCandCap * 8 <= (size_t)p.big_bytes;
    unsigned* cand_key = reinterpret_cast<unsigned*>(big + (in_smem ? (size_t)F * 4 : 0));
    int* cand_idx = reinterpret_cast<int*>(cand_key + kCandCap);
    const unsigned* gkey = reinterpret_cast<const unsigned*>(p.scores);
    {
      unsigned hv[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) { const int i = tid + q * NT; hv[q] = (i < 2048) ? __ldcg(p.ghist + i) : 0u; }
#pragma unroll
      for (int q = 0; q < 4; ++q) { const int i = tid + q * NT; if (i < 2048) sm.hist[i] = hv[q]; }
      if (tid < 256) sm.hist2[tid] = 0;
    }
    __syncthreads();
    PROX_TRACE(16);
    find_kth_fast<NT, 2048>(sm.hist, (unsigned)k2, sm.wsum, sm.res);
    const unsigned b1 = sm.res[0];
    unsigned kk = (unsigned)k2 - sm.res[1];
    PROX_TRACE(17);
    // scores -> shared memory, 256 channels per warp step (8 keys per lane);
    // members of the threshold bin become candidates; channels above it are
    // counted per chunk right away (they are selected whatever the exact threshold).
    unsigned* ccnt = sm.hist;                              // [q] kept, [1024 + q] ties, per 256-channel chunk
    const int nchk = (F + 255) / 256;                      // <= 256
    __syncthreads();                                       // find_kth_fast is done with sm.hist
    for (int q = warp; q < nchk; q += kFusedWarps) {
      const int base = q * 256 + lane * 8;
      uint4 kv[2];
#pragma unroll
      for (int hh = 0; hh < 2; ++hh)
        kv[hh] = (base + hh * 4 < F) ? __ldcg(reinterpret_cast<const uint4*>(gkey + base + hh * 4)) : make_uint4(0, 0, 0, 0);
      unsigned hi = 0;
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int i = base + hh * 4;
        if (i < F) {
          if (in_smem) *reinterpret_cast<uint4*>(skey + i) = kv[hh];
          const unsigned kk4[4] = {kv[hh].x, kv[hh].y, kv[hh].z, kv[hh].w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const unsigned bin = kk4[e] >> 20;
            hi += (bin > b1) ? 1u : 0u;
            if (bin == b1) {
              const unsigned slot = atomicAdd(&sm.ncand, 1u);
              if (slot < (unsigned)kCandCap) {
                cand_key[slot] = kk4[e]; cand_idx[slot] = i + e;
                atomicAdd(&sm.hist2[(kk4[e] >> 12) & 255u], 1u);
              }
            }
          }
        }
      }
      hi = __reduce_add_sync(0xffffffffu, hi);
      if (lane == 0) { ccnt[q] = hi; ccnt[1024 + q] = 0; }
    }
    __syncthreads();
    const unsigned ncand = sm.ncand;
    PROX_TRACE(18);
    unsigned T = 0, quota = 0;
    bool have_T = false;
    if (ncand <= (unsigned)kCandCap) {
      // second level (bits 19..12) over the candidates, found by every warp on its own
      unsigned above2;
      const unsigned b2 = find_kth_warp<256>(sm.hist2, kk, &above2);
      const unsigned kk2 = kk - above2;
      const unsigned pre2 = (b1 << 8) | b2;
      for (unsigned c = tid; c < ncand; c += NT) {
        const unsigned key = cand_key[c];
        if ((key >> 12) == pre2) {
          const unsigned slot = atomicAdd(&sm.ncand2, 1u);
          if (slot < (unsigned)kCand2Cap) { sm.cand2_key[slot] = key; sm.cand2_idx[slot] = cand_idx[c]; }
        }
      }
      __syncthreads();
      const unsigned n2 = sm.ncand2;
      PROX_TRACE(19);
      if (n2 <= (unsigned)kCand2Cap) {
        // rank the few that are left by (score descending, channel ascending)
        if (tid < (int)n2) {
          const unsigned key = sm.cand2_key[tid];
          const int id = sm.cand2_idx[tid];
          unsigned rank = 0, same_before = 0;
          for (unsigned c = 0; c < n2; ++c) {
            const unsigned ok = sm.cand2_key[c];
            const int oi = sm.cand2_idx[c];
            rank += (ok > key || (ok == key && oi < id)) ? 1u : 0u;
            same_before += (ok == key && oi < id) ? 1u : 0u;
          }
          if (rank == kk2 - 1u) { sm.res[2] = key; sm.res[3] = same_before + 1u; }
        }
        __syncthreads();
        T = sm.res[2]; quota = sm.res[3];
        PROX_TRACE(20);
        have_T = true;
      }
    }
    if (!have_T) {
      // Rare (massive ties, e.g. an all-zero input): plain radix refinement over all keys.
      unsigned prefix = b1;
      for (int lv = 1; lv < 3; ++lv) {
        const int sh = (lv == 1) ? 9 : 0, nb = (lv == 1) ? 11 : 9;
        __syncthreads();
        for (int i = tid; i < 2048; i += NT) sm.hist[i] = 0;
        __syncthreads();
        for (int i = tid; i < F; i += NT) {
          const unsigned key = in_smem ? skey[i] : __ldcg(gkey + i);
          if ((key >> (sh + nb)) == prefix) atomicAdd(&sm.hist[(key >> sh) & ((1u << nb) - 1u)], 1u);
        }
        __syncthreads();
        if (lv == 1) find_kth_fast<NT, 2048>(sm.hist, kk, sm.wsum, sm.res);
        else         find_kth_fast<NT, 512>(sm.hist, kk, sm.wsum, sm.res);
        prefix = (prefix << nb) | sm.res[0];
        kk -= sm.res[1];
      }
      T = prefix; quota = kk;
    }
    // Per-chunk counts: the channels above the threshold bin are counted already;
    // add the candidates that made it (key > T) and note the ties (key == T).
    bool counted = false;
    if (have_T && ncand <= (unsigned)kCandCap) {
      for (unsigned c = tid; c < ncand; c += NT) {
        const unsigned key = cand_key[c];
        const int chunk = cand_idx[c] >> 8;
        if (key > T) atomicAdd(&ccnt[chunk], 1u);
        else if (key == T) atomicAdd(&ccnt[1024 + chunk], 1u);
      }
      counted = true;
    }
    auto load8 = [&](int base, unsigned* key) {
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int i = base + hh * 4;
        uint4 kv = make_uint4(0, 0, 0, 0);
        if (i < F) kv = in_smem ? *reinterpret_cast<const uint4*>(skey + i)
                                : __ldcg(reinterpret_cast<const uint4*>(gkey + i));
        key[hh * 4 + 0] = kv.x; key[hh * 4 + 1] = kv.y; key[hh * 4 + 2] = kv.z; key[hh * 4 + 3] = kv.w;
      }
    };
    if (!counted) {                                        // rare path: count every chunk from the keys
      for (int q = warp; q < nchk; q += kFusedWarps) {
        const int base = q * 256 + lane * 8;
        unsigned key[8];
        load8(base, key);
        unsigned cg = 0, ce = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const bool in = base + e < F;
          cg += (in && key[e] > T) ? 1u : 0u;
          ce += (in && key[e] == T) ? 1u : 0u;
        }
        cg = __reduce_add_sync(0xffffffffu, cg);
        ce = __reduce_add_sync(0xffffffffu, ce);
        if (lane == 0) { ccnt[q] = cg; ccnt[1024 + q] = ce; }
      }
    }
    __syncthreads();
    PROX_TRACE(21);
    // Ordered compaction: only the chunks whose slice of the ascending list meets
    // [R0, R1) write anything.
    for (int q = warp; q < nchk; q += kFusedWarps) {
      unsigned bg = 0, be = 0;
      for (int j = lane; j < q; j += 32) { bg += ccnt[j]; be += ccnt[1024 + j]; }
      bg = __reduce_add_sync(0xffffffffu, bg);
      be = __reduce_add_sync(0xffffffffu, be);
      const unsigned cgq = ccnt[q], ceq = ccnt[1024 + q];
      const int first = (int)(bg + min(be, quota)), end = (int)(bg + cgq + min(be + ceq, quota));
      if (first >= R1 || end <= R0) continue;              // warp-uniform
      const int base = q * 256 + lane * 8;
      unsigned key[8];
      load8(base, key);
      unsigned gm = 0, em = 0;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const bool in = base + e < F;
        gm |= ((in && key[e] > T) ? 1u : 0u) << e;
        em |= ((in && key[e] == T) ? 1u : 0u) << e;
      }
      unsigned rg = bg + lane_prefix8(gm, lt_mask), re = be + lane_prefix8(em, lt_mask);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const bool gt = (gm >> e) & 1u, eq = (em >> e) & 1u;
        if (gt || (eq && re < quota)) {
          const int pos = (int)(rg + min(re, quota));
          if (pos >= R0 && pos < R1) {
            if (pos - R0 < kMySelCap) sm.mysel[pos - R0] = base + e;
            if (p.sel_out) p.sel_out[pos] = base + e;
          }
        }
        rg += gt ? 1u : 0u; re += eq ? 1u : 0u;
      }
    }
    fence_proxy_async();                      // the big buffer becomes a bulk-copy target next
    __syncthreads();
  }
  const int n_mine = alive ? min(R1 - R0, kMySelCap) : 0;

  PROX_TRACE(5);
  // -------------------------------- D + E: exact gate/up, SwiGLU, masked down
  const int nv = D / 8;                       // 16-byte vectors per row
  const uint32_t row_bytes2 = (uint32_t)D * 2u;
  const int NS = p.nslots;
  constexpr int TG = kFusedConsumers / NG;    // threads of one down-projection group
  constexpr int EV = 4;                       // 16-byte vectors a thread owns in the down projection
  float yr[EV][8];
#pragma unroll
  for (int m = 0; m < EV; ++m)
#pragma unroll
    for (int j = 0; j < 8; ++j) yr[m][j] = 0.f;

  if (warp >= kFusedConsumerWarps) {
    // ---- producer warps: lane 0 of each feeds every kFusedProducers-th slot of
    // the ring (one thread can only start a few million bulk copies a second)
    if (lane == 0) {
      const unsigned pq = (unsigned)(warp - kFusedConsumerWarps);
      unsigned seq = 0;
      int slot = 0;
      unsigned use = 0;
      bool dead = false;
      for (int b0 = 0; b0 < n_mine && !dead; b0 += kChanBatch) {
        const int nb = min(kChanBatch, n_mine - b0);
        for (int q = 0; q < 3 * nb; ++q, ++seq) {
          // A slot always belongs to the same producer: its uses are then armed
          // in program order, so the parity wait below is never two phases behind.
          if (((unsigned)slot & (unsigned)(kFusedProducers - 1)) == pq) {
            if (use > 0 && !mbar_wait(smem_u32(&sm.mbar_empty[slot]), (use - 1u) & 1u, abortp)) { dead = true; break; }
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
            atomicMax(&sm.prod_seq, seq + 1u);
          }
          if (++slot == NS) { slot = 0; ++use; }
        }
      }
    }
  } else {
    // ---- consumer warps
    const uint32_t xf_u32 = smem_u32(xf);
    unsigned base_seq = 0;
    for (int b0 = 0; b0 < n_mine; b0 += kChanBatch) {
      const int nb = min(kChanBatch, n_mine - b0);
      // D: warp w owns channels w, w+16, ... of the batch
      for (int c = warp; c < nb; c += kFusedConsumerWarps) {
        const unsigned sq = base_seq + 2u * (unsigned)c;
        const int sg = (int)(sq % (unsigned)NS), su = (int)((sq + 1u) % (unsigned)NS);
        const unsigned ug = sq / (unsigned)NS, uu = (sq + 1u) / (unsigned)NS;
        const bool ok1 = slot_wait(smem_u32(&sm.mbar_full[sg]), &sm.slot_use[sg], ug, abortp);
        const bool ok2 = slot_wait(smem_u32(&sm.mbar_full[su]), &sm.slot_use[su], uu, abortp);
        float ag = 0.f, au = 0.f, ag2 = 0.f, au2 = 0.f;
        if (ok1 && ok2) {
          const uint32_t pg = big_u32 + (uint32_t)sg * row_bytes2, pu = big_u32 + (uint32_t)su * row_bytes2;
#pragma unroll 2
          for (int v = lane; v < nv; v += 32) {
            const uint4 a = lds128(pg + (uint32_t)v * 16u);
            const uint4 b = lds128(pu + (uint32_t)v * 16u);
            const float4 x0 = lds128f(xf_u32 + (uint32_t)v * 32u);
            const float4 x1 = lds128f(xf_u32 + (uint32_t)v * 32u + 16u);
            ag = fmaf(bf16_lo(a.x), x0.x, ag); ag2 = fmaf(bf16_hi(a.x), x0.y, ag2);
            ag = fmaf(bf16_lo(a.y), x0.z, ag); ag2 = fmaf(bf16_hi(a.y), x0.w, ag2);
            ag = fmaf(bf16_lo(a.z), x1.x, ag); ag2 = fmaf(bf16_hi(a.z), x1.y, ag2);
            ag = fmaf(bf16_lo(a.w), x1.z, ag); ag2 = fmaf(bf16_hi(a.w), x1.w, ag2);
            au = fmaf(bf16_lo(b.x), x0.x, au); au2 = fmaf(bf16_hi(b.x), x0.y, au2);
            au = fmaf(bf16_lo(b.y), x0.z, au); au2 = fmaf(bf16_hi(b.y), x0.w, au2);
            au = fmaf(bf16_lo(b.z), x1.x, au); au2 = fmaf(bf16_hi(b.z), x1.y, au2);
            au = fmaf(bf16_lo(b.w), x1.z, au); au2 = fmaf(bf16_hi(b.w), x1.w, au2);
          }
        }
        ag = warp_sum(ag + ag2); au = warp_sum(au + au2);
        if (lane == 0) {
          const int j = sm.mysel[b0 + c];
          sm.hval[c] = (j >= 0 && j < F) ? au * silu_exact(ag) : 0.f;
          if (ok1 && ok2) {                       // never release a slot whose phase was not seen
            mbar_arrive_n(smem_u32(&sm.mbar_empty[sg]), kEmptyCount);
            mbar_arrive_n(smem_u32(&sm.mbar_empty[su]), kEmptyCount);
          }
        }
      }
      consumer_sync();
      // E: group gq (TG threads) owns rows gq, gq+NG, ... ; a thread owns EV vectors of y
      {
        const int gq = tid / TG, tg = tid % TG;
        for (int c = gq; c < nb; c += NG) {
          const unsigned sq = base_seq + 2u * (unsigned)nb + (unsigned)c;
          const int sd = (int)(sq % (unsigned)NS);
          const unsigned ud = sq / (unsigned)NS;
          const bool ok = slot_wait(smem_u32(&sm.mbar_full[sd]), &sm.slot_use[sd], ud, abortp);
          if (ok) {
            const float hv = sm.hval[c];
            const uint32_t pd = big_u32 + (uint32_t)sd * row_bytes2;
#pragma unroll
            for (int m = 0; m < EV; ++m) {
              const int v = tg + m * TG;
              if (v < nv) {
                const uint4 wv = lds128(pd + (uint32_t)v * 16u);
                yr[m][0] = fmaf(hv, bf16_lo(wv.x), yr[m][0]); yr[m][1] = fmaf(hv, bf16_hi(wv.x), yr[m][1]);
                yr[m][2] = fmaf(hv, bf16_lo(wv.y), yr[m][2]); yr[m][3] = fmaf(hv, bf16_hi(wv.y), yr[m][3]);
                yr[m][4] = fmaf(hv, bf16_lo(wv.z), yr[m][4]); yr[m][5] = fmaf(hv, bf16_hi(wv.z), yr[m][5]);
                yr[m][6] = fmaf(hv, bf16_lo(wv.w), yr[m][6]); yr[m][7] = fmaf(hv, bf16_hi(wv.w), yr[m][7]);
              }
            }
          }
          __syncwarp();
          if (lane == 0 && ok) mbar_arrive_n(smem_u32(&sm.mbar_empty[sd]), (uint32_t)NG);   // TG/32 warps * NG = 16
        }
      }
      consumer_sync();                           // hval is reused by the next batch; all ring reads are done
      base_seq += 3u * (unsigned)nb;
    }
    PROX_TRACE(7);
    // the NG partial vectors of the block meet in shared memory (the ring is idle now)
    if (n_mine > 0) {
      float* ysum = reinterpret_cast<float*>(big);
      const int gq = tid / TG, tg = tid % TG;
#pragma unroll
      for (int m = 0; m < EV; ++m) {
        const int v = tg + m * TG;
        if (v < nv) {
          float4* dst = reinterpret_cast<float4*>(ysum + (size_t)gq * D + (size_t)v * 8);
          dst[0] = make_float4(yr[m][0], yr[m][1], yr[m][2], yr[m][3]);
          dst[1] = make_float4(yr[m][4], yr[m][5], yr[m][6], yr[m][7]);
        }
      }
      consumer_sync();
      for (int v4 = tid; v4 < D / 4; v4 += kFusedConsumers) {
        float4 s = reinterpret_cast<const float4*>(ysum)[v4];
#pragma unroll
        for (int g2 = 1; g2 < NG; ++g2) {
          const float4 t = reinterpret_cast<const float4*>(ysum + (size_t)g2 * D)[v4];
          s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w;
        }
        atomicAdd(reinterpret_cast<float4*>(p.yacc) + v4, s);
      }
    }
  }

  // -------------------------------------- F: last block rounds y and cleans up
  __syncthreads();
  PROX_TRACE(8);
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
    __threadfence();                            // the block's atomics are out before the ticket is taken
    const unsigned t = atomicAdd(p.done_ticket, 1u);
    sm.s_last = (t == (unsigned)(G - 1));
    __threadfence();
  }
  __syncthreads();
  if (sm.s_last) {
    for (int i0 = tid * 4; i0 < D; i0 += NT * 4 * 4) {        // loads first: they must not queue behind the stores
      float4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * NT * 4;
        v[u] = (i < D) ? __ldcg(reinterpret_cast<const float4*>(p.yacc + i)) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * NT * 4;
        if (i < D) {
          *reinterpret_cast<float4*>(p.yacc + i) = make_float4(0.f, 0.f, 0.f, 0.f);
          if (p.out_fp32) {
            *reinterpret_cast<float4*>(reinterpret_cast<float*>(p.y) + i) = v[u];
          } else {
            __nv_bfloat162 lo = __floats2bfloat162_rn(v[u].x, v[u].y), hi = __floats2bfloat162_rn(v[u].z, v[u].w);
            uint2 pk;
            pk.x = *reinterpret_cast<unsigned*>(&lo); pk.y = *reinterpret_cast<unsigned*>(&hi);
            *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.y) + i) = pk;
          }
        }
      }
    }
    for (int i = tid; i < 2048; i += NT) p.ghist[i] = 0;
    if (tid == 0) *p.done_ticket = 0;
    __syncthreads();
    PROX_TRACE(9);
  }
}

}  // namespace prox
