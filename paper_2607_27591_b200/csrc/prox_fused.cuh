// One persistent kernel for the whole batch-1 path (Sec. 4.1 Stage 1 + Stage 2):
//
//   A  every block: exact top-k1 of |x| (redundantly; x is a few KB)
//   B  proxy GEMV on the tensor cores (tcgen05, integer MMA, accumulators in
//      tensor memory): a block owns 128-byte column tiles of the packed proxy
//      over ALL kept rows, so the sums of a tile need no exchange with other
//      blocks; the rows' bytes are the A operand as they lie in memory, x enters
//      as signed base-256 digits; the block writes the scores |u~ SiLU(g~)| of
//      its channels and adds them to a global 2048-bin histogram
//   -- one grid-wide barrier (bounded spin, self-resetting) --
//   C  every block (consumer warps only; the producer warps wait at the ring):
//      the histogram gives the threshold bin b1; channels in bins above b1 are
//      kept whatever the exact threshold is.  The kept list is laid out as
//      [those channels, ascending][kept members of b1, ascending] and block c
//      owns the c-th share of both parts.  Two passes over the scores list its
//      share of the first part and the ring starts; half of the consumer warps
//      then settle the exact threshold inside b1 (ordered list of its members,
//      8-bit histogram, rank among the few left) and append the block's share
//      of the second part, while the other half already consumes rows
//   D  gate/up rows of its channels stream through a shared-memory ring filled
//      by bulk async copies (cp.async.bulk + mbarrier, four issuing warps); a
//      consumer warp takes the next channel nobody has taken:
//      h_j = SiLU(x.g_j) (x.u_j)
//   E  the matching rows of channel-major W_down follow in the same ring; warp
//      groups own whole rows; partial y vectors meet in shared memory and are
//      added to an fp32 accumulator with vector atomics
//   F  the last block to finish (ticket) rounds y once and clears the scratch.
//
// Launch: cooperative (all blocks co-resident), one block per SM.
#pragma once

#include "prox_kernels.cuh"
#include "prox_umma.cuh"

namespace prox {

constexpr int kFusedConsumerWarps = 16;
constexpr int kFusedConsumers = kFusedConsumerWarps * 32;       // 512
constexpr int kSettlerWarps = 8;                                 // consumer warps that finish the channel mask
constexpr int kSettlers = kSettlerWarps * 32;
constexpr int kFusedProducers = 4;                               // warps whose lane 0 issues bulk copies
constexpr int kFusedThreads = kFusedConsumers + 32 * kFusedProducers;   // 640
constexpr int kFusedWarps = kFusedThreads / 32;                 // 20
constexpr int kMaxSlots = 32;
constexpr int kEmptyCount = 16;      // arrivals that free a ring slot
constexpr int kChanBatch = 256;      // channels whose h values are held at once
constexpr int kMySelCap = 512;       // channels one block may own
constexpr int kCandCap = 4096;       // threshold-bin candidates kept in shared memory
constexpr int kCand2Cap = 256;       // candidates left after the second refinement
constexpr int kPStages = 16;             // ring of 32-row stages of the proxy GEMV (one per loader warp)
constexpr int kPStageBytes = 9216;       // a stage: 4096 bytes of rows | 4096 low nibbles | 512 digits of x | pad
constexpr int kMaxSuper = 16;            // supergroups (4 scale groups) whose accumulators fit the tensor memory
constexpr unsigned kSpinLimit = 1u << 21;

struct FusedParams {
  const uint8_t* P; const __half* S;
  const uint16_t* wg; const uint16_t* wu; const uint16_t* wdt;
  const uint16_t* x; void* y;
  int D, F, k1, k2, gshift, out_fp32;
  int pstages;        // stages of the proxy ring that fit (<= kPStages)
  float* scores; unsigned* ghist; int* sel_out;
  int* idx_out;       // the kept input list as this kernel built it (block 0 writes it; for checking)
  unsigned spin_limit;        // polls after which a device-side wait gives up
  unsigned bar_bias;          // test knob: added to the grid barrier's target (0 in normal use)
  int* host_flag;             // mapped host word set to 1 when a wait expires (NULL = none)
  float* yacc; unsigned long long* bar_count; unsigned* done_ticket; int* status;
  int big_bytes;      // bytes of the large shared buffer
  int nslots;         // ring slots of D*2 bytes inside it
  unsigned long long* trace;   // optional [grid][32] phase time stamps (ns), NULL = off
  // Layer sub-block form (all NULL / 0 otherwise): the input is bf16(RMSNorm(xres) * norm_w) and the
  // result is xres + y, written as fp32 to xres_out (which may be xres itself).
  const float* xres; const uint16_t* norm_w; float* xres_out; RmsConst rc;
  // Threshold form (THRESH): keep |x_i| >= tau_x and score_j >= tau_s instead of the k1 / k2 largest.
  // tkey_x = smallest 15-bit bf16 magnitude that is >= tau_x, tkey_s = bits of tau_s (scores are >= 0, so
  // their bit patterns order like their values).  Counts go to cnt_x_out / count_out and into counters.
  unsigned tkey_x, tkey_s;
  int* cnt_x_out; int* count_out; unsigned long long* counters;
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
#define PROX_TRACE_AT(k, who) do { if (p.trace && tid == (who)) p.trace[(size_t)cta * 32 + (k)] = global_ns(); } while (0)
#define PROX_TRACE(k) do { if (p.trace && tid == 0) p.trace[(size_t)cta * 32 + (k)] = global_ns(); } while (0)
__device__ __forceinline__ bool elect_one() {          // the same lane every time for a full warp
  uint32_t pred;
  asm volatile("{\n\t.reg .pred P1;\n\telect.sync _|P1, 0xffffffff;\n\tselp.u32 %0, 1, 0, P1;\n\t}" : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ void settler_sync() {      // the lower half of the consumer warps
  asm volatile("bar.sync 3, %0;" ::"n"(kSettlers) : "memory");
}
__device__ __forceinline__ void consumer_sync() {     // the 512 consumer threads only
  asm volatile("bar.sync 1, %0;" ::"n"(kFusedConsumers) : "memory");
}

// Bounded wait on an mbarrier phase.  Gives up (and raises the block's abort
// flag) after kSpinLimit polls; once the flag is up every wait returns at once.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned limit = kSpinLimit) {
  if (mbar_try_wait(bar, parity)) return true;
  if (*abort_flag) return false;
#pragma unroll 1
  for (unsigned it = 0; it < limit; ++it) {
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
                                          volatile int* abort_flag, unsigned limit) {
  if (use > 0 && *seen < use) {
    bool ok = false;
#pragma unroll 1
    for (unsigned it = 0; it < limit; ++it) {
      if (*seen >= use) { ok = true; break; }
      if (it > 256) __nanosleep(32);
      if ((it & 255u) == 255u && *abort_flag) return false;
    }
    if (!ok) { *abort_flag = 1; return false; }
  }
  if (!mbar_wait(bar, use & 1u, abort_flag, limit)) return false;
  *seen = use + 1u;
  return true;
}

// The selection phases run once per call on every block, over code that is cold
// in the instruction caches: their time is set by the number of instructions
// fetched, not executed.  They are therefore written as small loops (one key per
// lane and trip) and the helpers below are shared between the phases.

__device__ __forceinline__ unsigned warp_scan_incl(unsigned v, int lane) {
#pragma unroll 1
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned t = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += t;
  }
  return v;
}

// k-th largest (k >= 1, counted from the top) among the 32 * BPL bins that end
// below index `top`.  One warp; every lane returns the same bin and the count
// above it.  Lane l owns the l-th slice of BPL bins from the top.
template <int BPL>
__device__ __forceinline__ unsigned kth_in_segment(const unsigned* hist, int top, unsigned k, int lane, unsigned* above) {
  const int base = top - (lane + 1) * BPL;
  unsigned s = 0;
#pragma unroll 1
  for (int j = 0; j < BPL; ++j) s += hist[base + j];
  const unsigned inc = warp_scan_incl(s, lane);
  const unsigned ex = inc - s;
  const unsigned m = __ballot_sync(0xffffffffu, ex < k && k <= inc);
  const int src = m ? (__ffs(m) - 1) : 31;
  unsigned run = __shfl_sync(0xffffffffu, ex, src);
  const int b0 = top - (src + 1) * BPL;                 // all lanes walk the same slice (broadcast reads)
  unsigned bin = (unsigned)b0, ab = run;
#pragma unroll 1
  for (int j = BPL - 1; j >= 0; --j) {
    const unsigned c = hist[b0 + j];
    if (run < k && k <= run + c) { bin = (unsigned)(b0 + j); ab = run; }
    run += c;
  }
  *above = ab;
  return bin;
}

// Same over 512 * BPL bins with the whole block (one block barrier inside):
// warps 0..15 total their segment, then every warp locates the segment and
// finishes on its own, so the result is in the registers of every thread.
// CONSUMERS_ONLY: called by the 16 consumer warps alone (named barrier).
template <int BPL, bool CONSUMERS_ONLY>
__device__ __forceinline__ unsigned kth_in_block(const unsigned* hist, unsigned k, unsigned* wsum, int lane, int warp,
                                                 unsigned* above) {
  constexpr int NB = 512 * BPL, SEG = 32 * BPL;
  if (warp < 16) {
    const int base = NB - warp * SEG - (lane + 1) * BPL;
    unsigned s = 0;
#pragma unroll 1
    for (int j = 0; j < BPL; ++j) s += hist[base + j];
    s = __reduce_add_sync(0xffffffffu, s);
    if (lane == 0) wsum[warp] = s;
  }
  if (CONSUMERS_ONLY) consumer_sync(); else __syncthreads();
  const unsigned v = (lane < 16) ? wsum[lane] : 0u;
  const unsigned inc = warp_scan_incl(v, lane);
  const unsigned ex = inc - v;
  const unsigned m = __ballot_sync(0xffffffffu, ex < k && k <= inc);
  const int seg = m ? (__ffs(m) - 1) : 15;
  const unsigned aseg = __shfl_sync(0xffffffffu, ex, seg);
  unsigned ab;
  const unsigned bin = kth_in_segment<BPL>(hist, NB - seg * SEG, k - aseg, lane, &ab);
  *above = aseg + ab;
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
  unsigned call_par;          // parity of the handle's call number: which of the two global histograms is this call's
  unsigned ncand;
  unsigned ncand2;
  unsigned prod_seq;       // rows the producers have armed so far (for the give-up path)
  unsigned next_c;         // next channel of the batch to take in the gate/up phase
  int go;                  // the producer warps may start
  int n_mine;              // channels of this block (for the producer warps)
  int nready;              // entries of mysel that are final (the definite share first, all of them later)
  int keys_done;           // the consumer warps no longer read the keys near the end of the big buffer
  int c_done;              // ... nor the list of the threshold bin's members
  int keys_s0, keys_s1;    // ring slots [s0, s1) that overlap the keys
  int list_s0, list_s1;    // ... and the list
  unsigned slot_use[kMaxSlots];   // uses of each ring slot whose data has been seen complete
  unsigned long long pempty[kPStages];   // proxy ring: the MMAs have read the stage of warp w
  unsigned long long acc_bar;            // all MMAs of a tile are complete (one arrival per loader warp)
  uint32_t tmem_base;
  int sstart[kMaxSuper + 2];             // first kept row of every supergroup (and k1)
  int bstart[kMaxSuper + 2];             // first 32-row block of every supergroup (and the block count)
  float soff[4 * kMaxSuper];             // per scale group: code offset (8 or 128) * sum of the kept x, as integers
  int gstart[4 * kMaxSuper + 2];         // first kept row of every scale group (and k1)
  unsigned soff_cnt;                     // warps that have finished their share of soff
  unsigned wmax[32];
  float nsum[kFusedWarps][2];     // RMSNorm: the warps' sums of squares (hi, lo)
  float ninv[2];                  // ... and 1 / sqrt(mean + eps) (hi, lo)
};

// NG = warp groups of the down projection (4: d_model <= 4096, 2: <= 8192, 1: <= 16384)
// NORM = layer sub-block form (RMSNorm in the prologue, residual add at the end); THRESH = threshold
// form of the two masks (Sec. 4.1 indicators with calibrated thresholds; no k-th element search at all).
// Instantiations of their own, so that the plain call carries none of their code or registers.
template <int BITS, int NG, bool NORM = false, bool THRESH = false>
__global__ void __launch_bounds__(kFusedThreads, 1) prox_fused_kernel(const FusedParams p) {
  constexpr int CH = ProxyFmt<BITS>::CH, NACC = ProxyFmt<BITS>::NACC;
  constexpr int NT = kFusedThreads;
  extern __shared__ __align__(128) uint8_t smem_raw[];
  FusedSmem& sm = *reinterpret_cast<FusedSmem*>(smem_raw);
  const int D = p.D, F = p.F, k2 = p.k2;
  int k1 = p.k1;                         // THRESH: becomes the number of kept inputs after phase A
  uint16_t* xs = reinterpret_cast<uint16_t*>(smem_raw + ((sizeof(FusedSmem) + 127) & ~size_t(127)));
  uint16_t* idx16 = xs + D;
  float* xf = reinterpret_cast<float*>(idx16 + D);
  uint8_t* big = reinterpret_cast<uint8_t*>(xf + D);           // 128-byte aligned: D % 128 == 0
  const uint32_t big_u32 = smem_u32(big);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, cta = blockIdx.x;
  volatile int* abortp = &sm.abort_flag;
  const unsigned lt_mask = (1u << lane) - 1u;
  const unsigned spin = p.spin_limit;

  // ------------------------------------------------------------------ set-up
  PROX_TRACE(0);
  if (tid < kMaxSlots) {
    mbar_init(smem_u32(&sm.mbar_full[tid]), 1);
    mbar_init(smem_u32(&sm.mbar_empty[tid]), kEmptyCount);
    fence_mbar_init();
  }
  if (warp == 0) tmem_alloc_all(smem_u32(&sm.tmem_base));      // all 512 columns: one block per SM
  if (tid < kPStages) {
    mbar_init(smem_u32(&sm.pempty[tid]), 1);
    if (tid == 0) mbar_init(smem_u32(&sm.acc_bar), kFusedConsumerWarps);
    fence_mbar_init();
  }
  if (tid == 0) sm.soff_cnt = 0;
  if (tid == 0) { sm.abort_flag = 0; sm.ncand = 0; sm.ncand2 = 0; sm.prod_seq = 0; sm.next_c = 0; sm.go = 0; }
  if (tid < kMaxSlots) sm.slot_use[tid] = 0;
  // the launch may have been set up while the previous kernel of the stream was still draining: nothing of
  // global memory is touched before that kernel has completed
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // Two global score histograms take turns: this call adds to one and clears the other for the next call (it was
  // last used by the previous call, which has completed), so nothing is left to clean up when the call ends.
  // The call number is the barrier counter over the grid size: the counter only grows, by one per block and
  // call, and this call's own increments cannot complete a multiple of the grid size before every block has
  // passed this point (each block adds its one after phase B).
  if (tid == NT - 1) {                          // a thread with no share of the input load below
    unsigned long long bc;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(bc) : "l"(p.bar_count) : "memory");
    sm.call_par = (unsigned)((bc / (unsigned long long)G) & 1ull);
  }
  if (NORM) {
    // FFN input = bf16(RMSNorm(residual stream) * norm weight), the correctly rounded value (the masks
    // depend on it).  Every block does all of it; x and w pass through shared memory once.
    float hi = 0.f, lo = 0.f;
    {
      // both loads of a round are issued before the first use (a load per dependent iteration would put
      // the latency of global memory on every one of them)
      const float4* x4 = reinterpret_cast<const float4*>(p.xres);
      const uint2* w2 = reinterpret_cast<const uint2*>(p.norm_w);
      const int n4 = D / 4;
#pragma unroll 1
      for (int i0 = tid; i0 < n4; i0 += 2 * NT) {
        const int i1 = i0 + NT;
        const bool two = i1 < n4;
        const float4 a = __ldcg(x4 + i0);
        const uint2 wa = __ldg(w2 + i0);
        const float4 b = two ? __ldcg(x4 + i1) : make_float4(0.f, 0.f, 0.f, 0.f);
        const uint2 wb = two ? __ldg(w2 + i1) : make_uint2(0u, 0u);
        reinterpret_cast<float4*>(xf)[i0] = a;
        reinterpret_cast<uint2*>(idx16)[i0] = wa;
        f2_add_square(hi, lo, a.x); f2_add_square(hi, lo, a.y); f2_add_square(hi, lo, a.z); f2_add_square(hi, lo, a.w);
        if (two) {
          reinterpret_cast<float4*>(xf)[i1] = b;
          reinterpret_cast<uint2*>(idx16)[i1] = wb;
          f2_add_square(hi, lo, b.x); f2_add_square(hi, lo, b.y); f2_add_square(hi, lo, b.z); f2_add_square(hi, lo, b.w);
        }
      }
    }
    for (int i = tid; i < 1024 + 32; i += NT) { if (i < 1024) sm.hist[i] = 0; else sm.hist2[i - 1024] = 0; }
    f2_warp_sum(hi, lo);
    if (lane == 0) { sm.nsum[warp][0] = hi; sm.nsum[warp][1] = lo; }
    __syncthreads();
    if (warp == 0) {
      hi = lane < kFusedWarps ? sm.nsum[lane][0] : 0.f;
      lo = lane < kFusedWarps ? sm.nsum[lane][1] : 0.f;
      f2_warp_sum(hi, lo);
      if (lane == 0) rms_inverse(hi, lo, p.rc, sm.ninv[0], sm.ninv[1]);
    }
    __syncthreads();
    const float ih = sm.ninv[0], il = sm.ninv[1];
#pragma unroll 1
    for (int i = tid; i < D; i += NT) {
      const uint16_t b = rms_scale_to_bf16(xf[i], __uint_as_float((uint32_t)idx16[i] << 16), ih, il);
      xs[i] = b;
      xf[i] = __uint_as_float((uint32_t)b << 16);
    }
  } else {
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
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  unsigned* const ghist = p.ghist + 2048u * sm.call_par;
  {
    unsigned* const other = p.ghist + 2048u * (sm.call_par ^ 1u);
    const int per = (2048 + G - 1) / G;
    for (int i = cta * per + tid; i < min(2048, (cta + 1) * per); i += NT) other[i] = 0u;
  }
  if (warp < 4) {
    // the accumulators of the proxy GEMV start at zero: 16 columns per supergroup, two sets 256 columns apart
    const int ngz = (p.gshift >= 31) ? 1 : (D >> p.gshift);
    const uint32_t tz = sm.tmem_base + ((uint32_t)(warp * 32) << 16);
#pragma unroll 1
    for (int c = 0; c < 16 * ((ngz + 3) >> 2); c += 16) { tmem_st16_zero(tz + (uint32_t)c); tmem_st16_zero(tz + 256u + (uint32_t)c); }
    tmem_st_wait();
    tc_fence_before();
  }
  PROX_TRACE(1);

  // ------------------------------------------------- A: input mask (top-k1 of |x|)
  int ebase = 1;
  const bool per_row_a = p.gshift >= 31;
  {
    const uint32_t* xs32 = reinterpret_cast<const uint32_t*>(xs);
    const bool all = THRESH ? (p.tkey_x == 0u) : (k1 >= D);
    unsigned T = 0, quota = 0;
    if (THRESH) {
      T = p.tkey_x - 1u;                 // kept: key > T, i.e. |x| >= tau_x; no ties to ration
    } else if (!all) {
      // level 1: the top 10 of the 15 key bits; level 2: the other 5
#pragma unroll 1
      for (int i = tid; i < D / 2; i += NT) {
        const uint32_t w = xs32[i];
        atomicAdd(&sm.hist[(w >> 5) & 0x3ffu], 1u);
        atomicAdd(&sm.hist[(w >> 21) & 0x3ffu], 1u);
      }
      __syncthreads();
      PROX_TRACE(10);
      unsigned above1;
      const unsigned bin1 = kth_in_block<2, false>(sm.hist, (unsigned)k1, sm.wsum, lane, warp, &above1);
      PROX_TRACE(11);
      // Inputs whose magnitude lies in a bin above the threshold bin are kept whatever the exact threshold:
      // their packed proxy rows are pulled into L2 now (every block a share of them, one bulk prefetch per
      // row), a few microseconds before the proxy GEMV asks for them.
      if (warp >= kFusedConsumerWarps) {
        const size_t prow = (size_t)(F / CH) * 16;
#pragma unroll 1
        for (int i = cta + (tid - kFusedConsumers) * G; i < D; i += G * 32 * kFusedProducers)
          if ((((unsigned)xs[i] & 0x7fffu) >> 5) > bin1)
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p.P + (size_t)i * prow), "r"((uint32_t)prow) : "memory");
      }
#pragma unroll 1
      for (int i = tid; i < D / 2; i += NT) {
        const uint32_t w = xs32[i];
        const unsigned ka = w & 0x7fffu, kb = (w >> 16) & 0x7fffu;
        if ((ka >> 5) == bin1) atomicAdd(&sm.hist2[ka & 31u], 1u);
        if ((kb >> 5) == bin1) atomicAdd(&sm.hist2[kb & 31u], 1u);
      }
      __syncthreads();
      PROX_TRACE(12);
      unsigned above2;
      const unsigned bin2 = kth_in_segment<1>(sm.hist2, 32, (unsigned)k1 - above1, lane, &above2);
      T = (bin1 << 5) | bin2;
      quota = (unsigned)k1 - above1 - above2;      // ties at T to accept, lowest index first
      PROX_TRACE(13);
    }
    // Ordered compaction: a consumer thread owns a run of 8-input groups, counts its kept
    // inputs and its ties (packed in one word), and places them behind those of the threads
    // in front (one warp scan plus the totals of the warps in front).
    const int ngrp = D / 8, gpt = (ngrp + kFusedConsumers - 1) / kFusedConsumers;
    const int g0 = min(ngrp, tid * gpt), g1 = (tid < kFusedConsumers) ? min(ngrp, g0 + gpt) : g0;
    unsigned cnt = 0, mk = 0;
#pragma unroll 1
    for (int g = g0; g < g1; ++g) {
      const uint4 kv = *reinterpret_cast<const uint4*>(xs + g * 8);
      const uint32_t w4[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const unsigned key = (w4[e >> 1] >> ((e & 1) * 16)) & 0x7fffu;
        cnt += ((all || key > T) ? 1u : 0u) | ((!all && key == T) ? 0x10000u : 0u);
        mk = max(mk, key);
      }
    }
    const unsigned inc = warp_scan_incl(cnt, lane);
    mk = __reduce_max_sync(0xffffffffu, mk);
    if (lane == 31) { sm.wsum[warp] = inc; sm.wmax[warp] = mk; }
    __syncthreads();
    PROX_TRACE(14);
    mk = __reduce_max_sync(0xffffffffu, (lane < kFusedWarps) ? sm.wmax[lane] : 0u);
    ebase = max(max((int)(mk >> 7), 1) - 22, 1);
    if (THRESH) {
      k1 = (int)__reduce_add_sync(0xffffffffu, (lane < kFusedWarps) ? (sm.wsum[lane] & 0xffffu) : 0u);
      if (cta == 0 && tid == 0) {
        if (p.cnt_x_out) p.cnt_x_out[0] = k1;
        if (p.counters) { atomicAdd(p.counters, 1ull); atomicAdd(p.counters + 1, (unsigned long long)k1); }
      }
    }
    {
      const unsigned ex = __reduce_add_sync(0xffffffffu, (lane < warp) ? sm.wsum[lane] : 0u) + inc - cnt;
      unsigned rg = ex & 0xffffu, re = ex >> 16;
      // (also, for the proxy GEMV: where every scale group starts in the list)
      const int gmask = per_row_a ? 0x7fffffff : ((1 << p.gshift) - 1);
#pragma unroll 1
      for (int g = g0; g < g1; ++g) {
        const uint4 kv = *reinterpret_cast<const uint4*>(xs + g * 8);
        const uint32_t w4[4] = {kv.x, kv.y, kv.z, kv.w};
        if (((g * 8) & gmask) == 0) sm.gstart[per_row_a ? 0 : ((g * 8) >> p.gshift)] = (int)(rg + min(re, quota));
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const unsigned key = (w4[e >> 1] >> ((e & 1) * 16)) & 0x7fffu;
          const bool gt = all || key > T, eq = !all && key == T;
          if (gt || (eq && re < quota)) idx16[rg + min(re, quota)] = (uint16_t)(g * 8 + e);
          rg += gt ? 1u : 0u; re += eq ? 1u : 0u;
        }
      }
    }
    if (tid == 0) sm.gstart[per_row_a ? 1 : (D >> p.gshift)] = k1;
    __syncthreads();
  }

  if (cta == 0 && p.idx_out) {
#pragma unroll 1
    for (int i = tid; i < k1; i += NT) p.idx_out[i] = (int)idx16[i];
  }
  PROX_TRACE(2);
  // --------------------------------------- B: proxy GEMV (tensor cores), scores, score histogram
  // Per scale group g:  sum_k x_k q_kj = 2^(ebase-134) * sum_k X_k (byte_kj - offset), X_k the integer
  // form of x_k (x_digits).  A block owns 128-byte tiles of the packed rows over all kept rows.  The kept
  // rows are cut into blocks of at most 32 rows that stay inside one supergroup (4 scale groups); block b
  // accumulates into 16 tensor-memory columns of its supergroup: column 4 * (g % 4) + d holds digit d of
  // group g.  16 loader warps bring the rows in with plain 16-byte loads (8 in flight per lane) and store
  // them (and the bytes with the high nibble masked off, and the digits of x) in a stage of the ring;
  // one thread issues the MMAs; after the last one the 16 warps read the accumulators, apply the
  // groups' scales and form the scores.
  {
    constexpr bool LO = (BITS == 4);
    const int nchunks = F / CH;
    const int row_bytes = nchunks * 16;
    const int ntiles = (row_bytes + 127) >> 7;
    const bool per_row = p.gshift >= 31;
    const int ng = per_row ? 1 : (D >> p.gshift);
    const int nsuper = (ng + 3) >> 2;
    const int sgshift = per_row ? 31 : p.gshift + 2;
    const uint32_t tbase = sm.tmem_base;
    // supergroup starts and blocks (one warp), the groups' offsets, the block's own score histogram
    if (warp == 0) {
      const int r0s = sm.gstart[min(4 * lane, ng)], r1s = sm.gstart[min(4 * lane + 4, ng)];
      const unsigned nb = lane < nsuper ? (unsigned)((r1s - r0s + 31) >> 5) : 0u;
      const unsigned incb = warp_scan_incl(nb, lane);
      if (lane <= nsuper) { sm.sstart[lane] = r0s; sm.bstart[lane] = (int)(incb - nb); }
    }
#pragma unroll 1
    for (int i = tid; i < 512; i += NT) reinterpret_cast<uint4*>(sm.hist)[i] = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();
    const int nblk = sm.bstart[nsuper];
    const uint32_t ring = (big_u32 + 1023u) & ~1023u;
    float* red = reinterpret_cast<float*>(big + (ring - big_u32) + (uint32_t)(kPStages * kPStageBytes));   // [3][128][2] partial sums of warps 4..15
    PROX_TRACE(29);
    if (warp < kFusedConsumerWarps) {
      // a warp owns one stage of the ring: it fills it and issues the stage's MMAs itself (the tensor core
      // takes accumulating MMAs from several threads into the same columns; integer sums do not depend on the order)
      const uint32_t stg = ring + (uint32_t)warp * (uint32_t)kPStageBytes;
      const uint64_t adesc = umma_smem_desc(stg, 4096u, 1024u, 2u);
      const uint64_t ldesc = umma_smem_desc(stg + 4096u, 4096u, 1024u, 2u);
      const uint64_t bdesc = umma_smem_desc(stg + 8192u, 128u, 512u, 0u);
      constexpr uint32_t idesc = umma_idesc_u8s8(128, 16);
      const uint32_t my_empty = smem_u32(&sm.pempty[warp]);
      const int q4 = warp & 3, part = warp >> 2;
      const int col = q4 * 32 + lane;                          // byte column of the tile = data path lane
      const int c = lane & 7, kq = lane >> 3;
      unsigned uses = 0;                                       // stages this warp has handed to the tensor core
      int tile_iter = 0;
#pragma unroll 1
      for (int tile = cta; tile < ntiles; tile += G, ++tile_iter) {
        // ---- scales of this thread's byte column for the groups it will read back
        const int chunk = tile * 8 + (col >> 4);
        const bool col_ok = chunk < nchunks;
        const bool c_ok = tile * 8 + c < nchunks;
        bool alive_b = true;
        int sg = 0;
#pragma unroll 1
        for (int b = warp; b < nblk; b += kFusedConsumerWarps) {
          while (sm.bstart[sg + 1] <= b) ++sg;
          const int r0 = sm.sstart[sg] + ((b - sm.bstart[sg]) << 5);
          const int nrows = min(32, sm.sstart[sg + 1] - r0);
          uint4 v[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int kk = j * 4 + kq;
            v[j] = make_uint4(0u, 0u, 0u, 0u);
            if (kk < nrows && c_ok)
              v[j] = ld_stream(p.P + (size_t)idx16[r0 + kk] * (size_t)row_bytes + (size_t)tile * 128 + (size_t)c * 16);
          }
          if (b == 0) PROX_TRACE(22);
          uint4 brow = make_uint4(0u, 0u, 0u, 0u);
          if (lane < nrows) {
            const int i = idx16[r0 + lane];
            const uint32_t dg = x_digits(xs[i], ebase);
            const int slot = per_row ? 0 : ((i >> p.gshift) & 3);
            brow.x = slot == 0 ? dg : 0u; brow.y = slot == 1 ? dg : 0u; brow.z = slot == 2 ? dg : 0u; brow.w = slot == 3 ? dg : 0u;
          }
          const bool free_ok = uses == 0 || mbar_wait(my_empty, (uses - 1u) & 1u, abortp, spin);
          if (!__all_sync(0xffffffffu, free_ok)) { alive_b = false; break; }
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int kk = j * 4 + kq;
            const uint32_t dst = stg + (uint32_t)((kk >> 3) * 1024 + (kk & 7) * 128 + ((c ^ (kk & 7)) << 4));
            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(dst), "r"(v[j].x), "r"(v[j].y), "r"(v[j].z), "r"(v[j].w) : "memory");
            if (LO)
              asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(dst + 4096u), "r"(v[j].x & 0x0f0f0f0fu), "r"(v[j].y & 0x0f0f0f0fu),
                           "r"(v[j].z & 0x0f0f0f0fu), "r"(v[j].w & 0x0f0f0f0fu) : "memory");
          }
          asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(stg + 8192u + (uint32_t)lane * 16u), "r"(brow.x), "r"(brow.y), "r"(brow.z), "r"(brow.w) : "memory");
          fence_proxy_async();                 // the tensor core reads the stage through the async proxy
          __syncwarp();
          if (elect_one()) {
            umma_i8(tbase + (uint32_t)(16 * sg), adesc, bdesc, idesc, 1u);
            if (LO) umma_i8(tbase + 256u + (uint32_t)(16 * sg), ldesc, bdesc, idesc, 1u);
            umma_commit(my_empty);
          }
          __syncwarp();
          ++uses;
          if (b == 0) PROX_TRACE(23);
        }
        if (elect_one()) umma_commit(smem_u32(&sm.acc_bar));   // one arrival per warp once its MMAs are complete
        __syncwarp();
        PROX_TRACE(24);
        // ---- read the accumulators back: thread = byte column, warp part p takes supergroups p, p + 4, ...
        // (the four groups' scales of this byte column: gate / up scales sit in the order of the bytes)
        auto load_scales = [&](int sgq, uint32_t* dst) {
#pragma unroll
          for (int gq = 0; gq < 4; ++gq) {
            const int g = 4 * sgq + gq;
            dst[gq] = 0u;
            if (col_ok && g < ng) {
              if (LO) dst[gq] = __ldg(reinterpret_cast<const uint32_t*>(p.S + ((size_t)g * nchunks + chunk) * 32) + (col & 15));
              else dst[gq] = (uint32_t)__ldg(reinterpret_cast<const uint16_t*>(p.S + ((size_t)g * nchunks + chunk) * 16) + (col & 15));
            }
          }
        };
        uint32_t scn[4];
        load_scales(part, scn);
        const bool acc_ok = __all_sync(0xffffffffu, alive_b && mbar_wait(smem_u32(&sm.acc_bar), (unsigned)tile_iter & 1u, abortp, spin));
        tc_fence_after();
        if (tile_iter == 0) {                  // the groups' offsets come from the four warps that do not load
#pragma unroll 1
          for (unsigned it = 0; *reinterpret_cast<volatile unsigned*>(&sm.soff_cnt) < (unsigned)kFusedProducers && it < spin; ++it) __nanosleep(32);
          __threadfence_block();
        }
        PROX_TRACE(25);
        float t0 = 0.f, t1 = 0.f;              // 4-bit: sums of the low / high nibble's channel; 8-bit: t0 only
        const bool more = tile + G < ntiles;
#pragma unroll 1
        for (int sgd = part; sgd < nsuper; sgd += 4) {
          if (!acc_ok) break;
          uint32_t a[16], l[16];
          const uint32_t ta = tbase + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(16 * sgd);
          tmem_ld16(ta, a);
          if (LO) tmem_ld16(ta + 256u, l);
          uint32_t sc4[4];
#pragma unroll
          for (int gq = 0; gq < 4; ++gq) sc4[gq] = scn[gq];
          load_scales(sgd + 4, scn);           // the next round's scales are on their way during this one
          tmem_ld_wait();
          if (more) { tmem_st16_zero(ta); if (LO) tmem_st16_zero(ta + 256u); }
#pragma unroll
          for (int gq = 0; gq < 4; ++gq) {
            const int g = 4 * sgd + gq;
            const float off = sm.soff[min(g, ng - 1)];
            const float fa = digits_to_float(a[4 * gq], a[4 * gq + 1], a[4 * gq + 2], a[4 * gq + 3]);
            if (LO) {
              const float fl = digits_to_float(l[4 * gq], l[4 * gq + 1], l[4 * gq + 2], l[4 * gq + 3]);
              const float2 sc = __half22float2(*reinterpret_cast<const __half2*>(&sc4[gq]));
              t0 = fmaf(sc.x, fl - off, t0);
              t1 = fmaf(sc.y, fmaf(fa - fl, 0.0625f, -off), t1);
            } else {
              const float sc = __half2float(__ushort_as_half((unsigned short)sc4[gq]));
              t0 = fmaf(sc, fa - off, t0);
            }
          }
        }
        PROX_TRACE(26);
        if (more) { tmem_st_wait(); tc_fence_before(); }
        if (part > 0) { red[((part - 1) * 128 + col) * 2] = t0; red[((part - 1) * 128 + col) * 2 + 1] = t1; }
        consumer_sync();
        if (more) tc_fence_after();            // every warp's columns are back at zero before the next tile's MMAs
        if (part == 0) {
#pragma unroll
          for (int pp = 0; pp < 3; ++pp) { t0 += red[(pp * 128 + col) * 2]; t1 += red[(pp * 128 + col) * 2 + 1]; }
          t0 = scalbnf(t0, ebase - 134); t1 = scalbnf(t1, ebase - 134);
          // bytes 0..7 of a chunk hold gate codes, bytes 8..15 the up codes of the same channels
          const float u0 = __shfl_xor_sync(0xffffffffu, t0, 8), u1 = __shfl_xor_sync(0xffffffffu, t1, 8);
          if ((col & 8) == 0 && col_ok) {
            if (LO) {
              const int ch = chunk * 16 + 2 * (col & 7);
              const float s0 = fabsf(u0 * silu_fast(t0)), s1 = fabsf(u1 * silu_fast(t1));
              __stcg(reinterpret_cast<float2*>(p.scores + ch), make_float2(s0, s1));
              atomicAdd(&sm.hist[__float_as_uint(s0) >> 20], 1u);
              atomicAdd(&sm.hist[__float_as_uint(s1) >> 20], 1u);
            } else {
              const int ch = chunk * 8 + (col & 7);
              const float s0 = fabsf(u0 * silu_fast(t0));
              __stcg(p.scores + ch, s0);
              atomicAdd(&sm.hist[__float_as_uint(s0) >> 20], 1u);
            }
          }
        }
        if (more) consumer_sync();             // red is free again
      }
      // nothing may be in flight when the block frees the tensor memory (only a block whose wait expired gets here early)
      if (sm.abort_flag && lane == 0) {
#pragma unroll 1
        for (unsigned it = 0; it < 65536u && uses > 0; ++it) {
          if (mbar_try_wait(my_empty, (uses - 1u) & 1u)) break;
          __nanosleep(64);
        }
      }
    }
    else {
      // Blocks without a tile pull the kept rows into L2 (whole rows, one bulk prefetch each): the loader
      // warps of the other blocks then find them there instead of waiting for HBM one by one.
      if (cta >= ntiles && lane < 8) {
        const int nidle = G - ntiles, slot_i = (cta - ntiles) * (kFusedProducers * 8) + (warp - kFusedConsumerWarps) * 8 + lane;
#pragma unroll 1
        for (int r = slot_i; r < k1; r += nidle * kFusedProducers * 8)
          asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p.P + (size_t)idx16[r] * (size_t)row_bytes), "r"((uint32_t)row_bytes) : "memory");
      }
      // the other four warps: per scale group, offset * sum of the kept x as integers (for the codes' offset binary)
#pragma unroll 1
      for (int g = warp - kFusedConsumerWarps; g < ng; g += kFusedProducers) {
        int d0 = 0, d1 = 0, d2 = 0, d3 = 0;
#pragma unroll 1
        for (int r = sm.gstart[g] + lane; r < sm.gstart[g + 1]; r += 32) {
          const uint32_t dg = x_digits(xs[idx16[r]], ebase);
          d0 += (int)(int8_t)(dg & 0xffu); d1 += (int)(int8_t)((dg >> 8) & 0xffu);
          d2 += (int)(int8_t)((dg >> 16) & 0xffu); d3 += (int)(int8_t)(dg >> 24);
        }
        d0 = __reduce_add_sync(0xffffffffu, d0); d1 = __reduce_add_sync(0xffffffffu, d1);
        d2 = __reduce_add_sync(0xffffffffu, d2); d3 = __reduce_add_sync(0xffffffffu, d3);
        if (lane == 0) sm.soff[g] = (LO ? 8.f : 128.f) * digits_to_float((uint32_t)d0, (uint32_t)d1, (uint32_t)d2, (uint32_t)d3);
      }
      __syncwarp();
      if (lane == 0) { __threadfence_block(); atomicAdd(&sm.soff_cnt, 1u); }
    }
    // the tensor memory is not used after this phase
    tc_fence_before();
    __syncthreads();
    if (cta < ntiles) {
      // one atomic per occupied bin and block (thousands of single increments on a few hot bins serialise in L2)
#pragma unroll 1
      for (int i = tid; i < 2048; i += NT) { const unsigned v = sm.hist[i]; if (v) atomicAdd(ghist + i, v); }
    }
    if (warp == 0) tmem_free_all(tbase);
  }

  PROX_TRACE(3);
  // -------------------------------------------------------------- grid barrier
  // One counter that only grows: a block adds 1 and waits until the count
  // reaches the next multiple of the grid size (no reset, no generation word).
  fence_proxy_async();                        // phase B's plain accesses to the big buffer come before the ring's bulk copies
  __syncthreads();
  if (tid == 0) {
    // release (cumulative): publishes the block's writes seen through the barrier above
    unsigned long long old;
    asm volatile("atom.acq_rel.gpu.global.add.u64 %0, [%1], 1;" : "=l"(old) : "l"(p.bar_count) : "memory");
    // the count is reset by the host long before 2^32 calls; the low word is enough for the division
    const unsigned long long target = old - (unsigned long long)((unsigned)old % (unsigned)G) + (unsigned long long)G +
                                      (unsigned long long)p.bar_bias;
    bool ok = (old + 1ull == target);
#pragma unroll 1
    for (unsigned it = 0; !ok && it < spin; ++it) {
      unsigned long long cur;
      asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(cur) : "l"(p.bar_count) : "memory");
      ok = cur >= target;
      if (!ok && it > 64) __nanosleep(32);
    }
    if (!ok) { sm.abort_flag = 1; atomicOr(p.status, kWaitExpired); if (p.host_flag) *reinterpret_cast<volatile int*>(p.host_flag) = 1; }
  }
  __syncthreads();
  const bool alive = sm.abort_flag == 0;      // block-uniform; a dead block skips to the end
  PROX_TRACE(4);

  // ---------------------------------------- C: channel mask (top-k2 of the scores)
  // The first histogram level tells which channels are kept whatever the exact
  // threshold turns out to be (their bin lies above the threshold bin b1:
  // "definite", nd of them) and which are still open (the nb1 members of b1).
  // The kept list is laid out as [definite, ascending][kept members of b1,
  // ascending]; block c owns the c-th share of either part.  Its definite share
  // is known after two passes over the scores, so its weight rows start to stream
  // while the consumer warps still settle the threshold inside b1.
  int n_mine = 0;
  if (alive && warp < kFusedConsumerWarps) {          // the producer warps wait at the ring for the go flag
    // Shared-memory plan: the keys (score bits) sit at the END of the big buffer (the ring fills
    // from slot 0 and reaches those slots last); the ascending list of b1's members goes where
    // the input index list was (free since phase B), or in front of the keys if it is long.
    const bool in_smem = (size_t)F * 4 + 256 <= (size_t)p.big_bytes;
    const uint32_t key_off = in_smem ? (((uint32_t)p.big_bytes - (uint32_t)F * 4u) & ~127u) : 0u;
    const uint32_t skey_u32 = big_u32 + key_off;
    const unsigned* gkey = reinterpret_cast<const unsigned*>(p.scores);
    auto key_at = [&](int i) -> unsigned {
      unsigned v;
      if (in_smem) asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(skey_u32 + (uint32_t)i * 4u));
      else v = __ldcg(gkey + i);
      return v;
    };
    auto key4_at = [&](int i) -> uint4 {                  // i % 4 == 0
      return in_smem ? lds128(skey_u32 + (uint32_t)i * 4u) : __ldcg(reinterpret_cast<const uint4*>(gkey + i));
    };
    if (!THRESH && tid < 512) cp_async16(smem_u32(sm.hist) + (uint32_t)tid * 16u, ghist + tid * 4);
    cp_async_commit();
    if (in_smem) {
#pragma unroll 1
      for (int i = tid; i < F / 4; i += kFusedConsumers) cp_async16(skey_u32 + (uint32_t)i * 16u, gkey + 4 * i);
    }
    cp_async_commit();
    if (tid < 256) sm.hist2[tid] = 0;
    cp_async_wait<1>();                                    // the histogram (the keys may still be on their way)
    consumer_sync();
    PROX_TRACE(16);
    unsigned nd = 0;                                       // channels above bin b1 (THRESH: at or above tau_s)
    unsigned b1 = 0, kk = 0, nb1 = 0;
    if (!THRESH) {
      b1 = kth_in_block<4, true>(sm.hist, (unsigned)k2, sm.wsum, lane, warp, &nd);
      kk = (unsigned)k2 - nd;                              // members of b1 to keep (>= 1)
      nb1 = sm.hist[b1];
    }
    uint32_t list_u32 = smem_u32(idx16);                   // 2 * D bytes: room for D / 4 members
    uint32_t list_off = 0;                                 // offset in the big buffer when it has to go there
    bool list_in_big = false;
    bool staged = in_smem;                                 // the same in every block
    if (in_smem && (size_t)nb1 * 8 > (size_t)D * 2) {
      if ((size_t)nb1 * 8 + 128 <= (size_t)key_off) {
        list_off = (key_off - nb1 * 8u) & ~127u; list_u32 = big_u32 + list_off; list_in_big = true;
      } else {
        staged = false;
      }
    }
    const int per = ((F + 32 * kFusedConsumerWarps - 1) / (32 * kFusedConsumerWarps)) * 32;        // channels per warp run (slow path)
    const int i0 = min(F, warp * per), i1 = min(F, i0 + per);
    cp_async_wait<0>();
    PROX_TRACE(17);
    consumer_sync();                                       // the keys are there for everyone; wsum is free again
    if (staged) {
      // k2 * G < 2^31 is checked on the host, so the share bounds fit 32 bits
      // (THRESH: nd is only known after the counting pass; the bounds are set there)
      int Rd0 = (int)((nd * (unsigned)cta) / (unsigned)G);
      const int Rc0 = (int)((kk * (unsigned)cta) / (unsigned)G);
      int ndm = min((int)((nd * (unsigned)(cta + 1)) / (unsigned)G) - Rd0, kMySelCap);
      const int ncm = THRESH ? 0 : min((int)((kk * (unsigned)(cta + 1)) / (unsigned)G) - Rc0, kMySelCap - ndm);
      int Rd1 = Rd0 + ndm;
      const int Rc1 = Rc0 + ncm;
      n_mine = ndm + ncm;
      // pass 1: a consumer thread owns a run of 4-channel groups and counts its definite
      // channels and its members of b1 (packed in one word); one warp scan, warp totals
      const int nq = F / 4, qpt = (nq + kFusedConsumers - 1) / kFusedConsumers;
      const int q0 = min(nq, tid * qpt), q1 = (tid < kFusedConsumers) ? min(nq, q0 + qpt) : q0;
      // (with up to 64 channels per thread it also keeps them as two bit masks, so that the later
      // passes walk set bits instead of reading and comparing the scores again)
      const bool masks = qpt <= 16;
      unsigned dm[2] = {0u, 0u}, cm[2] = {0u, 0u};           // channels 0..31 and 32..63 of the thread's run
      unsigned cnt = 0;
#pragma unroll 1
      for (int q = q0; q < q1; ++q) {
        const uint4 kv = key4_at(q * 4);
        const unsigned k4[4] = {kv.x, kv.y, kv.z, kv.w};
        unsigned d4 = 0, c4 = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (THRESH) {
            d4 |= ((k4[e] >= p.tkey_s) ? 1u : 0u) << e;
          } else {
            const unsigned bin = k4[e] >> 20;
            d4 |= ((bin > b1) ? 1u : 0u) << e;
            c4 |= ((bin == b1) ? 1u : 0u) << e;
          }
        }
        cnt += (unsigned)__popc(d4) | ((unsigned)__popc(c4) << 16);
        if (masks) {
          const int rel = q - q0, sh = (rel & 7) * 4;
          if (rel < 8) { dm[0] |= d4 << sh; cm[0] |= c4 << sh; } else { dm[1] |= d4 << sh; cm[1] |= c4 << sh; }
        }
      }
      const unsigned inc = warp_scan_incl(cnt, lane);
      if (lane == 31) sm.wsum[warp] = inc;
      if (THRESH) {
        consumer_sync();                                   // the warps' totals: how many channels are kept
        nd = __reduce_add_sync(0xffffffffu, (lane < kFusedConsumerWarps) ? (sm.wsum[lane] & 0xffffu) : 0u);
        Rd0 = (int)((nd * (unsigned)cta) / (unsigned)G);
        ndm = min((int)((nd * (unsigned)(cta + 1)) / (unsigned)G) - Rd0, kMySelCap);
        Rd1 = Rd0 + ndm;
        n_mine = ndm;
        if (cta == 0 && tid == 0) {
          if (p.count_out) p.count_out[0] = (int)nd;
          if (p.counters) atomicAdd(p.counters + 2, (unsigned long long)nd);
        }
      }
      if (tid == 0) {
        const uint32_t rb = (uint32_t)D * 2u;
        sm.keys_s0 = (int)(key_off / rb); sm.keys_s1 = (int)((key_off + (uint32_t)F * 4u + rb - 1u) / rb);
        sm.list_s0 = list_in_big ? (int)(list_off / rb) : 0;
        sm.list_s1 = list_in_big ? (int)((list_off + nb1 * 8u + rb - 1u) / rb) : 0;
        sm.n_mine = n_mine; sm.nready = ndm; sm.keys_done = (ncm == 0) ? 1 : 0; sm.c_done = (ncm == 0) ? 1 : 0;
      }
      consumer_sync();
      PROX_TRACE(18);
      // pass 2: the threads whose definite channels meet the block's share write them out
      const unsigned ex = __reduce_add_sync(0xffffffffu, (lane < warp) ? sm.wsum[lane] : 0u) + inc - cnt;
      {
        int dpos = (int)(ex & 0xffffu);
        const int cdef = (int)(cnt & 0xffffu);
        if (masks && cdef > 0 && dpos < Rd1 && dpos + cdef > Rd0) {
#pragma unroll 1
          for (int hw = 0; hw < 2; ++hw) {
#pragma unroll 1
            for (unsigned m = dm[hw]; m; m &= m - 1) {
              if (dpos >= Rd0 && dpos < Rd1) {
                const int ch = q0 * 4 + hw * 32 + __ffs((int)m) - 1;
                sm.mysel[dpos - Rd0] = ch;
                if (p.sel_out) p.sel_out[dpos] = ch;
              }
              ++dpos;
            }
          }
        } else if (cdef > 0 && dpos < Rd1 && dpos + cdef > Rd0) {
#pragma unroll 1
          for (int q = q0; q < q1; ++q) {
            const uint4 kv = key4_at(q * 4);
            const unsigned k4[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              if (THRESH ? (k4[e] >= p.tkey_s) : ((k4[e] >> 20) > b1)) {
                if (dpos >= Rd0 && dpos < Rd1) {
                  sm.mysel[dpos - Rd0] = q * 4 + e;
                  if (p.sel_out) p.sel_out[dpos] = q * 4 + e;
                }
                ++dpos;
              }
            }
          }
        }
      }
      __threadfence_block();
      consumer_sync();                          // the definite share is listed
      if (tid == 0) *reinterpret_cast<volatile int*>(&sm.go) = 1;      // the producer warps leave for the ring
      PROX_TRACE(21);
      if (ncm > 0 && warp < kFusedConsumerWarps) {
        // ---- consumer warps only (named barrier): list b1's members in channel order ...
        const uint32_t lkey_u32 = list_u32, lidx_u32 = lkey_u32 + nb1 * 4u;
        auto lds32 = [](uint32_t a) -> unsigned { unsigned v; asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a)); return v; };
        auto sts32 = [](uint32_t a, unsigned v) { asm volatile("st.shared.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory"); };
        if (masks) {
          unsigned cpos = ex >> 16;
#pragma unroll 1
          for (int hw = 0; hw < 2; ++hw) {
#pragma unroll 1
            for (unsigned m = cm[hw]; m; m &= m - 1) {
              const int ch = q0 * 4 + hw * 32 + __ffs((int)m) - 1;
              if (cpos < nb1) { sts32(lkey_u32 + cpos * 4u, key_at(ch)); sts32(lidx_u32 + cpos * 4u, (unsigned)ch); }
              ++cpos;
            }
          }
        } else if (cnt >> 16) {
          unsigned cpos = ex >> 16;
#pragma unroll 1
          for (int q = q0; q < q1; ++q) {
            const uint4 kv = key4_at(q * 4);
            const unsigned k4[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              if ((k4[e] >> 20) == b1) {
                if (cpos < nb1) { sts32(lkey_u32 + cpos * 4u, k4[e]); sts32(lidx_u32 + cpos * 4u, (unsigned)(q * 4 + e)); }
                ++cpos;
              }
            }
          }
        }
        // The upper half of the consumer warps goes on to the gate/up rows that are streaming in
        // already; the lower half ("settlers") finishes the mask and joins them later.
        if (warp >= kSettlerWarps) {
          asm volatile("bar.arrive 2, %0;" ::"n"(kFusedConsumers) : "memory");
        } else {
        asm volatile("bar.sync 2, %0;" ::"n"(kFusedConsumers) : "memory");      // the list is complete, the keys are free
        if (tid == 0) *reinterpret_cast<volatile int*>(&sm.keys_done) = 1;
        PROX_TRACE(15);
        // ... settle the threshold inside b1: histogram of bits 19..12, then the few left ...
#pragma unroll 1
        for (unsigned c = tid; c < nb1; c += kSettlers)
          atomicAdd(&sm.hist2[(lds32(lkey_u32 + c * 4u) >> 12) & 255u], 1u);
        settler_sync();
        unsigned above2;
        const unsigned b2 = kth_in_segment<8>(sm.hist2, 256, kk, lane, &above2);     // every warp on its own
        unsigned kk2 = kk - above2;
        const unsigned pre2 = (b1 << 8) | b2;
#pragma unroll 1
        for (unsigned c = tid; c < nb1; c += kSettlers) {
          const unsigned key = lds32(lkey_u32 + c * 4u);
          if ((key >> 12) == pre2) {
            const unsigned slot = atomicAdd(&sm.ncand2, 1u);
            if (slot < (unsigned)kCand2Cap) { sm.cand2_key[slot] = key; sm.cand2_idx[slot] = (int)lds32(lidx_u32 + c * 4u); }
          }
        }
        settler_sync();
        const unsigned n2 = sm.ncand2;
        PROX_TRACE(19);
        unsigned T, quota;
        if (n2 <= (unsigned)kCand2Cap) {
          // rank the few that are left by (score descending, channel ascending)
          if (tid < (int)n2) {
            const unsigned key = sm.cand2_key[tid];
            const int id = sm.cand2_idx[tid];
            unsigned rank = 0, same_before = 0;
#pragma unroll 1
            for (unsigned c = 0; c < n2; ++c) {
              const unsigned ok = sm.cand2_key[c];
              const int oi = sm.cand2_idx[c];
              rank += (ok > key || (ok == key && oi < id)) ? 1u : 0u;
              same_before += (ok == key && oi < id) ? 1u : 0u;
            }
            if (rank == kk2 - 1u) { sm.res[2] = key; sm.res[3] = same_before + 1u; }
          }
          settler_sync();
          T = sm.res[2]; quota = sm.res[3];
        } else {
          // many scores agree in their top 20 bits: two more radix steps of 6 bits over the list
          unsigned prefix = pre2;
#pragma unroll 1
          for (int sh = 6; sh >= 0; sh -= 6) {
            settler_sync();                               // everyone is done with the previous histogram
            if (tid < 64) sm.hist2[tid] = 0;
            settler_sync();
#pragma unroll 1
            for (unsigned c = tid; c < nb1; c += kSettlers) {
              const unsigned key = lds32(lkey_u32 + c * 4u);
              if ((key >> (sh + 6)) == prefix) atomicAdd(&sm.hist2[(key >> sh) & 63u], 1u);
            }
            settler_sync();
            unsigned ab;
            const unsigned bb = kth_in_segment<2>(sm.hist2, 64, kk2, lane, &ab);
            prefix = (prefix << 6) | bb;
            kk2 -= ab;
          }
          T = prefix; quota = kk2;
        }
        PROX_TRACE(20);
        // ... and keep the block's share of the members above T plus the first `quota` ties at T:
        // a thread owns a run of the list, counts first (packed in one word), then the places
        const int ept = ((int)nb1 + kSettlers - 1) / kSettlers;
        const int c0 = min((int)nb1, tid * ept), c1 = min((int)nb1, c0 + ept);
        unsigned wt = 0;
#pragma unroll 1
        for (int c = c0; c < c1; ++c) {
          const unsigned key = lds32(lkey_u32 + (uint32_t)c * 4u);
          wt += ((key > T) ? 1u : 0u) | ((key == T) ? 0x10000u : 0u);
        }
        const unsigned inc3 = warp_scan_incl(wt, lane);
        if (lane == 31) sm.warp_cnt[warp][0] = inc3;
        settler_sync();
        {
          // the totals of the warps in front (every lane reads them itself: the warp may have diverged)
          unsigned bs = 0;
#pragma unroll 1
          for (int w = 0; w < warp; ++w) bs += sm.warp_cnt[w][0];
          const unsigned ex3 = bs + inc3 - wt;
          unsigned ra = ex3 & 0xffffu, re = ex3 >> 16;
#pragma unroll 1
          for (int c = c0; c < c1; ++c) {
            const unsigned key = lds32(lkey_u32 + (uint32_t)c * 4u);
            const bool gt = key > T, eq = key == T;
            const int pos = (int)(ra + min(re, quota));
            if ((gt || (eq && re < quota)) && pos >= Rc0 && pos < Rc1) {
              const int ch = (int)lds32(lidx_u32 + (uint32_t)c * 4u);
              sm.mysel[ndm + pos - Rc0] = ch;
              if (p.sel_out) p.sel_out[(int)nd + pos] = ch;
            }
            ra += gt ? 1u : 0u; re += eq ? 1u : 0u;
          }
        }
        __threadfence_block();
        settler_sync();                          // the list is free from here on
        if (tid == 0) {
          *reinterpret_cast<volatile int*>(&sm.nready) = n_mine;
          __threadfence_block();
          *reinterpret_cast<volatile int*>(&sm.c_done) = 1;
        }
        PROX_TRACE(6);
        }
      }
    } else {
      // No room in shared memory for the keys plus the list of b1's members (a very large
      // d_ff, or a huge threshold bin such as an all-zero input gives): the whole block
      // settles the threshold by two radix steps of 10 bits over all keys and keeps its
      // share of the plain ascending list before the ring starts.
      const int R0 = (int)(((unsigned)k2 * (unsigned)cta) / (unsigned)G), R1 = (int)(((unsigned)k2 * (unsigned)(cta + 1)) / (unsigned)G);
      n_mine = min(R1 - R0, kMySelCap);
      unsigned prefix = b1, kleft = kk;
#pragma unroll 1
      for (int sh = 10; sh >= 0; sh -= 10) {
        consumer_sync();
        for (int i = tid; i < 1024; i += kFusedConsumers) sm.hist[i] = 0;
        consumer_sync();
#pragma unroll 1
        for (int i = tid; i < F; i += kFusedConsumers) {
          const unsigned key = key_at(i);
          if ((key >> (sh + 10)) == prefix) atomicAdd(&sm.hist[(key >> sh) & 1023u], 1u);
        }
        consumer_sync();
        unsigned ab;
        const unsigned bb = kth_in_block<2, true>(sm.hist, kleft, sm.wsum, lane, warp, &ab);
        prefix = (prefix << 10) | bb;
        kleft -= ab;
      }
      const unsigned T = prefix, quota = kleft;
      consumer_sync();
      {
        unsigned cg = 0, ce = 0;                 // separate words: the ties alone may be 65536
#pragma unroll 1
        for (int i = i0 + lane; i < i1; i += 32) {
          const unsigned key = key_at(i);
          cg += (key > T) ? 1u : 0u; ce += (key == T) ? 1u : 0u;
        }
        cg = __reduce_add_sync(0xffffffffu, cg);
        ce = __reduce_add_sync(0xffffffffu, ce);
        if (lane == 0) { sm.wsum[warp] = cg; sm.warp_cnt[warp][1] = ce; }
      }
      consumer_sync();
      {
        unsigned bg = __reduce_add_sync(0xffffffffu, (lane < warp) ? sm.wsum[lane] : 0u);
        unsigned be = __reduce_add_sync(0xffffffffu, (lane < warp) ? sm.warp_cnt[lane][1] : 0u);
        const int first = (int)(bg + min(be, quota));
        const int end = (int)(bg + sm.wsum[warp] + min(be + sm.warp_cnt[warp][1], quota));
        if (first < R1 && end > R0) {
#pragma unroll 1
          for (int ib = i0; ib < i1; ib += 32) {
            const int i = ib + lane;
            const unsigned key = key_at(min(i, F - 1));
            const bool gt = i < i1 && key > T, eq = i < i1 && key == T;
            const unsigned mg = __ballot_sync(0xffffffffu, gt), me = __ballot_sync(0xffffffffu, eq);
            const unsigned myre = be + (unsigned)__popc(me & lt_mask);
            const int pos = (int)(bg + (unsigned)__popc(mg & lt_mask) + min(myre, quota));
            if ((gt || (eq && myre < quota)) && pos >= R0 && pos < R0 + n_mine) {
              sm.mysel[pos - R0] = i;
              if (p.sel_out) p.sel_out[pos] = i;
            }
            bg += (unsigned)__popc(mg); be += (unsigned)__popc(me);
          }
        }
      }
      __threadfence_block();
      consumer_sync();
      if (tid == 0) {
        sm.keys_s0 = sm.keys_s1 = sm.list_s0 = sm.list_s1 = 0;
        sm.n_mine = n_mine; sm.nready = n_mine; sm.keys_done = 1; sm.c_done = 1;
        __threadfence_block();
        *reinterpret_cast<volatile int*>(&sm.go) = 1;
      }
    }
  }

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
    if (lane == 0 && alive) {
      // wait (bounded) until the consumer warps have listed the block's definite share
      bool go = false;
#pragma unroll 1
      for (unsigned it = 0; it < spin; ++it) {
        if (*reinterpret_cast<volatile int*>(&sm.go)) { go = true; break; }
        if (*abortp) break;
        __nanosleep(32);
      }
      if (!go) sm.abort_flag = 1;
      __threadfence_block();
      fence_proxy_async();                      // the big buffer becomes a bulk-copy target now
      n_mine = go ? *reinterpret_cast<volatile int*>(&sm.n_mine) : 0;
      const unsigned pq = (unsigned)(warp - kFusedConsumerWarps);
      unsigned seq = 0;
      int slot = 0;
      unsigned use = 0;
      bool dead = false;
      int ready = *reinterpret_cast<volatile int*>(&sm.nready);
      bool kdone = *reinterpret_cast<volatile int*>(&sm.keys_done) != 0;
      bool cdone = *reinterpret_cast<volatile int*>(&sm.c_done) != 0;
      const int ks0 = sm.keys_s0, ks1 = sm.keys_s1, ls0 = sm.list_s0, ls1 = sm.list_s1;
      for (int b0 = 0; b0 < n_mine && !dead; b0 += kChanBatch) {
        const int nb = min(kChanBatch, n_mine - b0);
        for (int q = 0; q < 3 * nb; ++q, ++seq) {
          // A slot always belongs to the same producer: its uses are then armed
          // in program order, so the parity wait below is never two phases behind.
          if (((unsigned)slot & (unsigned)(kFusedProducers - 1)) == pq) {
            const int mi = b0 + ((q < 2 * nb) ? (q >> 1) : (q - 2 * nb));
            // The tail of the list (the share of the threshold bin) is written late, and the ring
            // may not touch the slots under the keys before the consumer warps are done with them.
            auto blocked = [&]() {
              return mi >= ready || (!kdone && slot >= ks0 && slot < ks1) || (!cdone && slot >= ls0 && slot < ls1);
            };
            if (blocked()) {
#pragma unroll 1
              for (unsigned it = 0; it < spin; ++it) {
                ready = *reinterpret_cast<volatile int*>(&sm.nready);
                kdone = *reinterpret_cast<volatile int*>(&sm.keys_done) != 0;
                cdone = *reinterpret_cast<volatile int*>(&sm.c_done) != 0;
                if (!blocked() || *abortp) break;
                __nanosleep(64);
              }
              if (blocked()) { sm.abort_flag = 1; dead = true; break; }
            }
            if (use > 0 && !mbar_wait(smem_u32(&sm.mbar_empty[slot]), (use - 1u) & 1u, abortp, spin)) { dead = true; break; }
            const uint16_t* src;
            if (q < 2 * nb) {
              src = ((q & 1) ? p.wu : p.wg) + (size_t)sm.mysel[mi] * D;
            } else {
              src = p.wdt + (size_t)sm.mysel[mi] * D;
            }
            const uint32_t bar = smem_u32(&sm.mbar_full[slot]);
            if (seq == 0) PROX_TRACE_AT(28, tid);
            if (seq == 2u * (unsigned)min(n_mine, kChanBatch)) PROX_TRACE_AT(30, tid);
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
      // D: a warp takes the next channel of the batch that nobody has taken yet (the warps
      // that finish the channel mask join late; rows are consumed in the order they arrive)
      for (;;) {
        int c = 0;
        if (lane == 0) c = (int)atomicAdd(&sm.next_c, 1u);
        c = __shfl_sync(0xffffffffu, c, 0);
        if (c >= nb) break;
        const unsigned sq = base_seq + 2u * (unsigned)c;
        const int sg = (int)(sq % (unsigned)NS), su = (int)((sq + 1u) % (unsigned)NS);
        const unsigned ug = sq / (unsigned)NS, uu = (sq + 1u) / (unsigned)NS;
        const bool ok1 = slot_wait(smem_u32(&sm.mbar_full[sg]), &sm.slot_use[sg], ug, abortp, spin);
        const bool ok2 = slot_wait(smem_u32(&sm.mbar_full[su]), &sm.slot_use[su], uu, abortp, spin);
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
      if (tid == 0) sm.next_c = 0;               // for the next batch (nobody takes channels during E)
      // E: group gq (TG threads) owns rows gq, gq+NG, ... ; a thread owns EV vectors of y
      {
        const int gq = tid / TG, tg = tid % TG;
        for (int c = gq; c < nb; c += NG) {
          const unsigned sq = base_seq + 2u * (unsigned)nb + (unsigned)c;
          const int sd = (int)(sq % (unsigned)NS);
          const unsigned ud = sq / (unsigned)NS;
          const bool ok = slot_wait(smem_u32(&sm.mbar_full[sd]), &sm.slot_use[sd], ud, abortp, spin);
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
        // layer form run in place on the residual stream: the block's share of y goes straight into it (every
        // block read its input before the grid barrier), and there is nothing left to round at the end
        atomicAdd(reinterpret_cast<float4*>((NORM && p.xres_out == p.xres) ? p.xres_out : p.yacc) + v4, s);
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
      if (p.host_flag) *reinterpret_cast<volatile int*>(p.host_flag) = 1;
      const unsigned issued = sm.prod_seq;
      const unsigned first = issued > (unsigned)NS ? issued - (unsigned)NS : 0u;
      for (unsigned q = first; q < issued; ++q) {        // the latest use of every slot
        const uint32_t bar = smem_u32(&sm.mbar_full[q % (unsigned)NS]);
#pragma unroll 1
        for (unsigned it = 0; it < 8192u; ++it) {
          if (mbar_try_wait(bar, (q / (unsigned)NS) & 1u)) break;
          __nanosleep(256);
        }
      }
    }
    __syncthreads();
    return;
  }
  if (NORM && p.xres_out == p.xres) return;     // y went straight into the residual stream: nothing to round, nothing to clean
  if (tid == 0) {
    // release: the block's atomics (ordered before this thread by the barrier above) are out before the ticket is
    // taken; acquire: the block that draws the last ticket sees every other block's
    unsigned t;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(t) : "l"(p.done_ticket) : "memory");
    sm.s_last = (t == (unsigned)(G - 1));
  }
  __syncthreads();
  if (sm.s_last) {
    for (int i0 = tid * 4; i0 < D; i0 += NT * 4 * 4) {        // loads first: they must not queue behind the stores
      float4 v[4], r[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * NT * 4;
        v[u] = (i < D) ? __ldcg(reinterpret_cast<const float4*>(p.yacc + i)) : make_float4(0.f, 0.f, 0.f, 0.f);
        r[u] = (NORM && i < D) ? __ldcg(reinterpret_cast<const float4*>(p.xres + i)) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * NT * 4;
        if (i < D) {
          *reinterpret_cast<float4*>(p.yacc + i) = make_float4(0.f, 0.f, 0.f, 0.f);
          if (NORM) {
            *reinterpret_cast<float4*>(p.xres_out + i) =
                make_float4(r[u].x + v[u].x, r[u].y + v[u].y, r[u].z + v[u].z, r[u].w + v[u].w);
          } else if (p.out_fp32) {
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
    if (tid == 0) *p.done_ticket = 0;
    __syncthreads();
    PROX_TRACE(9);
  }
}

// The persistent kernel lists the kept channels as [definite][share of the
// threshold bin]; callers of the mask get it in ascending order.  One block:
// mark the members in a flag array, then an ordered compaction.  Off the hot path.
__global__ void __launch_bounds__(1024) mask_ascending_kernel(const int* __restrict__ sel, int k2, int F,
                                                              int* __restrict__ flags, int* __restrict__ out) {
  __shared__ unsigned long long ws[33];
  const int tid = threadIdx.x;
  for (int i = tid; i < F; i += 1024) flags[i] = 0;
  __syncthreads();
  for (int i = tid; i < k2; i += 1024) { const int j = sel[i]; if (j >= 0 && j < F) flags[j] = 1; }
  __syncthreads();
  unsigned long long run = 0;
  for (int base = 0; base < F; base += 1024) {
    const int j = base + tid;
    const unsigned long long f = (j < F && flags[j]) ? 1ull : 0ull;
    unsigned long long tot;
    const unsigned long long ex = block_scan_excl<1024>(f, ws, &tot);
    if (f && run + ex < (unsigned long long)k2) out[run + ex] = j;
    run += tot;
  }
}

}  // namespace prox
