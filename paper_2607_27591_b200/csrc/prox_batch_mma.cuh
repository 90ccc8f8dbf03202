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
#include "prox_fused.cuh"

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

// Union of the tokens' kept channels for the tensor-core path, in two small
// kernels: every (token, kept channel) sets the token's bit in a byte per channel;
// one block then lists the channels whose byte is not zero in ascending order,
// copies the byte next to the list and clears it for the next call.
__global__ void __launch_bounds__(256)
union_mark_kernel(const int* __restrict__ lists, int stride, int k, int B, int n, unsigned* __restrict__ mask32,
                  int* __restrict__ status) {
  pdl_enter();
  const int i = blockIdx.x * 256 + threadIdx.x;
  if (i >= B * k) return;
  const int b = i / k, r = i % k;
  const int id = lists[(size_t)b * stride + r];
  if (id >= 0 && id < n) atomicOr(mask32 + (id >> 2), (1u << b) << (8 * (id & 3)));
  else atomicOr(status, kBadChannel);
}

__global__ void __launch_bounds__(1024)
union_compact_kernel(unsigned* __restrict__ mask32, int n, int* __restrict__ ulist, int* __restrict__ nu_out,
                     uint8_t* __restrict__ umask, int staged) {
  pdl_enter();
  // staged: the list is put together in shared memory (a thread's entries land anywhere in it) and leaves in
  // whole lines; otherwise (a layer too wide for that) the entries go to global memory one by one
  extern __shared__ __align__(16) uint8_t uc_smem[];
  int* slist = staged ? reinterpret_cast<int*>(uc_smem) : ulist;              // [n] channel ids
  uint8_t* smask = staged ? uc_smem + (size_t)n * 4 : umask;                  // [n] token bits
  __shared__ unsigned long long ws[33];
  const int tid = threadIdx.x;
  const int nw = (n + 3) / 4, per = (nw + 1023) / 1024;          // mask words per thread (consecutive), at most 16
  const int w0 = min(nw, tid * per), w1 = min(nw, w0 + per);
  unsigned m[16];
  unsigned cnt = 0;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    m[i] = (w0 + i < w1) ? __ldcg(mask32 + w0 + i) : 0u;
    cnt += ((m[i] & 0xffu) ? 1u : 0u) + ((m[i] & 0xff00u) ? 1u : 0u) + ((m[i] & 0xff0000u) ? 1u : 0u) + ((m[i] >> 24) ? 1u : 0u);
  }
  unsigned long long tot;
  unsigned pos = (unsigned)block_scan_excl<1024>((unsigned long long)cnt, ws, &tot);
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    if (w0 + i < w1) {
      mask32[w0 + i] = 0;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const unsigned by = (m[i] >> (8 * q)) & 0xffu;
        const int ch = (w0 + i) * 4 + q;
        if (by && ch < n) { slist[pos] = ch; smask[pos] = (uint8_t)by; ++pos; }
      }
    }
  }
  __syncthreads();
  const int nu = (int)tot;
  if (staged) {
    for (int i = tid; i < nu; i += 1024) ulist[i] = slist[i];
    for (int i = tid; i < (nu + 3) / 4; i += 1024)               // four bytes at a time (the tail may carry stale bytes: unused)
      reinterpret_cast<unsigned*>(umask)[i] = reinterpret_cast<const unsigned*>(smask)[i];
  }
  if (tid == 0) *nu_out = nu;
}

// ----------------------------------------------------------------------------
// Stage 2a with the weight rows streamed by bulk async copies (d_model <= 4096).
// Plain loads of rows that are gathered 64 bytes at a time stay near 4.5 TB/s;
// whole rows through cp.async.bulk, as in the batch-1 kernel, do not.
// One block per SM: 16 consumer warps + one producer warp whose 32 lanes issue the
// copies.  A tile is 8 union channels = 16 rows: rows 0..7 of the MMA's A operand
// are the gate rows, rows 8..15 the up rows of the same channels, so one MMA gives
// both pre-activations of a channel to the same lane.  A ring slot holds up to 4 KB
// of a row (+ 64 bytes of padding: the fragment loads of eight rows then fall into
// different banks); a longer row comes as two sections, so that several tiles are
// in flight.  A consumer warp owns a sixteenth of every section; its share of x
// (the B operand) lives in registers for the whole kernel.
// The warps' partial sums of a tile meet in shared memory and h is written at
// once: no accumulator in global memory and no finishing kernel.
// ----------------------------------------------------------------------------
constexpr int kGrThreads = kMmaThreads + 32;        // 16 consumer warps + one producer warp
constexpr int kGrMaxSlots = 64;
constexpr int kGrMaxTiles = 64;                     // tiles of a block whose channels are staged in shared memory
constexpr int kGrPiece = 4096;                      // bytes of a row in one ring slot (a whole row if it is shorter)

__global__ void __launch_bounds__(kGrThreads, 1)
gateup_rows_kernel(const uint16_t* __restrict__ wg, const uint16_t* __restrict__ wu,
                   const uint16_t* __restrict__ x, int B, const int* __restrict__ ulist,
                   const uint8_t* __restrict__ umask, const int* __restrict__ nu_ptr, int D, int nslots,
                   float* __restrict__ h_out, int* __restrict__ status) {
  pdl_enter();
  extern __shared__ __align__(128) uint8_t mm_smem[];
  __shared__ unsigned long long bar_full[kGrMaxSlots / 16], bar_empty[kGrMaxSlots / 16];   // per section of 16 slots
  __shared__ int abort_flag;
  __shared__ unsigned n_issued;                                 // sections armed so far (for the give-up path)
  __shared__ int my_ch[kGrMaxTiles * 8];
  const int NSEC = nslots / 16;                                 // sections (16 slots) in the ring
  const uint32_t piece = (uint32_t)min(kGrPiece, D * 2);        // bytes of a row per slot
  const int nsec = (D * 2) / (int)piece;                        // sections of a row (1 or 2 up to d_model 4096)
  const uint32_t pitch = piece + 64u;
  float* red = reinterpret_cast<float*>(mm_smem + (size_t)NSEC * 16 * pitch);     // [16 warps][128]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const int nu = *nu_ptr;
  if (nu <= 0) return;
  if (tid < NSEC) {
    mbar_init(smem_u32(&bar_full[tid]), 1);
    mbar_init(smem_u32(&bar_empty[tid]), kMmaWarps);
    fence_mbar_init();
  }
  if (tid == 0) { abort_flag = 0; n_issued = 0; }
  const int ntile = (nu + 7) / 8;
  // the union channels of this block's tiles, so that a producer does not wait for global memory per copy
  for (int i = tid; i < kGrMaxTiles * 8; i += kGrThreads) {
    const int tile = blockIdx.x + (i >> 3) * gridDim.x;
    my_ch[i] = (tile < ntile) ? ulist[min(tile * 8 + (i & 7), nu - 1)] : 0;
  }
  fence_proxy_async();
  __syncthreads();
  volatile int* abortp = &abort_flag;
  const uint32_t ring_u32 = smem_u32(mm_smem);
  if (warp >= kMmaWarps) {
    // ---- producer warp: one thread starts well under a million copies a second here, so all 32
    // lanes issue: lanes 0..15 the 16 rows of one section, lanes 16..31 those of the next one.
    // (One warp, in program order: the use of a slot is always armed after its previous use.)
    const int per_tile = nsec;                                  // sections per tile
    const int my_tiles = (ntile - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    const int nsect = my_tiles * per_tile;                      // sections of this block
    const int r = lane & 15;
    bool dead = false;
    for (int s0 = 0; s0 < nsect && !dead; s0 += 2) {
      const int si = s0 + (lane >> 4);                          // this lane's section
      const int ss = si % NSEC;                                 // its place in the ring (16 slots, one barrier pair)
      const unsigned use = (unsigned)(si / NSEC);
      bool ok = true;
      if (si < nsect && use > 0 && r == 0) ok = mbar_wait(smem_u32(&bar_empty[ss]), (use - 1u) & 1u, abortp);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { dead = true; break; }
      if (si < nsect) {
        const int ti = si / per_tile, sec = si - ti * per_tile;
        const int tile = (int)blockIdx.x + ti * (int)gridDim.x;
        const uint32_t bar = smem_u32(&bar_full[ss]);
        if (r == 0) { mbar_expect_tx(bar, 16u * piece); atomicMax(&n_issued, (unsigned)si + 1u); }
        __syncwarp();
        const int ch = (ti < kGrMaxTiles) ? my_ch[ti * 8 + (r & 7)] : ulist[min(tile * 8 + (r & 7), nu - 1)];
        const uint8_t* src = reinterpret_cast<const uint8_t*>((r < 8 ? wg : wu) + (size_t)ch * D) + (size_t)sec * piece;
        bulk_g2s(ring_u32 + (uint32_t)(ss * 16 + r) * pitch, src, piece, bar);
      } else {
        __syncwarp();
      }
    }
  } else {
    // ---- consumer warps
    const int npw = (int)piece / 1024;                          // 32-input pieces of a section per warp (<= 4)
    uint4 xv[8];                                                // x of token g: sections x pieces of this warp
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int sec = i >> 2, pc = i & 3;
      xv[i] = make_uint4(0, 0, 0, 0);
      if (sec < nsec && pc < npw && g < B)
        xv[i] = __ldg(reinterpret_cast<const uint4*>(x + (size_t)g * D + sec * ((int)piece / 2) + (warp * npw + pc) * 32 + t * 8));
    }
    unsigned sidx = 0;                 // running section number of this block
    bool dead = false;                 // a wait expired: go on without touching the ring, but keep every barrier
    for (int tile = blockIdx.x; tile < ntile; tile += gridDim.x) {
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int sec = 0; sec < 2; ++sec) {
        if (sec < nsec) {
          // this lane reads the gate row and the up row of channel g of the tile
          const int ss = (int)(sidx % (unsigned)NSEC);
          const int sg = ss * 16 + g, su = ss * 16 + 8 + g;
          // One thread alone waits for the 16 rows of the section: hundreds of threads polling the
          // barrier slow the copies down.  The others learn of it at a block barrier.
          if (tid == 0 && !dead) {
            if (!mbar_wait(smem_u32(&bar_full[ss]), (sidx / (unsigned)NSEC) & 1u, abortp)) abort_flag = 1;
          }
          asm volatile("bar.sync 1, %0;" ::"n"(kMmaThreads) : "memory");
          if (*abortp) dead = true;
          if (!dead) {
            const uint32_t pg = ring_u32 + (uint32_t)sg * pitch + (uint32_t)(warp * npw) * 64u + (uint32_t)t * 16u;
            const uint32_t pu = ring_u32 + (uint32_t)su * pitch + (uint32_t)(warp * npw) * 64u + (uint32_t)t * 16u;
#pragma unroll
            for (int pc = 0; pc < 4; ++pc) {
              if (pc < npw) {
                const uint4 gl = lds128(pg + (uint32_t)pc * 64u), ul = lds128(pu + (uint32_t)pc * 64u);
                const uint4 xw = xv[sec * 4 + pc];
                mma_bf16(acc, gl.x, ul.x, gl.y, ul.y, xw.x, xw.y);
                mma_bf16(acc, gl.z, ul.z, gl.w, ul.w, xw.z, xw.w);
              }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive_n(smem_u32(&bar_empty[ss]), 1u);       // this warp is done with the section
          }
          ++sidx;
        }
      }
      // the warps' partial sums meet: [gate | up][channel g][token]
      float* mine = red + warp * 128;
      mine[g * 8 + 2 * t] = acc[0]; mine[g * 8 + 2 * t + 1] = acc[1];
      mine[64 + g * 8 + 2 * t] = acc[2]; mine[64 + g * 8 + 2 * t + 1] = acc[3];
      asm volatile("bar.sync 1, %0;" ::"n"(kMmaThreads) : "memory");
      if (tid < 64) {
        float gate = 0.f, up = 0.f;
#pragma unroll
        for (int w = 0; w < kMmaWarps; ++w) { gate += red[w * 128 + tid]; up += red[w * 128 + 64 + tid]; }
        const int r = tile * 8 + (tid >> 3), b = tid & 7;
        if (r < nu) h_out[(size_t)r * kBT + b] = (b < B && ((umask[r] >> b) & 1u)) ? up * silu_exact(gate) : 0.f;
      }
      asm volatile("bar.sync 1, %0;" ::"n"(kMmaThreads) : "memory");
    }
  }
  __syncthreads();
  if (abort_flag && tid == 0) {
    // a wait expired: the copies that were armed last may still be on their way; wait for them
    // (bounded) so that none lands after the block has left
    atomicOr(status, kWaitExpired);
    const unsigned issued = n_issued;                           // sections armed
    const unsigned first = issued > (unsigned)NSEC ? issued - (unsigned)NSEC : 0u;
    for (unsigned q = first; q < issued; ++q) {
      const uint32_t bar = smem_u32(&bar_full[q % (unsigned)NSEC]);
      for (unsigned it = 0; it < 8192u; ++it) {
        if (mbar_try_wait(bar, (q / (unsigned)NSEC) & 1u)) break;
        __nanosleep(256);
      }
    }
  }
}

// h[r][b] = SiLU(gate) * up for the tokens that kept channel r, 0 for the others;
// the accumulator is cleared for the next call.
__global__ void __launch_bounds__(256)
gateup_finish_kernel(float* __restrict__ gacc, const uint8_t* __restrict__ umask, const int* __restrict__ nu_ptr,
                     int B, float* __restrict__ h_out) {
  const int nu = *nu_ptr;
  for (int i = blockIdx.x * 256 + threadIdx.x; i < nu * kBT; i += gridDim.x * 256) {
    const int r = i / kBT, b = i % kBT;
    const float gate = gacc[(size_t)r * 16 + b], up = gacc[(size_t)r * 16 + 8 + b];
    gacc[(size_t)r * 16 + b] = 0.f; gacc[(size_t)r * 16 + 8 + b] = 0.f;
    h_out[i] = (b < B && ((umask[r] >> b) & 1u)) ? up * silu_exact(gate) : 0.f;
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
  pdl_enter();
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
    auto rows_of = [&](int kb, int (&j)[4]) {                  // W_downT rows of the unit's four K slots
      const int c0 = kb * 16 + 2 * t;
      const int cr[4] = {c0, c0 + 1, c0 + 8, c0 + 9};
#pragma unroll
      for (int q = 0; q < 4; ++q) j[q] = __ldg(ulist + min(cr[q], nu - 1));
    };
    auto load_unit = [&](int kb, const int (&j)[4], uint4 (&w)[4], float (&hv)[4]) {
      const int c0 = kb * 16 + 2 * t;
      const int cr[4] = {c0, c0 + 1, c0 + 8, c0 + 9};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        w[q] = ld_stream(colp + (size_t)j[q] * D);
        hv[q] = (cr[q] < nu) ? __ldg(h + (size_t)cr[q] * kBT + g) : 0.f;
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
    int ja[4], jb[4];
    if (a + warp < b) rows_of(a + warp, ja);
    if (a + warp + kMmaWarps < b) rows_of(a + warp + kMmaWarps, jb);
    for (int kb = a + warp; kb < b; kb += 2 * kMmaWarps) {      // two units in flight per warp
      uint4 wa[4], wb[4];
      float ha[4], hb[4];
      const bool two = kb + kMmaWarps < b;
      load_unit(kb, ja, wa, ha);
      if (two) load_unit(kb + kMmaWarps, jb, wb, hb);
      if (kb + 2 * kMmaWarps < b) rows_of(kb + 2 * kMmaWarps, ja);
      if (kb + 3 * kMmaWarps < b) rows_of(kb + 3 * kMmaWarps, jb);
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

namespace prox {

// ----------------------------------------------------------------------------
// Input preparation of Stage 1 for B > 1 (the GEMM itself is the tcgen05 kernel
// of prox_batch_umma.cuh): the step-wise fallback for shapes whose input mask
// does not fit the one-block-per-token kernel further down.
// ----------------------------------------------------------------------------
// One block per token slot.  The token's kept inputs (its ascending index list)
// become an fp16 vector over ALL inputs: x * s at a kept input, 0 elsewhere, with
// s the power of two that puts max |x| into [2^13, 2^14).  With eight tokens the
// union of the kept inputs is nearly everything, so the proxy GEMM simply runs
// over all rows and needs no union list; a dropped input contributes 0 * code.
// tokfac[b] = 2^24 / s undoes the scaling (and the 2^-24 of the codes).
__global__ void __launch_bounds__(512)
proxy_xprep_kernel(const uint16_t* __restrict__ x, const int* __restrict__ idx, int stride, int k1, int B, int D,
                   __half* __restrict__ xh, float* __restrict__ tokfac) {
  __shared__ unsigned smax;
  const int b = blockIdx.x, tid = threadIdx.x;
  __half* row = xh + (size_t)b * D;
  if (tid == 0) smax = 0;
  __syncthreads();
  unsigned m = 0;
  if (b < B) for (int r = tid; r < k1; r += 512) m = max(m, (unsigned)(x[(size_t)b * D + idx[(size_t)b * stride + r]] & 0x7fffu));
  m = __reduce_max_sync(0xffffffffu, m);
  if ((tid & 31) == 0 && m) atomicMax(&smax, m);
  for (int i = tid; i < D / 8; i += 512) reinterpret_cast<uint4*>(row)[i] = make_uint4(0, 0, 0, 0);
  __syncthreads();
  int se = 0;
  if (smax) se = 13 - ((int)(smax >> 7) - 127);                  // bf16 magnitude bits: exponent in bits 14..7
  se = max(-100, min(100, se));
  const float s = __uint_as_float((unsigned)(se + 127) << 23);
  if (tid == 0) tokfac[b] = __uint_as_float((unsigned)(24 - se + 127) << 23);
  if (b < B) {
    for (int r = tid; r < k1; r += 512) {
      const int i = idx[(size_t)b * stride + r];
      const float v = __uint_as_float(((uint32_t)x[(size_t)b * D + i]) << 16) * s;
      row[i] = __float2half_rn(v);
    }
  }
}

// ----------------------------------------------------------------------------
// Per-token masks of the tensor-core batch path, one 640-thread block per token,
// built from the selection code of the persistent batch-1 kernel (short loops,
// thread-owned runs, one warp scan per pass).
// ----------------------------------------------------------------------------

// Input mask m_x of a token straight into the proxy GEMM's operand: exact top-k1
// of |x| (ties: lower index first), then xh[b][i] = fp16(x_i * s) at the kept
// inputs and 0 elsewhere, s the power of two that puts max |x| into [2^13, 2^14);
// tokfac[b] = 2^24 / s.  Token slots beyond B are cleared.
__global__ void __launch_bounds__(kFusedThreads)
batch_input_mask_kernel(const uint16_t* __restrict__ x, int B, int D, int k1, __half* __restrict__ xh,
                        float* __restrict__ tokfac, uint32_t* __restrict__ xd, float* __restrict__ soff) {
  extern __shared__ __align__(16) uint8_t bm_smem[];
  uint16_t* xs = reinterpret_cast<uint16_t*>(bm_smem);           // [D] bf16 bits of the token
  __shared__ unsigned hist[1024], hist2[32], wsum[32], smax;
  __shared__ int sd[128 * 4];                                     // digit sums of the units of 128 inputs
  constexpr int NT = kFusedThreads;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_enter();                                    // the proxy GEMM may set up and start on the weights
  __half* row = xh + (size_t)b * D;
  if (b >= B) {
    if (xd) {
      for (int i = tid; i < D; i += NT) xd[(size_t)(i >> 5) * 256 + (b >> 2) * 128 + (i & 31) * 4 + (b & 3)] = 0u;
      for (int u = tid; u < (D >> 7); u += NT) soff[(size_t)u * kBT + b] = 0.f;
    } else {
      for (int i = tid; i < D / 8; i += NT) reinterpret_cast<uint4*>(row)[i] = make_uint4(0, 0, 0, 0);
    }
    if (tid == 0) tokfac[b] = 16777216.f;
    return;
  }
  for (int i = tid; i < 512; i += NT) sd[i] = 0;
  if (tid == 0) smax = 0;
  for (int i = tid; i < 1024 + 32; i += NT) { if (i < 1024) hist[i] = 0; else hist2[i - 1024] = 0; }
  __syncthreads();
  unsigned m = 0;
  for (int i = tid; i < D / 8; i += NT) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(x + (size_t)b * D) + i);
    reinterpret_cast<uint4*>(xs)[i] = v;
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) m = max(m, max(w[e] & 0x7fffu, (w[e] >> 16) & 0x7fffu));
  }
  m = __reduce_max_sync(0xffffffffu, m);
  if (lane == 0 && m) atomicMax(&smax, m);
  __syncthreads();
  int se = 0;
  if (smax) se = 13 - ((int)(smax >> 7) - 127);                  // bf16 magnitude bits: exponent in bits 14..7
  se = max(-100, min(100, se));
  const float sf = __uint_as_float((unsigned)(se + 127) << 23);
  if (tid == 0) tokfac[b] = __uint_as_float((unsigned)(24 - se + 127) << 23);
  const uint32_t* xs32 = reinterpret_cast<const uint32_t*>(xs);
  const bool all = k1 >= D;
  unsigned T = 0, quota = 0;
  if (!all) {
    // level 1: the top 10 of the 15 key bits; level 2: the other 5
#pragma unroll 1
    for (int i = tid; i < D / 2; i += NT) {
      const uint32_t w = xs32[i];
      atomicAdd(&hist[(w >> 5) & 0x3ffu], 1u);
      atomicAdd(&hist[(w >> 21) & 0x3ffu], 1u);
    }
    __syncthreads();
    unsigned above1;
    const unsigned bin1 = kth_in_block<2, false>(hist, (unsigned)k1, wsum, lane, warp, &above1);
#pragma unroll 1
    for (int i = tid; i < D / 2; i += NT) {
      const uint32_t w = xs32[i];
      const unsigned ka = w & 0x7fffu, kb = (w >> 16) & 0x7fffu;
      if ((ka >> 5) == bin1) atomicAdd(&hist2[ka & 31u], 1u);
      if ((kb >> 5) == bin1) atomicAdd(&hist2[kb & 31u], 1u);
    }
    __syncthreads();
    unsigned above2;
    const unsigned bin2 = kth_in_segment<1>(hist2, 32, (unsigned)k1 - above1, lane, &above2);
    T = (bin1 << 5) | bin2;
    quota = (unsigned)k1 - above1 - above2;        // ties at T to accept, lowest index first
  }
  // a thread owns a run of 8-input groups; only the ties need their rank (one warp scan + warp totals)
  const int ngrp = D / 8, gpt = (ngrp + NT - 1) / NT;
  const int g0 = min(ngrp, tid * gpt), g1 = min(ngrp, g0 + gpt);
  unsigned ties = 0;
#pragma unroll 1
  for (int g = g0; g < g1; ++g) {
    const uint4 kv = *reinterpret_cast<const uint4*>(xs + g * 8);
    const uint32_t w4[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
    for (int e = 0; e < 8; ++e) ties += (!all && ((w4[e >> 1] >> ((e & 1) * 16)) & 0x7fffu) == T) ? 1u : 0u;
  }
  const unsigned inc = warp_scan_incl(ties, lane);
  __syncthreads();                                 // every warp is done with wsum (k-th search above)
  if (lane == 31) wsum[warp] = inc;
  __syncthreads();
  unsigned re = __reduce_add_sync(0xffffffffu, (lane < warp) ? wsum[lane] : 0u) + inc - ties;
#pragma unroll 1
  for (int g = g0; g < g1; ++g) {
    const uint4 kv = *reinterpret_cast<const uint4*>(xs + g * 8);
    const uint32_t w4[4] = {kv.x, kv.y, kv.z, kv.w};
    uint32_t o[4];
    int d0 = 0, d1 = 0, d2 = 0, d3 = 0;
    uint32_t* dst = xd ? xd + (size_t)(g >> 2) * 256 + (b >> 2) * 128 + ((g & 3) * 8) * 4 + (b & 3) : nullptr;
#pragma unroll
    for (int e2 = 0; e2 < 4; ++e2) {
      __half hv[2];
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const unsigned bits = (w4[e2] >> (hh * 16)) & 0xffffu, key = bits & 0x7fffu;
        const bool gt = all || key > T, eq = !all && key == T;
        const bool keep = gt || (eq && re < quota);
        re += eq ? 1u : 0u;
        hv[hh] = __float2half_rn(keep ? __uint_as_float(bits << 16) * sf : 0.f);
        if (xd) {
          // integer form of the masked, scaled fp16 input: X = x_h * 2^16 as four signed base-256 digits
          const int X = __float2int_rn(__half2float(hv[hh]) * 65536.f);
          const uint32_t dg = ((uint32_t)X + 0x00808080u) ^ 0x00808080u;
          dst[(e2 * 2 + hh) * 4] = dg;
          d0 += (int)(int8_t)(dg & 0xffu); d1 += (int)(int8_t)((dg >> 8) & 0xffu);
          d2 += (int)(int8_t)((dg >> 16) & 0xffu); d3 += (int)(int8_t)(dg >> 24);
        }
      }
      o[e2] = (uint32_t)__half_as_ushort(hv[0]) | ((uint32_t)__half_as_ushort(hv[1]) << 16);
    }
    if (xd) {
      int* sdg = sd + 4 * (g >> 4);
      if (d0) atomicAdd(sdg, d0);
      if (d1) atomicAdd(sdg + 1, d1);
      if (d2) atomicAdd(sdg + 2, d2);
      if (d3) atomicAdd(sdg + 3, d3);
    } else {
      reinterpret_cast<uint4*>(row)[g] = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
  if (xd) {
    __syncthreads();
    for (int u = tid; u < (D >> 7); u += NT)
      soff[(size_t)u * kBT + b] = digits_to_float((uint32_t)sd[u * 4], (uint32_t)sd[u * 4 + 1], (uint32_t)sd[u * 4 + 2],
                                                  (uint32_t)sd[u * 4 + 3]);
  }
}

// One mask for the whole batch (a policy beyond the paper): the channels are ranked by the sum of the
// tokens' proxy scores, added token after token in fp32.
__global__ void __launch_bounds__(256) shared_score_kernel(const float* __restrict__ scores, int B, int F,
                                                           float* __restrict__ out) {
  pdl_enter();
  const int j = blockIdx.x * 256 + threadIdx.x;
  if (j >= F) return;
  float s = 0.f;
  for (int b = 0; b < B; ++b) s += scores[(size_t)b * F + j];
  out[j] = s;
}

// ... and every token's row of the mask output is that one list.
__global__ void __launch_bounds__(256) replicate_mask_kernel(int* __restrict__ sel, int sel_stride, int k2, int B) {
  pdl_enter();
  const int r = blockIdx.x * 256 + threadIdx.x;
  if (r >= k2) return;
  const int v = sel[r];
  for (int b = 1; b < B; ++b) sel[(size_t)b * sel_stride + r] = v;
}

// Channel mask m_s of a token from its scores: exact top-k2 (ties: lower channel
// first) by three radix steps over the score bits held in shared memory, then an
// ordered list of the kept channels; the token's bit is also set in the channel's
// byte of cmask (the union of the tokens' masks is read off those bytes).
// token_bits = 0: block b is token b and sets bit b.  Otherwise (one shared mask for the batch: one block
// over the summed scores) the kept channels get all of token_bits.
constexpr int kCmThreads = 1024;                   // channel-mask kernel: all 32 warps of a block
__global__ void __launch_bounds__(kCmThreads)
batch_channel_mask_kernel(const float* __restrict__ scores, int F, int k2, int* __restrict__ sel_out, int sel_stride,
                          unsigned* __restrict__ cmask, unsigned token_bits, float* __restrict__ pacc, int nrep,
                          int* __restrict__ ulist, uint8_t* __restrict__ umask, int* __restrict__ nu_out) {
  pdl_enter();
  extern __shared__ __align__(16) uint8_t bm_smem[];
  unsigned* skey = reinterpret_cast<unsigned*>(bm_smem);         // [F] score bits
  __shared__ unsigned hist[2048], wsum[32], wsum2[32];
  constexpr int NT = kCmThreads;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned* gkey = reinterpret_cast<const unsigned*>(scores) + (size_t)b * F;
  const uint32_t skey_u32 = smem_u32(skey);
  for (int i = tid; i < 2048; i += NT) hist[i] = 0;
  __syncthreads();
  if (pacc) {
    // scores straight from the proxy sums of the tensor-core GEMM ([token][gate | up][channel]); the token's
    // entries are cleared for the next call.  Four rounds of loads are issued before the first use: one round per
    // dependent iteration would put the latency of global memory on every one of them.
    float4* pg = reinterpret_cast<float4*>(pacc + (size_t)b * 2 * F);
    float4* pu = pg + F / 4;
    const int n4 = F / 4;
#pragma unroll 1
    for (int i0 = tid; i0 < n4; i0 += 4 * NT) {
      float4 g[4], u[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int i = i0 + r * NT;
        g[r] = i < n4 ? __ldcg(pg + i) : make_float4(0.f, 0.f, 0.f, 0.f);
        u[r] = i < n4 ? __ldcg(pu + i) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int i = i0 + r * NT;
        if (i < n4) {
          pg[i] = make_float4(0.f, 0.f, 0.f, 0.f); pu[i] = make_float4(0.f, 0.f, 0.f, 0.f);
          const uint4 k = make_uint4(__float_as_uint(fabsf(u[r].x * silu_fast(g[r].x))), __float_as_uint(fabsf(u[r].y * silu_fast(g[r].y))),
                                     __float_as_uint(fabsf(u[r].z * silu_fast(g[r].z))), __float_as_uint(fabsf(u[r].w * silu_fast(g[r].w))));
          reinterpret_cast<uint4*>(skey)[i] = k;
          atomicAdd(&hist[k.x >> 20], 1u); atomicAdd(&hist[k.y >> 20], 1u);
          atomicAdd(&hist[k.z >> 20], 1u); atomicAdd(&hist[k.w >> 20], 1u);
        }
      }
    }
  } else {
    for (int i = tid; i < F / 4; i += NT) cp_async16(skey_u32 + (uint32_t)i * 16u, gkey + 4 * i);
    cp_async_commit();
    cp_async_wait<0>();
    __syncthreads();
#pragma unroll 1
    for (int i = tid; i < F; i += NT) atomicAdd(&hist[skey[i] >> 20], 1u);
  }
  __syncthreads();
  unsigned ab;
  unsigned prefix = kth_in_block<4, false>(hist, (unsigned)k2, wsum, lane, warp, &ab);
  unsigned kleft = (unsigned)k2 - ab;
#pragma unroll 1
  for (int sh = 10; sh >= 0; sh -= 10) {           // two more steps of 10 bits
    __syncthreads();
    for (int i = tid; i < 1024; i += NT) hist[i] = 0;
    __syncthreads();
#pragma unroll 1
    for (int i = tid; i < F; i += NT) {
      const unsigned key = skey[i];
      if ((key >> (sh + 10)) == prefix) atomicAdd(&hist[(key >> sh) & 1023u], 1u);
    }
    __syncthreads();
    const unsigned bb = kth_in_block<2, false>(hist, kleft, wsum, lane, warp, &ab);
    prefix = (prefix << 10) | bb;
    kleft -= ab;
  }
  const unsigned T = prefix, quota = kleft;
  // ordered list: a thread owns a run of 4-channel groups
  const int nq = F / 4, qpt = (nq + NT - 1) / NT;
  const int q0 = min(nq, tid * qpt), q1 = min(nq, q0 + qpt);
  unsigned cg = 0, ce = 0;
#pragma unroll 1
  for (int q = q0; q < q1; ++q) {
    const uint4 kv = *reinterpret_cast<const uint4*>(skey + q * 4);
    const unsigned k4[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) { cg += (k4[e] > T) ? 1u : 0u; ce += (k4[e] == T) ? 1u : 0u; }
  }
  const unsigned ig = warp_scan_incl(cg, lane), ie = warp_scan_incl(ce, lane);
  __syncthreads();                                 // every warp is done with wsum (k-th search above)
  if (lane == 31) { wsum[warp] = ig; wsum2[warp] = ie; }
  __syncthreads();
  unsigned rg = __reduce_add_sync(0xffffffffu, (lane < warp) ? wsum[lane] : 0u) + ig - cg;
  unsigned re = __reduce_add_sync(0xffffffffu, (lane < warp) ? wsum2[lane] : 0u) + ie - ce;
  int* out = sel_out + (size_t)b * sel_stride;
#pragma unroll 1
  for (int q = q0; q < q1; ++q) {
    const uint4 kv = *reinterpret_cast<const uint4*>(skey + q * 4);
    const unsigned k4[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const bool gt = k4[e] > T, eq = k4[e] == T;
      if (gt || (eq && re < quota)) {
        const int ch = q * 4 + e;
        if (nrep > 1) reinterpret_cast<int*>(skey + F)[rg + min(re, quota)] = ch;     // staged: every token's row gets the list
        else out[rg + min(re, quota)] = ch;
        if (cmask) atomicOr(cmask + (ch >> 2), (token_bits ? token_bits : (1u << b)) << (8 * (ch & 3)));
      }
      rg += gt ? 1u : 0u; re += eq ? 1u : 0u;
    }
  }
  if (nrep > 1) {
    // one mask for the batch: the list goes to every token's row, in whole lines
    __syncthreads();
    const int* slist = reinterpret_cast<const int*>(skey + F);
    for (int r = 0; r < nrep; ++r)
      for (int i = tid; i < k2; i += NT) sel_out[(size_t)r * sel_stride + i] = slist[i];
    if (ulist) {
      // ... and it is the union of the tokens' masks as well: every kept channel belongs to every token
      for (int i = tid; i < k2; i += NT) { ulist[i] = slist[i]; umask[i] = (uint8_t)token_bits; }
      if (tid == 0) *nu_out = k2;
    }
  }
}

// One mask for the whole batch straight from the proxy sums of the tensor-core GEMM: out[j] = sum over the
// tokens of |up~ SiLU(gate~)|, added token after token in fp32; the accumulator is cleared for the next call.
__global__ void __launch_bounds__(256) shared_score_from_sums_kernel(float* __restrict__ pacc, int B, int F,
                                                                     float* __restrict__ out) {
  pdl_enter();
  const int j = blockIdx.x * 256 + threadIdx.x;
  if (j >= F) return;
  // all loads first (a load behind every store would put the latency of global memory on every token)
  float gate[kBT], up[kBT];
#pragma unroll
  for (int b = 0; b < kBT; ++b) {
    const float* pg = pacc + (size_t)b * 2 * F + j;
    gate[b] = __ldcg(pg); up[b] = __ldcg(pg + F);
  }
  float s = 0.f;
#pragma unroll
  for (int b = 0; b < kBT; ++b) {
    float* pg = pacc + (size_t)b * 2 * F + j;
    pg[0] = 0.f; pg[F] = 0.f;
    if (b < B) s += fabsf(up[b] * silu_fast(gate[b]));
  }
  out[j] = s;
}

}  // namespace prox
