// Host side of libprox: argument validation, memory ownership, launches.
// Declarations and per-call documentation live in include/prox.h.
#include "prox.h"

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "prox_kernels.cuh"
#include "prox_fused.cuh"
#include "prox_batch_mma.cuh"
#include "prox_batch_umma.cuh"

using namespace prox;

enum KernelKind { kKInput = 0, kKProxy, kKChannel, kKGateUp, kKDown, kKFinalize, kKFused, kKUnion };
struct ProfRec { int kind; cudaEvent_t a, b; };

struct prox_ffn {
  prox_ffn_config_t cfg;
  const uint16_t* wg;
  const uint16_t* wu;
  const uint16_t* wd;
  int device;
  int sm_count;
  // packed state (owned)
  int bits, group;          // group = actual group length (D when per-row)
  bool quantized;
  uint8_t* P;               // [D][F*bits/4]
  size_t p_bytes;
  __half* S;                // [ngroups][nchunks][2][CH]
  size_t s_count;
  float* s_plain;           // [2][F][ngroups] fp32 copy of the scales
  uint16_t* wdt;            // [F][D]
  // scratch (owned)
  int* idx_x;               // [maxB][D]
  int* cnt_x;               // [maxB]
  float* part;              // split-K partial sums
  size_t part_floats;
  unsigned* ticket;         // [maxB][nstrips_max]
  float* scores;            // [maxB][F]
  float* svals;             // [maxB][F] signed proxy values (proxy-values-into-down variant)
  uint16_t* xn;             // [maxB][D] bf16 FFN input of the layer sub-block form (step-wise path)
  const float* fin_resid;   // while a layer sub-block call is enqueued: the residual stream to add ...
  float* fin_out;           // ... and where the sum goes
  int* sel;                 // [maxB][F]
  int* cnt_s;               // [maxB]
  float* hbuf;              // [maxB][F]
  float* yacc;              // [maxB][D]
  int* dev_status;
  unsigned long long* counters;  // [0] tokens, [1] kept inputs, [2] kept channels
  unsigned* syncbuf;        // fused kernel: [0..4095] two score histograms (calls alternate), [4096] barrier count,
                            // (64-bit, [4096..4097]), [4098] finish ticket
  int smem_optin;           // largest dynamic shared memory a block may ask for
  int coop;                 // device supports cooperative launch
  int sel_unordered;        // the last forward left its mask in the persistent kernel's own order
  int use_fused;            // batch-1 forward runs as one persistent kernel
  int use_union;            // batch > 1 reads weights once for the union of the tokens' masks
  unsigned long long* trace;  // optional phase time stamps of the persistent kernel (debug)
  unsigned spin_limit;      // polls after which a device-side wait gives up
  unsigned bar_bias;        // test knob: keeps the grid barrier of the persistent kernel from completing
  int* host_flag;           // pinned, mapped word the kernels set when a wait expires
  int* host_flag_dev;
  // batch > 1: unions of the tokens' masks (allocated when max_batch > 1)
  int* u_in; int* u_ch;     // [D], [F] ascending union lists
  int* u_cnt;               // [0] union inputs, [1] union channels
  float* xu;                // [D][8]  x of every token at a union input (0 if dropped)
  float* member;            // [F][8]  1 / 0 membership of every token at a union channel
  float* hb;                // [F][8]  h of every token at a union channel
  float* gacc;              // [F rounded up to 16][2][8] gate / up pre-activations (tensor-core batch path), kept at zero
  int use_mma;              // batch > 1: Stage 2 and the 4-bit proxy GEMM run on the tensor cores
  float* pacc;              // [8 tokens][gate | up][F] proxy sums of the tensor-core batch path, kept at zero
  int mask_policy;          // batch > 1: 0 = every token its own channel mask, 1 = one mask from the summed scores
  int cmask_marked;         // Stage 1 of the running forward call has set the tokens' bits in cmask already
  unsigned* cmask;          // [F / 4] one byte per channel: which tokens kept it (kept at zero between calls)
  uint8_t* umask;           // [F] that byte for every union row
  __half* xh;               // [8][D] masked, scaled fp16 x of the tensor-core proxy GEMM
  float* tokfac;            // [8] per token: what undoes its scaling
  uint32_t* xd;             // [D][8] digit words of the tokens' masked inputs (tcgen05 proxy GEMM)
  float* soffb;             // [D / 128][8] per 128-input unit and token: sum of the integer inputs
  CUtensorMap pmap;         // the packed proxy as a 2-D byte tensor (TMA descriptor of the batched Stage 1)
  const void* pmap_P; int pmap_row_bytes, pmap_D;   // what pmap was encoded for
  void* x_stage;            // device staging for the host-buffer entry point
  void* y_stage;
  int64_t launches;
  bool profiling;
  std::vector<ProfRec>* prof;
};

namespace {

#define CK(expr)                                   \
  do {                                             \
    cudaError_t e_ = (expr);                       \
    if (e_ != cudaSuccess) return map_cuda(e_);    \
  } while (0)

thread_local cudaError_t g_last_cuda = cudaSuccess;

prox_status_t map_cuda(cudaError_t e) {
  g_last_cuda = e;
  (void)cudaGetLastError();                       // do not leave a sticky-looking launch error behind
  if (e == cudaErrorMemoryAllocation) return PROX_ERR_OOM;
  return PROX_ERR_CUDA;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int ch_per_chunk(int bits) { return bits == 4 ? 16 : (bits == 8 ? 8 : 4); }

template <typename T>
cudaError_t dev_alloc(T** p, size_t count) {
  *p = nullptr;
  return cudaMalloc(reinterpret_cast<void**>(p), count * sizeof(T) > 0 ? count * sizeof(T) : 16);
}

void free_packed(prox_ffn* h) {
  cudaFree(h->P); cudaFree(h->S); cudaFree(h->s_plain); cudaFree(h->wdt);
  h->P = nullptr; h->S = nullptr; h->s_plain = nullptr; h->wdt = nullptr;
  h->quantized = false;
}

prox_status_t alloc_packed(prox_ffn* h, int bits, int group_len) {
  const int D = h->cfg.d_model, F = h->cfg.d_ff;
  free_packed(h);
  h->bits = bits;
  h->group = group_len;
  const int CH = ch_per_chunk(bits);
  const int nchunks = F / CH, ngroups = D / group_len;
  h->p_bytes = (size_t)D * nchunks * 16;
  h->s_count = (size_t)ngroups * nchunks * 2 * CH;
  CK(dev_alloc(&h->P, h->p_bytes));
  CK(dev_alloc(&h->S, h->s_count));
  CK(dev_alloc(&h->s_plain, (size_t)2 * F * ngroups));
  CK(dev_alloc(&h->wdt, (size_t)F * D));
  return PROX_OK;
}

int nstrips_for(int F, int bits) {
  const int per_strip = 32 * ch_per_chunk(bits);
  return (F + per_strip - 1) / per_strip;
}

// Row split of the step-wise proxy GEMV: as many blocks as are resident at once (one wave; a few
// blocks more would run as a second wave and double the time).
int ksplit_for(const prox_ffn* h, int B, int n_rows) {
  const int ns = nstrips_for(h->cfg.d_ff, h->bits);
  static int occ[3] = {0, 0, 0};
  const int fi = h->bits == 4 ? 0 : (h->bits == 8 ? 1 : 2);
  if (!occ[fi]) {
    int nb = 0;
    const void* fn = fi == 0 ? (const void*)proxy_gemv_kernel<4> : fi == 1 ? (const void*)proxy_gemv_kernel<8>
                                                                           : (const void*)proxy_gemv_kernel<16>;
    const size_t smem = (size_t)kProxyWarps * 2 * ch_per_chunk(h->bits) * 32 * sizeof(float);
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, fn, kProxyThreads, smem) != cudaSuccess || nb < 1) nb = 1;
    occ[fi] = nb;
  }
  const int target = occ[fi] * h->sm_count;
  int ks = target / (ns * B);
  const int by_rows = n_rows / 32 > 1 ? n_rows / 32 : 1;   // keep >= 4 rows per warp
  if (ks > by_rows) ks = by_rows;
  if (ks > 32) ks = 32;
  if (ks < 1) ks = 1;
  return ks;
}

// Function attributes (dynamic shared memory limits) are per device: one flag per (call site, device).
enum AttrSite { kAtGateupBatch = 0, kAtBatchS1, kAtProxyB4, kAtProxyB8, kAtMma, kAtRows, kAtStage2, kAtFused0, kAtSites = 24 };
bool& attr_done(int site, int device) {
  static bool done[kAtSites][64] = {};
  return done[site][device & 63];
}

prox_status_t check_common(const prox_ffn* h, const void* x, int B) {
  if (!h || !x) return PROX_ERR_INVALID_ARG;
  int cur = -1;
  if (cudaGetDevice(&cur) != cudaSuccess || cur != h->device) return PROX_ERR_INVALID_ARG;   // the handle's GPU must be current
  if (B < 1 || B > h->cfg.max_batch) return PROX_ERR_INVALID_ARG;
  if (!aligned16(x)) return PROX_ERR_INVALID_ARG;
  return PROX_OK;
}

// Launch with programmatic stream serialization: the kernel is set up while its predecessor on the stream still
// runs and waits for it (pdl_enter in the kernel) before it touches anything; the chain of small kernels of the
// batch path then runs without the launch gaps between them.  Falls back to a plain launch if refused.
template <typename... KArgs, typename... Args>
cudaError_t launch_dep(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  static int use_pdl = getenv("PROX_NO_PDL") ? 0 : 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = use_pdl ? 1 : 0;
  cudaError_t e = cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
  if (e != cudaSuccess && use_pdl) {
    (void)cudaGetLastError();
    use_pdl = 0; cfg.numAttrs = 0;
    e = cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
  }
  return e;
}

// Brackets one launch with events when the handle's timing hook is on.
struct LaunchScope {
  prox_ffn* h; cudaStream_t st; ProfRec rec; bool on;
  LaunchScope(prox_ffn* h_, int kind, cudaStream_t st_) : h(h_), st(st_), on(h_->profiling) {
    rec.kind = kind; rec.a = rec.b = nullptr;
    if (on) {
      if (cudaEventCreate(&rec.a) != cudaSuccess || cudaEventCreate(&rec.b) != cudaSuccess) { on = false; return; }
      cudaEventRecord(rec.a, st);
    }
  }
  ~LaunchScope() {
    h->launches++;
    if (on) { cudaEventRecord(rec.b, st); h->prof->push_back(rec); }
  }
};

// ---- launches ---------------------------------------------------------------
prox_status_t launch_input_select(prox_ffn* h, const void* x, int B, int k1, float tau, int use_tau,
                                  int* idx, int stride, int* cnt, cudaStream_t st) {
  {
    LaunchScope ls(h, kKInput, st);
    input_select_kernel<<<B, kSelThreads, 0, st>>>(static_cast<const uint16_t*>(x), h->cfg.d_model, k1,
                                                   tau, use_tau, idx, stride, cnt);
  }
  CK(cudaGetLastError());
  return PROX_OK;
}

prox_status_t launch_proxy(prox_ffn* h, const void* x, int B, const int* idx, int stride,
                           const int* cnt, int k1, float* scores, cudaStream_t st, float* values = nullptr) {
  const int D = h->cfg.d_model, F = h->cfg.d_ff;
  const int ns = nstrips_for(F, h->bits);
  const int ks = ksplit_for(h, B, k1);
  const int gshift = (h->group == D) ? 31 : 7;
  dim3 grid(ns, ks, B);
  const size_t need = (size_t)B * ks * ns * 2 * ch_per_chunk(h->bits) * 32;
  if (ks > 1 && need > h->part_floats) return PROX_ERR_UNSUPPORTED;
  LaunchScope ls(h, kKProxy, st);
  if (h->bits == 4) {
    const size_t smem = (size_t)kProxyWarps * ProxyFmt<4>::NACC * 32 * sizeof(float);
    proxy_gemv_kernel<4><<<grid, kProxyThreads, smem, st>>>(
        h->P, h->S, static_cast<const uint16_t*>(x), idx, stride, cnt, k1, D, F, gshift, h->part,
        h->ticket, scores, values, h->dev_status);
  } else if (h->bits == 8) {
    const size_t smem = (size_t)kProxyWarps * ProxyFmt<8>::NACC * 32 * sizeof(float);
    proxy_gemv_kernel<8><<<grid, kProxyThreads, smem, st>>>(
        h->P, h->S, static_cast<const uint16_t*>(x), idx, stride, cnt, k1, D, F, gshift, h->part,
        h->ticket, scores, values, h->dev_status);
  } else {
    const size_t smem = (size_t)kProxyWarps * ProxyFmt<16>::NACC * 32 * sizeof(float);
    proxy_gemv_kernel<16><<<grid, kProxyThreads, smem, st>>>(
        h->P, h->S, static_cast<const uint16_t*>(x), idx, stride, cnt, k1, D, F, gshift, h->part,
        h->ticket, scores, values, h->dev_status);
  }
  CK(cudaGetLastError());
  return PROX_OK;
}

prox_status_t launch_channel_select(prox_ffn* h, const float* scores, int B, int k2, float tau,
                                    int use_tau, int* sel, int stride, int* cnt, cudaStream_t st) {
  {
    LaunchScope ls(h, kKChannel, st);
    channel_select_kernel<<<B, kSelThreads, 0, st>>>(scores, h->cfg.d_ff, k2, tau, use_tau, sel, stride, cnt);
  }
  CK(cudaGetLastError());
  return PROX_OK;
}

prox_status_t launch_down(prox_ffn* h, int B, const int* sel, int stride, const int* cnt, int k2, void* y,
                          cudaStream_t st);

prox_status_t launch_stage2(prox_ffn* h, const void* x, int B, const int* sel, int stride,
                            const int* cnt, int k2, void* y, cudaStream_t st) {
  const int D = h->cfg.d_model, F = h->cfg.d_ff;
  const int wpb = kGateUpThreads / 32;
  dim3 g1((k2 + wpb - 1) / wpb, B);
  {
    LaunchScope ls(h, kKGateUp, st);
    gateup_kernel<<<g1, kGateUpThreads, (size_t)D * 2, st>>>(
        h->wg, h->wu, static_cast<const uint16_t*>(x), sel, stride, cnt, k2, D, F, h->hbuf, F,
        h->dev_status);
  }
  CK(cudaGetLastError());
  return launch_down(h, B, sel, stride, cnt, k2, y, st);
}

prox_status_t launch_down(prox_ffn* h, int B, const int* sel, int stride, const int* cnt, int k2, void* y,
                          cudaStream_t st) {
  const int D = h->cfg.d_model, F = h->cfg.d_ff;
  const int dtiles = (D + kDownThreads * 8 - 1) / (kDownThreads * 8);
  int nsplit = (2 * h->sm_count + dtiles * B - 1) / (dtiles * B);
  if (nsplit > k2) nsplit = k2;
  if (nsplit < 1) nsplit = 1;
  dim3 g2(dtiles, nsplit, B);
  {
    LaunchScope ls(h, kKDown, st);
    down_kernel<<<g2, kDownThreads, 0, st>>>(h->wdt, h->hbuf, F, sel, stride, cnt, k2, D, F, h->yacc);
  }
  CK(cudaGetLastError());
  const int n = B * D;
  {
    LaunchScope ls(h, kKFinalize, st);
    finalize_kernel<<<(n + 255) / 256, 256, 0, st>>>(h->yacc, h->fin_resid ? (void*)h->fin_out : y, n,
                                                     h->cfg.out_dtype, h->fin_resid);
  }
  CK(cudaGetLastError());
  return PROX_OK;
}

// ---- batch > 1: union path -----------------------------------------------------
bool batch_path_ok(const prox_ffn* h, int B, bool stage1 = false) {
  if (B < 2 || !h->u_in) return false;
  if (stage1 && h->bits == 16) return false;             // the batch Stage 1 reads integer proxies
  const size_t xs_bytes = (size_t)B * h->cfg.d_model * 2;
  const size_t red_bytes = (size_t)4 * kBT * 128 * (h->bits == 4 ? 8 : 4) * sizeof(float);
  const size_t ubits = (size_t)(B + 2) * ((h->cfg.d_ff + 31) / 32) * 4;
  const size_t lim = (size_t)h->smem_optin - 4096;
  return xs_bytes <= lim && red_bytes <= lim && ubits <= lim;
}

prox_status_t launch_union(prox_ffn* h, const int* lists, int stride, const int* cnt, int k, int B, int n,
                           const void* x, int* ulist, int* nu, float* val, cudaStream_t st) {
  const size_t smem = (size_t)(B + 2) * ((n + 31) / 32) * sizeof(unsigned);
  bool& attr = attr_done(kAtStage2, h->device);
  if (!attr) { CK(cudaFuncSetAttribute(union_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, h->smem_optin - 4096)); attr = true; }
  {
    LaunchScope ls(h, kKUnion, st);
    union_kernel<<<1, 1024, smem, st>>>(lists, stride, cnt, k, B, n, static_cast<const uint16_t*>(x), ulist, nu, val,
                                        h->dev_status);
  }
  CK(cudaGetLastError());
  return PROX_OK;
}

// the tensor-core Stage 2 needs x of eight tokens (padded rows) plus a reduction buffer in shared memory
size_t stage2_mma_smem(const prox_ffn* h) {
  return (size_t)8 * (h->cfg.d_model * 2 + kXPad) + (size_t)kMmaWarps * 256 * sizeof(float);
}
bool stage2_mma_ok(const prox_ffn* h) {
  return h->use_mma && h->gacc && stage2_mma_smem(h) <= (size_t)h->smem_optin - 4096;
}

// TMA descriptor of the packed proxy rows: bytes [D][row_bytes], box = 128 bytes x 128 rows, 128-byte swizzle
// (what the integer MMA's A operand wants).  The driver entry point is looked up at run time: the library
// does not link against the driver.
prox_status_t ensure_pmap(prox_ffn* h, int row_bytes) {
  const int D = h->cfg.d_model;
  if (h->pmap_P == h->P && h->pmap_row_bytes == row_bytes && h->pmap_D == D) return PROX_OK;
  typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static encode_fn encode = nullptr;
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qr;
    CK(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr));
    if (!fn || qr != cudaDriverEntryPointSuccess) return PROX_ERR_UNSUPPORTED;
    encode = reinterpret_cast<encode_fn>(fn);
  }
  const cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)D};
  const cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
  const cuuint32_t box[2] = {128u, 128u}, estr[2] = {1u, 1u};
  const CUresult r = encode(&h->pmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(h->P), dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return PROX_ERR_CUDA;
  h->pmap_P = h->P; h->pmap_row_bytes = row_bytes; h->pmap_D = D;
  return PROX_OK;
}

// mark_mask: also set the tokens' bits in the per-channel bytes that the tensor-core Stage 2 of the
// SAME call turns into the union (only prox_ffn_forward asks for it: the bytes must be consumed)
prox_status_t launch_stage1_batch(prox_ffn* h, const void* x, int B, int k1, int k2, int* sel, int sel_stride,
                                  float* scores, cudaStream_t st, bool mark_mask = false, bool want_scores = true) {
  h->cmask_marked = 0;
  const int D = h->cfg.d_model, F = h->cfg.d_ff;
  prox_status_t s;
  const int gshift_m = (h->group == D) ? 31 : 7;
  if (h->use_mma && h->pacc && (h->bits == 4 || h->bits == 8) && F % 64 == 0) {
    // tensor-core path over all inputs (no union list): per-token masked, scaled fp16 x, then equal
    // ranges of (strip, K-block) units per block, then the per-token channel masks
    const size_t lim = (size_t)h->smem_optin - 16384;
    const bool fast_masks = (size_t)D * 2 <= lim && (size_t)F * 4 <= lim;
    bool& attr_p = attr_done(kAtBatchS1, h->device);
    if (!attr_p) {
      CK(cudaFuncSetAttribute(proxy_umma_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, kBuSmem4));
      CK(cudaFuncSetAttribute(proxy_umma_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, kBuSmem8));
      CK(cudaFuncSetAttribute(batch_input_mask_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lim));
      CK(cudaFuncSetAttribute(batch_channel_mask_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lim));
      attr_p = true;
    }
    if (fast_masks) {
      LaunchScope ls(h, kKInput, st);
      CK(launch_dep(batch_input_mask_kernel, dim3(kBT), dim3(kFusedThreads), (size_t)D * 2, st, static_cast<const uint16_t*>(x), B, D, k1,
                    h->xh, h->tokfac, h->xd, h->soffb));
    } else {
      if ((s = launch_input_select(h, x, B, k1, 0.f, 0, h->idx_x, D, nullptr, st)) != PROX_OK) return s;
      LaunchScope ls(h, kKInput, st);
      proxy_xprep_kernel<<<kBT, 512, 0, st>>>(static_cast<const uint16_t*>(x), h->idx_x, D, k1, B, D, h->xh, h->tokfac);
      batch_digits_kernel<<<kBT, 512, 0, st>>>(h->xh, D, h->xd, h->soffb);
    }
    bool direct = false;
    {
      LaunchScope ls(h, kKProxy, st);
      const int row_bytes = (F / ch_per_chunk(h->bits)) * 16, ntiles = (row_bytes + 127) / 128, nunits = D / 128;
      int usplit = (2 * h->sm_count + ntiles - 1) / ntiles;
      if (usplit > nunits) usplit = nunits;
      if (usplit < 1) usplit = 1;
      const int nitems = ntiles * usplit;
      const int grid = nitems < h->sm_count ? nitems : h->sm_count;
      const size_t smem = (size_t)(h->bits == 4 ? kBuSmem4 : kBuSmem8);
      if ((s = ensure_pmap(h, row_bytes)) != PROX_OK) return s;
      {
        // programmatic dependent launch: the kernel sets up and requests its first weight tiles while the
        // kernel that masks the inputs still runs; it waits for that kernel before it reads anything of this call
        static int use_pdl = getenv("PROX_NO_PDL") ? 0 : 1;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3(kBuThreads); cfg.dynamicSmemBytes = smem; cfg.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = at; cfg.numAttrs = use_pdl ? 1 : 0;
        const __half* Sp = h->S; const uint32_t* xdp = h->xd; const float* sop = h->soffb; const float* tfp = h->tokfac;
        int Dv = D, Fv = F, gs = gshift_m, us = usplit; float* pa = h->pacc; int* stp = h->dev_status;
        void* args[] = {&h->pmap, &Sp, &xdp, &sop, &tfp, &Dv, &Fv, &gs, &us, &pa, &stp};
        const void* fn = h->bits == 4 ? reinterpret_cast<const void*>(&proxy_umma_kernel<4>) : reinterpret_cast<const void*>(&proxy_umma_kernel<8>);
        cudaError_t e = cudaLaunchKernelExC(&cfg, fn, args);
        if (e != cudaSuccess && use_pdl) {              // attribute not accepted here: plain launch from now on
          (void)cudaGetLastError();
          use_pdl = 0; cfg.numAttrs = 0;
          e = cudaLaunchKernelExC(&cfg, fn, args);
        }
        CK(e);
      }
      direct = fast_masks && !want_scores;
      if (!direct) CK(launch_dep(proxy_umma_finish_kernel, dim3(2 * h->sm_count), dim3(256), 0, st, h->pacc, B, F, scores));
    }
    CK(cudaGetLastError());
    if (h->mask_policy == 1) {
      if (!fast_masks) return PROX_ERR_UNSUPPORTED;
      LaunchScope ls(h, kKChannel, st);
      if (direct) CK(launch_dep(shared_score_from_sums_kernel, dim3((F + 255) / 256), dim3(256), 0, st, h->pacc, B, F, h->svals));
      else CK(launch_dep(shared_score_kernel, dim3((F + 255) / 256), dim3(256), 0, st, (const float*)scores, B, F, h->svals));
      if ((size_t)F * 4 + (size_t)k2 * 4 <= lim) {
        // the one block also writes the list into every token's row
        CK(launch_dep(batch_channel_mask_kernel, dim3(1), dim3(kCmThreads), (size_t)F * 4 + (size_t)k2 * 4, st, (const float*)h->svals, F, k2, sel,
                      sel_stride, (unsigned*)nullptr, (1u << B) - 1u, (float*)nullptr, B, mark_mask ? h->u_ch : (int*)nullptr, h->umask,
                      h->u_cnt + 1));
        CK(cudaGetLastError());
        if (mark_mask) h->cmask_marked = 2;          // the union is listed already: it is the mask itself
        return PROX_OK;
      } else {
        CK(launch_dep(batch_channel_mask_kernel, dim3(1), dim3(kCmThreads), (size_t)F * 4, st, (const float*)h->svals, F, k2, sel, sel_stride,
                      mark_mask ? h->cmask : (unsigned*)nullptr, (1u << B) - 1u, (float*)nullptr, 1, (int*)nullptr, (uint8_t*)nullptr,
                      (int*)nullptr));
        CK(launch_dep(replicate_mask_kernel, dim3((k2 + 255) / 256), dim3(256), 0, st, sel, sel_stride, k2, B));
      }
      CK(cudaGetLastError());
      if (mark_mask) h->cmask_marked = 1;
      return PROX_OK;
    }
    if (!fast_masks) return launch_channel_select(h, scores, B, k2, 0.f, 0, sel, sel_stride, nullptr, st);
    {
      LaunchScope ls(h, kKChannel, st);
      CK(launch_dep(batch_channel_mask_kernel, dim3(B), dim3(kCmThreads), (size_t)F * 4, st, (const float*)scores, F, k2, sel, sel_stride,
                    mark_mask ? h->cmask : (unsigned*)nullptr, 0u, (direct && h->mask_policy == 0) ? h->pacc : (float*)nullptr, 1,
                    (int*)nullptr, (uint8_t*)nullptr, (int*)nullptr));
    }
    CK(cudaGetLastError());
    if (mark_mask) h->cmask_marked = 1;
    return PROX_OK;
  }
  if (h->mask_policy == 1) return PROX_ERR_UNSUPPORTED;      // the shared mask is built by the tensor-core path only
  if ((s = launch_input_select(h, x, B, k1, 0.f, 0, h->idx_x, D, nullptr, st)) != PROX_OK) return s;
  if ((s = launch_union(h, h->idx_x, D, nullptr, k1, B, D, x, h->u_in, h->u_cnt, h->xu, st)) != PROX_OK) return s;
  const int ns = nstrips_for(F, h->bits);
  const int nval = 128 * (h->bits == 4 ? 8 : 4);
  int ks = h->sm_count / ns;
  if (ks < 1) ks = 1;
  if (ks > 16) ks = 16;
  while (ks > 1 && (size_t)ks * ns * kBT * nval > h->part_floats) --ks;
  if ((size_t)ks * ns * kBT * nval > h->part_floats && ks > 1) return PROX_ERR_UNSUPPORTED;
  const size_t smem = (size_t)4 * kBT * nval * sizeof(float);
  const int gshift = (h->group == D) ? 31 : 7;
  dim3 grid(ns, ks);
  {
    LaunchScope ls(h, kKProxy, st);
    if (h->bits == 4) {
      bool& attr4 = attr_done(kAtProxyB4, h->device);
      if (!attr4) { CK(cudaFuncSetAttribute(proxy_batch_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); attr4 = true; }
      proxy_batch_kernel<4><<<grid, kPBThreads, smem, st>>>(h->P, h->S, h->u_in, h->u_cnt, h->xu, B, D, F, gshift,
                                                           h->part, h->ticket, scores);
    } else {
      bool& attr8 = attr_done(kAtProxyB8, h->device);
      if (!attr8) { CK(cudaFuncSetAttribute(proxy_batch_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); attr8 = true; }
      proxy_batch_kernel<8><<<grid, kPBThreads, smem, st>>>(h->P, h->S, h->u_in, h->u_cnt, h->xu, B, D, F, gshift,
                                                           h->part, h->ticket, scores);
    }
  }
  CK(cudaGetLastError());
  return launch_channel_select(h, scores, B, k2, 0.f, 0, sel, sel_stride, nullptr, st);
}

prox_status_t launch_stage2_batch(prox_ffn* h, const void* x, int B, const int* sel, int sel_stride, int k2,
                                  void* y, cudaStream_t st, bool marked = false) {
  const int D = h->cfg.d_model, F = h->cfg.d_ff;
  prox_status_t s;
  const size_t mma_smem = stage2_mma_smem(h);
  const bool mma = stage2_mma_ok(h);
  if (mma) {
    LaunchScope ls(h, kKUnion, st);
    const int listed = marked ? h->cmask_marked : 0;       // 1: bits set by Stage 1 of this call, 2: the union list is there already
    h->cmask_marked = 0;
    if (!listed)
      CK(launch_dep(union_mark_kernel, dim3((B * k2 + 255) / 256), dim3(256), 0, st, sel, sel_stride, k2, B, F, h->cmask, h->dev_status));
    if (listed != 2) {
      const size_t need = (size_t)F * 5 + 16;
      const int staged = need <= (size_t)h->smem_optin - 4096 ? 1 : 0;
      bool& attr_u = attr_done(kAtFused0, h->device);
      if (!attr_u) { CK(cudaFuncSetAttribute(union_compact_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, h->smem_optin - 4096)); attr_u = true; }
      CK(launch_dep(union_compact_kernel, dim3(1), dim3(1024), staged ? need : (size_t)0, st, h->cmask, F, h->u_ch, h->u_cnt + 1, h->umask, staged));
    }
    CK(cudaGetLastError());
  } else if ((s = launch_union(h, sel, sel_stride, nullptr, k2, B, F, nullptr, h->u_ch, h->u_cnt + 1, h->member, st)) != PROX_OK) {
    return s;
  }
  if (mma) {
    // tensor-core path: equal ranges of weight units per block, two blocks per SM for gate/up
    bool& attr_mma = attr_done(kAtMma, h->device);
    if (!attr_mma) {
      CK(cudaFuncSetAttribute(gateup_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, h->smem_optin - 4096));
      CK(cudaFuncSetAttribute(down_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, h->smem_optin - 4096));
      attr_mma = true;
    }
    const int per_sm = (2 * (mma_smem + 1024) <= (size_t)h->smem_optin) ? 2 : 1;
    // whole rows through a ring of bulk copies when 16 of them (a tile) plus a few more fit in shared memory
    const size_t row_pitch = (size_t)(D * 2 < kGrPiece ? D * 2 : kGrPiece) + 64;
    int ring_slots = (int)(((size_t)h->smem_optin - 4096 - (size_t)kMmaWarps * 128 * sizeof(float)) / row_pitch);
    if (ring_slots > kGrMaxSlots) ring_slots = kGrMaxSlots;
    {
      LaunchScope ls(h, kKGateUp, st);
      if (D % 512 == 0 && D <= 4096 && ring_slots >= 40) {
        bool& attr_r = attr_done(kAtRows, h->device);
        if (!attr_r) {
          CK(cudaFuncSetAttribute(gateup_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, h->smem_optin - 4096));
          attr_r = true;
        }
        CK(launch_dep(gateup_rows_kernel, dim3(h->sm_count), dim3(kGrThreads),
                      (size_t)ring_slots * row_pitch + (size_t)kMmaWarps * 128 * sizeof(float), st,
                      h->wg, h->wu, static_cast<const uint16_t*>(x), B, h->u_ch, h->umask, h->u_cnt + 1, D, ring_slots, h->hb,
                      h->dev_status));
      } else {
        gateup_mma_kernel<<<per_sm * h->sm_count, kMmaThreads, mma_smem, st>>>(
            h->wg, h->wu, static_cast<const uint16_t*>(x), B, h->u_ch, h->u_cnt + 1, D, h->gacc);
        gateup_finish_kernel<<<h->sm_count, 256, 0, st>>>(h->gacc, h->umask, h->u_cnt + 1, B, h->hb);
      }
    }
    CK(cudaGetLastError());
    {
      LaunchScope ls(h, kKDown, st);
      CK(launch_dep(down_mma_kernel, dim3(h->sm_count), dim3(kMmaThreads), (size_t)kMmaWarps * 512 * sizeof(float), st,
                    h->wdt, h->hb, h->u_ch, h->u_cnt + 1, B, D, h->yacc));
    }
    CK(cudaGetLastError());
  } else {
  const size_t smem = (size_t)B * D * 2;
  bool& attr = attr_done(kAtGateupBatch, h->device);
  if (!attr) { CK(cudaFuncSetAttribute(gateup_batch_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, h->smem_optin - 4096)); attr = true; }
  int blocks = (F + kGBThreads / 32 - 1) / (kGBThreads / 32);
  const int cap = 8 * h->sm_count;
  if (blocks > cap) blocks = cap;
  {
    LaunchScope ls(h, kKGateUp, st);
    gateup_batch_kernel<<<blocks, kGBThreads, smem, st>>>(h->wg, h->wu, static_cast<const uint16_t*>(x), B, h->u_ch,
                                                         h->u_cnt + 1, h->member, D, F, h->hb);
  }
  CK(cudaGetLastError());
  const int dtiles = (D + kDownThreads * 8 - 1) / (kDownThreads * 8);
  int nsplit = (h->sm_count + dtiles - 1) / dtiles;
  if (nsplit < 1) nsplit = 1;
  dim3 g2(dtiles, nsplit);
  {
    LaunchScope ls(h, kKDown, st);
    down_batch_kernel<<<g2, kDownThreads, 0, st>>>(h->wdt, h->hb, h->u_ch, h->u_cnt + 1, B, D, h->yacc);
  }
  CK(cudaGetLastError());
  }
  const int n = B * D;
  {
    LaunchScope ls(h, kKFinalize, st);
    CK(launch_dep(finalize_kernel, dim3((n + 255) / 256), dim3(256), 0, st, h->yacc, h->fin_resid ? (void*)h->fin_out : y, n,
                  h->cfg.out_dtype, (const float*)h->fin_resid));
  }
  CK(cudaGetLastError());
  return PROX_OK;
}

// ---- fused persistent kernel (batch 1) ----------------------------------------
struct FusedPlan {
  bool ok;
  int grid, pstages, big_bytes, nslots, xch;
  size_t smem;
  int device;           // the handle's GPU
  int optin;            // the device's opt-in limit: what the kernels' dynamic shared memory attribute is set to
};

FusedPlan plan_fused(const prox_ffn* h, int k1, int k2, bool thresh = false) {
  FusedPlan pl;
  std::memset(&pl, 0, sizeof(pl));
  const int D = h->cfg.d_model, F = h->cfg.d_ff;
  if (!h->use_fused || !h->coop || h->bits == 16) return pl;       // the fused kernel reads integer proxies
  const int G = h->sm_count;
  const size_t fixed = ((sizeof(FusedSmem) + 127) & ~size_t(127)) + (size_t)8 * D;   // + x bf16, idx, x fp32
  if ((size_t)h->smem_optin < fixed + (size_t)6 * D + 16384) return pl;
  pl.big_bytes = (int)(((size_t)h->smem_optin - fixed) & ~size_t(127));
  pl.nslots = pl.big_bytes / (2 * D);
  if (pl.nslots > kMaxSlots) pl.nslots = kMaxSlots;
  if (pl.nslots < 3) return pl;
  // the proxy GEMV keeps 16 tensor-memory columns per supergroup (4 scale groups), two sets of up to 256
  if ((D / h->group + 3) / 4 > kMaxSuper) return pl;
  pl.pstages = (pl.big_bytes - 1024 - 3072) / kPStageBytes;
  if (pl.pstages > kPStages) pl.pstages = kPStages;
  if (pl.pstages < kPStages) return pl;                                   // every loader warp owns a stage
  if (pl.big_bytes < 4 * D * 4) return pl;                                // partial y vectors of the down projection
  if ((k2 + G - 1) / G + 2 > kMySelCap) return pl;       // a block's share: definite part + part of the threshold bin
  if (thresh) {
    // any number of channels may pass the threshold: a block's share of all of them must fit, the scores
    // must fit in shared memory (no radix fallback in this form), counts are kept in 16 bits
    if ((F + G - 1) / G + 2 > kMySelCap || (size_t)F * 4 + 256 > (size_t)pl.big_bytes || F >= 65536) return pl;
  }
  (void)k1;
  pl.grid = G;
  pl.xch = D <= 4096 ? 4 : (D <= 8192 ? 2 : 1);          // warp groups of the down projection
  pl.smem = fixed + (size_t)pl.big_bytes;
  pl.optin = h->smem_optin;
  pl.device = h->device;
  pl.ok = true;
  return pl;
}

template <int BITS, int NG, bool NORM, bool THRESH>
cudaError_t launch_fused_tn(const FusedPlan& pl, const FusedParams& prm, cudaStream_t st) {
  static bool attr_dev[64] = {};     // per instantiation and device: the attribute belongs to the function on a device
  auto kern = prox_fused_kernel<BITS, NG, NORM, THRESH>;
  bool& attr_set = attr_dev[pl.device & 63];
  if (!attr_set) {
    // the limit, not this plan's size: another handle's shape may need a few bytes more
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.optin);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  cudaLaunchConfig_t cfg;
  std::memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(pl.grid);
  cfg.blockDim = dim3(kFusedThreads);
  cfg.dynamicSmemBytes = pl.smem;
  cfg.stream = st;
  // Cooperative (all blocks co-resident: the kernel has a grid barrier) and, if the driver takes the two
  // together, programmatic stream serialization: the next launch on the stream is set up while this one
  // drains, and its blocks wait (griddepcontrol.wait) for this grid to complete before they read anything.
  static int use_pdl = getenv("PROX_NO_PDL") ? 0 : 1;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeCooperative;
  at[0].val.cooperative = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = use_pdl ? 2 : 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, kern, prm);
  if (e != cudaSuccess && use_pdl) {
    (void)cudaGetLastError();
    use_pdl = 0;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, kern, prm);
  }
  return e;
}

template <int BITS, int NG>
cudaError_t launch_fused_t(const FusedPlan& pl, const FusedParams& prm, cudaStream_t st) {
  if (prm.count_out)                                                                   // threshold form
    return prm.xres ? launch_fused_tn<BITS, NG, true, true>(pl, prm, st)
                    : launch_fused_tn<BITS, NG, false, true>(pl, prm, st);
  return prm.xres ? launch_fused_tn<BITS, NG, true, false>(pl, prm, st)
                  : launch_fused_tn<BITS, NG, false, false>(pl, prm, st);
}

// 1/d_model and eps as pairs of floats for the device-side RMSNorm
RmsConst rms_const(int D, double eps) {
  RmsConst c;
  const double inv_d = 1.0 / (double)D;
  c.idh = (float)inv_d; c.idl = (float)(inv_d - (double)c.idh);
  c.eh = (float)eps; c.el = (float)(eps - (double)c.eh);
  return c;
}

prox_status_t launch_fused(prox_ffn* h, const FusedPlan& pl, const void* x, int k1, int k2, void* y,
                           int* sel_out, cudaStream_t st, const float* xres = nullptr,
                           const uint16_t* norm_w = nullptr, double eps = 0.0, float* xres_out = nullptr,
                           const float* taus = nullptr) {
  FusedParams prm;
  std::memset(&prm, 0, sizeof(prm));
  prm.P = h->P; prm.S = h->S; prm.wg = h->wg; prm.wu = h->wu; prm.wdt = h->wdt;
  prm.x = static_cast<const uint16_t*>(x); prm.y = y;
  prm.D = h->cfg.d_model; prm.F = h->cfg.d_ff; prm.k1 = k1; prm.k2 = k2;
  prm.gshift = (h->group == h->cfg.d_model) ? 31 : 7;
  prm.out_fp32 = h->cfg.out_dtype;
  prm.pstages = pl.pstages;
  prm.scores = h->scores; prm.ghist = h->syncbuf; prm.idx_out = h->idx_x;
  prm.spin_limit = h->spin_limit; prm.bar_bias = h->bar_bias; prm.host_flag = h->host_flag_dev;
  prm.sel_out = sel_out; prm.yacc = h->yacc;
  prm.bar_count = reinterpret_cast<unsigned long long*>(h->syncbuf + 4096); prm.done_ticket = h->syncbuf + 4098;
  prm.status = h->dev_status;
  prm.big_bytes = pl.big_bytes; prm.nslots = pl.nslots;
  prm.trace = h->trace;
  prm.xres = xres; prm.norm_w = norm_w; prm.rc = rms_const(h->cfg.d_model, eps); prm.xres_out = xres_out;
  if (taus) {
    // |x| >= tau_x  <=>  15-bit bf16 magnitude >= ceil(bits(tau_x) / 2^16);  score >= tau_s  <=>  bits >= bits
    uint32_t bx, bs;
    const float tx = std::fabs(taus[0]), ts = std::fabs(taus[1]);        // -0.0f is the threshold 0
    std::memcpy(&bx, &tx, 4); std::memcpy(&bs, &ts, 4);
    prm.tkey_x = (bx >> 16) + ((bx & 0xffffu) ? 1u : 0u);
    prm.tkey_s = bs;
    prm.cnt_x_out = h->cnt_x; prm.count_out = h->cnt_s; prm.counters = h->counters;
  }
  cudaError_t e;
  {
    LaunchScope ls(h, kKFused, st);
    if (h->bits == 4) {
      e = pl.xch == 4 ? launch_fused_t<4, 4>(pl, prm, st)
        : pl.xch == 2 ? launch_fused_t<4, 2>(pl, prm, st) : launch_fused_t<4, 1>(pl, prm, st);
    } else {
      e = pl.xch == 4 ? launch_fused_t<8, 4>(pl, prm, st)
        : pl.xch == 2 ? launch_fused_t<8, 2>(pl, prm, st) : launch_fused_t<8, 1>(pl, prm, st);
    }
  }
  CK(e);
  return PROX_OK;
}

// Everything of a forward call but the persistent kernel: batch path, or the step-wise kernels.
prox_status_t forward_kernels(prox_ffn* h, const void* x, int B, int k1, int k2, void* y, cudaStream_t st) {
  prox_status_t s;
  const int D = h->cfg.d_model, F = h->cfg.d_ff;
  h->sel_unordered = 0;
  if (B > 1 && h->mask_policy == 1 && !(h->use_union && batch_path_ok(h, B, true))) return PROX_ERR_UNSUPPORTED;
  if (h->use_union && batch_path_ok(h, B, true)) {
    if ((s = launch_stage1_batch(h, x, B, k1, k2, h->sel, F, h->scores, st, stage2_mma_ok(h), false)) != PROX_OK) return s;
    return launch_stage2_batch(h, x, B, h->sel, F, k2, y, st, true);
  }
  if ((s = launch_input_select(h, x, B, k1, 0.f, 0, h->idx_x, D, nullptr, st)) != PROX_OK) return s;
  if ((s = launch_proxy(h, x, B, h->idx_x, D, nullptr, k1, h->scores, st)) != PROX_OK) return s;
  if ((s = launch_channel_select(h, h->scores, B, k2, 0.f, 0, h->sel, F, nullptr, st)) != PROX_OK) return s;
  if (h->use_union && batch_path_ok(h, B)) return launch_stage2_batch(h, x, B, h->sel, F, k2, y, st, false);
  return launch_stage2(h, x, B, h->sel, F, nullptr, k2, y, st);
}

// A block gave up on a wait: counters shared between blocks may be left half-way.  Put every one of
// them back to its idle state (the stream is idle when this runs).
prox_status_t reset_shared_state(prox_ffn* h, cudaStream_t st) {
  const int ns_max = nstrips_for(h->cfg.d_ff, 8);
  CK(cudaMemsetAsync(h->syncbuf, 0, (4096 + 64) * sizeof(unsigned), st));
  CK(cudaMemsetAsync(h->ticket, 0, (size_t)h->cfg.max_batch * ns_max * sizeof(unsigned), st));
  CK(cudaMemsetAsync(h->yacc, 0, (size_t)h->cfg.max_batch * h->cfg.d_model * sizeof(float), st));
  if (h->gacc) {                               // accumulators of the tensor-core batch path (kept at zero between calls)
    const size_t F = (size_t)h->cfg.d_ff;
    CK(cudaMemsetAsync(h->gacc, 0, ((F + 15) / 16) * 256 * sizeof(float), st));
    CK(cudaMemsetAsync(h->pacc, 0, (F / 64) * 1024 * sizeof(float), st));
    CK(cudaMemsetAsync(h->cmask, 0, ((F + 3) / 4) * sizeof(unsigned), st));
    h->cmask_marked = 0;
  }
  CK(cudaStreamSynchronize(st));
  if (h->host_flag) *h->host_flag = 0;
  return PROX_OK;
}

}  // namespace

// ============================================================================
extern "C" {

prox_status_t prox_ffn_create(const prox_ffn_config_t* cfg, const void* w_gate, const void* w_up,
                              const void* w_down, void* stream, prox_ffn_t** out) {
  (void)stream;
  if (!out) return PROX_ERR_INVALID_ARG;
  *out = nullptr;
  if (!cfg || !w_gate || !w_up || !w_down) return PROX_ERR_INVALID_ARG;
  if (!aligned16(w_gate) || !aligned16(w_up) || !aligned16(w_down)) return PROX_ERR_INVALID_ARG;
  if (cfg->max_batch < 1 || cfg->max_batch > kMaxBatch) return PROX_ERR_INVALID_ARG;
  if (cfg->out_dtype != 0 && cfg->out_dtype != 1) return PROX_ERR_INVALID_ARG;
  if (cfg->d_model <= 0 || cfg->d_ff <= 0) return PROX_ERR_INVALID_ARG;
  if (cfg->d_model % 128 || cfg->d_model > 16384) return PROX_ERR_UNSUPPORTED;
  if (cfg->d_ff % 64 || cfg->d_ff > 65536) return PROX_ERR_UNSUPPORTED;

  prox_ffn* h = new (std::nothrow) prox_ffn();
  if (!h) return PROX_ERR_OOM;
  std::memset(h, 0, sizeof(*h));
  h->prof = new (std::nothrow) std::vector<ProfRec>();
  if (!h->prof) { delete h; return PROX_ERR_OOM; }
  h->cfg = *cfg;
  h->wg = static_cast<const uint16_t*>(w_gate);
  h->wu = static_cast<const uint16_t*>(w_up);
  h->wd = static_cast<const uint16_t*>(w_down);
  cudaError_t e = cudaGetDevice(&h->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device);
  if (e != cudaSuccess) { delete h; return PROX_ERR_CUDA; }

  const int D = cfg->d_model, F = cfg->d_ff, MB = cfg->max_batch;
  const int ns_max = nstrips_for(F, 8);            // 8-bit strips are narrower -> more of them
  h->part_floats = ((size_t)2 * h->sm_count + (size_t)MB * ns_max + 64) * 1024;
  if (MB > 1) {                                    // union path: [row split][strip][8 tokens][1024]
    const size_t need = ((size_t)h->sm_count + ns_max) * kBT * 1024;
    if (need > h->part_floats) h->part_floats = need;
  }
  prox_status_t st = PROX_OK;
  auto A = [&](cudaError_t er) { if (er != cudaSuccess && st == PROX_OK) st = map_cuda(er); };
  A(dev_alloc(&h->idx_x, (size_t)MB * D));
  A(dev_alloc(&h->cnt_x, (size_t)MB));
  A(dev_alloc(&h->part, h->part_floats));
  A(dev_alloc(&h->ticket, (size_t)MB * ns_max));
  A(dev_alloc(&h->scores, (size_t)MB * F));
  A(dev_alloc(&h->svals, (size_t)MB * F));      // (allocated here, not on first use: a first use may be under graph capture)
  A(dev_alloc(&h->xn, (size_t)MB * D));
  A(dev_alloc(&h->sel, (size_t)MB * F));
  A(dev_alloc(&h->cnt_s, (size_t)MB));
  A(dev_alloc(&h->hbuf, (size_t)MB * F));
  A(dev_alloc(&h->yacc, (size_t)MB * D));
  A(dev_alloc(&h->dev_status, (size_t)1));
  A(dev_alloc(&h->counters, (size_t)4));
  A(dev_alloc(&h->syncbuf, (size_t)4096 + 64));
  if (MB > 1) {
    A(dev_alloc(&h->u_in, (size_t)D)); A(dev_alloc(&h->u_ch, (size_t)F)); A(dev_alloc(&h->u_cnt, (size_t)4));
    A(dev_alloc(&h->xu, (size_t)D * kBT)); A(dev_alloc(&h->member, (size_t)F * kBT));
    A(dev_alloc(&h->hb, (size_t)F * kBT));
    A(dev_alloc(&h->gacc, (size_t)((F + 15) / 16) * 256));
    {
      A(dev_alloc(&h->pacc, (size_t)(F / 64) * 1024));
      if (st == PROX_OK) A(cudaMemset(h->pacc, 0, (size_t)(F / 64) * 1024 * sizeof(float)));
      A(dev_alloc(&h->xh, (size_t)kBT * D));
      A(dev_alloc(&h->cmask, (size_t)(F + 3) / 4)); A(dev_alloc(&h->umask, (size_t)F));
      if (st == PROX_OK) A(cudaMemset(h->cmask, 0, (size_t)((F + 3) / 4) * sizeof(unsigned)));
      A(dev_alloc(&h->tokfac, (size_t)kBT));
      A(dev_alloc(&h->xd, (size_t)D * kBT)); A(dev_alloc(&h->soffb, (size_t)(D / 128) * kBT));
    }
    if (st == PROX_OK) A(cudaMemset(h->gacc, 0, (size_t)((F + 15) / 16) * 256 * sizeof(float)));
  }
  A(cudaDeviceGetAttribute(&h->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, h->device));
  A(cudaDeviceGetAttribute(&h->coop, cudaDevAttrCooperativeLaunch, h->device));
  h->spin_limit = kSpinLimit;
  if (st == PROX_OK) {
    A(cudaHostAlloc(reinterpret_cast<void**>(&h->host_flag), sizeof(int), cudaHostAllocMapped));
    if (st == PROX_OK) { *h->host_flag = 0; A(cudaHostGetDevicePointer(reinterpret_cast<void**>(&h->host_flag_dev), h->host_flag, 0)); }
  }
  h->use_fused = 1;
  h->use_union = 1;
  h->use_mma = 1;
  if (st == PROX_OK) A(cudaMemset(h->syncbuf, 0, (4096 + 64) * sizeof(unsigned)));
  A(dev_alloc(reinterpret_cast<uint16_t**>(&h->x_stage), (size_t)MB * D));
  A(dev_alloc(reinterpret_cast<float**>(&h->y_stage), (size_t)MB * D));
  if (st == PROX_OK) {
    A(cudaMemset(h->ticket, 0, (size_t)MB * ns_max * sizeof(unsigned)));
    A(cudaMemset(h->yacc, 0, (size_t)MB * D * sizeof(float)));
    A(cudaMemset(h->dev_status, 0, sizeof(int)));
    A(cudaMemset(h->counters, 0, 4 * sizeof(unsigned long long)));
  }
  if (st != PROX_OK) { prox_ffn_destroy(h); return st; }
  *out = h;
  return PROX_OK;
}

void prox_ffn_destroy(prox_ffn_t* h) {
  if (!h) return;
  free_packed(h);
  cudaFree(h->idx_x); cudaFree(h->cnt_x); cudaFree(h->part); cudaFree(h->ticket);
  cudaFree(h->scores); cudaFree(h->svals); cudaFree(h->xn); cudaFree(h->sel); cudaFree(h->cnt_s); cudaFree(h->hbuf);
  cudaFree(h->yacc); cudaFree(h->dev_status); cudaFree(h->counters); cudaFree(h->syncbuf); cudaFree(h->trace);
  cudaFree(h->u_in); cudaFree(h->u_ch); cudaFree(h->u_cnt); cudaFree(h->xu); cudaFree(h->member); cudaFree(h->hb); cudaFree(h->gacc); cudaFree(h->pacc); cudaFree(h->xh); cudaFree(h->tokfac); cudaFree(h->xd); cudaFree(h->soffb); cudaFree(h->cmask); cudaFree(h->umask);
  cudaFree(h->x_stage); cudaFree(h->y_stage);
  if (h->host_flag) cudaFreeHost(h->host_flag);
  if (h->prof) {
    for (auto& r : *h->prof) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    delete h->prof;
  }
  delete h;
}

prox_status_t prox_quantize_proxy(prox_ffn_t* h, int bits, int group_size, void* stream) {
  if (!h) return PROX_ERR_INVALID_ARG;
  if (bits != 4 && bits != 8 && bits != 16) return PROX_ERR_UNSUPPORTED;
  if (group_size != 0 && group_size != 128) return PROX_ERR_UNSUPPORTED;
  if (bits == 16 && group_size != 0) return PROX_ERR_UNSUPPORTED;   // 16-bit proxies are the weights: no scales
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int D = h->cfg.d_model, F = h->cfg.d_ff;
  const int G = group_size == 0 ? D : group_size;
  prox_status_t s = alloc_packed(h, bits, G);
  if (s != PROX_OK) { free_packed(h); return s; }
  const int ngroups = D / G;
  if (bits == 16) {
    const long long total = (long long)(F / 4) * 4 * D;
    const int bs = 256;
    CK(cudaMemsetAsync(h->S, 0, h->s_count * sizeof(__half), st));
    CK(cudaMemsetAsync(h->s_plain, 0, (size_t)2 * F * ngroups * sizeof(float), st));
    proxy_pack16_kernel<<<(unsigned)((total + bs - 1) / bs), bs, 0, st>>>(h->wg, h->wu, D, F,
                                                                         reinterpret_cast<uint32_t*>(h->P));
    h->launches++;
    CK(cudaGetLastError());
  } else {
  {
    const long long warps = 2ll * F * ngroups;
    const long long threads = warps * 32;
    const int bs = 256;
    proxy_scale_kernel<<<(unsigned)((threads + bs - 1) / bs), bs, 0, st>>>(
        reinterpret_cast<const __nv_bfloat16*>(h->wg), reinterpret_cast<const __nv_bfloat16*>(h->wu), D,
        F, G, bits, h->S, h->s_plain);
    h->launches++;
    CK(cudaGetLastError());
  }
  {
    const long long total = (long long)(F / ch_per_chunk(bits)) * 4 * D;
    const int bs = 256;
    proxy_pack_kernel<<<(unsigned)((total + bs - 1) / bs), bs, 0, st>>>(
        reinterpret_cast<const __nv_bfloat16*>(h->wg), reinterpret_cast<const __nv_bfloat16*>(h->wu), D,
        F, G, bits, h->s_plain, reinterpret_cast<uint32_t*>(h->P));
    h->launches++;
    CK(cudaGetLastError());
  }
  }
  {
    dim3 grid((F + 31) / 32, (D + 31) / 32), block(32, 8);
    transpose_bf16_kernel<<<grid, block, 0, st>>>(h->wd, h->wdt, D, F);
    h->launches++;
    CK(cudaGetLastError());
  }
  h->quantized = true;
  return PROX_OK;
}

prox_status_t prox_input_topk(prox_ffn_t* h, const void* x, int B, int k1, int32_t* idx, void* stream) {
  prox_status_t s = check_common(h, x, B);
  if (s != PROX_OK) return s;
  if (!idx || k1 < 1 || k1 > h->cfg.d_model) return PROX_ERR_INVALID_ARG;
  return launch_input_select(h, x, B, k1, 0.f, 0, idx, k1, nullptr, static_cast<cudaStream_t>(stream));
}

prox_status_t prox_stage1_mask(prox_ffn_t* h, const void* x, int B, int k1, int k2, int32_t* sel,
                               float* scores, void* stream) {
  prox_status_t s = check_common(h, x, B);
  if (s != PROX_OK) return s;
  if (!sel) return PROX_ERR_INVALID_ARG;
  if (k1 < 1 || k1 > h->cfg.d_model || k2 < 1 || k2 > h->cfg.d_ff) return PROX_ERR_INVALID_ARG;
  if (!h->quantized) return PROX_ERR_NOT_QUANTIZED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int D = h->cfg.d_model;
  float* sc = scores ? scores : h->scores;
  if (B > 1 && h->mask_policy == 1 && !(h->use_union && batch_path_ok(h, B, true))) return PROX_ERR_UNSUPPORTED;
  if (h->use_union && batch_path_ok(h, B, true)) return launch_stage1_batch(h, x, B, k1, k2, sel, k2, sc, st, false, scores != nullptr);
  if ((s = launch_input_select(h, x, B, k1, 0.f, 0, h->idx_x, D, nullptr, st)) != PROX_OK) return s;
  if ((s = launch_proxy(h, x, B, h->idx_x, D, nullptr, k1, sc, st)) != PROX_OK) return s;
  return launch_channel_select(h, sc, B, k2, 0.f, 0, sel, k2, nullptr, st);
}

prox_status_t prox_stage2_ffn(prox_ffn_t* h, const void* x, int B, const int32_t* sel, int k2, void* y,
                              void* stream) {
  prox_status_t s = check_common(h, x, B);
  if (s != PROX_OK) return s;
  if (!sel || !y || !aligned16(y)) return PROX_ERR_INVALID_ARG;
  if (k2 < 1 || k2 > h->cfg.d_ff) return PROX_ERR_INVALID_ARG;
  if (!h->quantized) return PROX_ERR_NOT_QUANTIZED;
  if (h->use_union && batch_path_ok(h, B))
    return launch_stage2_batch(h, x, B, sel, k2, k2, y, static_cast<cudaStream_t>(stream));
  return launch_stage2(h, x, B, sel, k2, nullptr, k2, y, static_cast<cudaStream_t>(stream));
}

prox_status_t prox_ffn_forward(prox_ffn_t* h, const void* x, int B, int k1, int k2, void* y, void* stream) {
  prox_status_t s = check_common(h, x, B);
  if (s != PROX_OK) return s;
  if (!y || !aligned16(y)) return PROX_ERR_INVALID_ARG;
  if (k1 < 1 || k1 > h->cfg.d_model || k2 < 1 || k2 > h->cfg.d_ff) return PROX_ERR_INVALID_ARG;
  if (!h->quantized) return PROX_ERR_NOT_QUANTIZED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int D = h->cfg.d_model, F = h->cfg.d_ff;
  if (B == 1) {
    const FusedPlan pl = plan_fused(h, k1, k2);
    if (pl.ok) { h->sel_unordered = 1; return launch_fused(h, pl, x, k1, k2, y, h->sel, st); }
  }
  return forward_kernels(h, x, B, k1, k2, y, st);
}

/* One layer's FFN sub-block on the residual stream. */
prox_status_t prox_ffn_block_forward(prox_ffn_t* h, const float* x_res, const void* norm_w, double eps, int B,
                                     int k1, int k2, float* x_res_out, void* stream) {
  prox_status_t s = check_common(h, x_res, B);
  if (s != PROX_OK) return s;
  if (!norm_w || !x_res_out || !aligned16(x_res_out) || !aligned16(norm_w)) return PROX_ERR_INVALID_ARG;
  if (!(eps >= 0.0)) return PROX_ERR_INVALID_ARG;
  if (k1 < 1 || k1 > h->cfg.d_model || k2 < 1 || k2 > h->cfg.d_ff) return PROX_ERR_INVALID_ARG;
  if (!h->quantized) return PROX_ERR_NOT_QUANTIZED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int D = h->cfg.d_model;
  if (B == 1) {
    const FusedPlan pl = plan_fused(h, k1, k2);
    if (pl.ok) {
      h->sel_unordered = 1;
      return launch_fused(h, pl, nullptr, k1, k2, nullptr, h->sel, st, x_res,
                          static_cast<const uint16_t*>(norm_w), eps, x_res_out);
    }
  }
  rmsnorm_kernel<<<B, 256, 0, st>>>(x_res, static_cast<const uint16_t*>(norm_w), rms_const(D, eps), D, h->xn);
  h->launches++;
  CK(cudaGetLastError());
  h->fin_resid = x_res; h->fin_out = x_res_out;          // the last kernel adds the residual stream
  s = forward_kernels(h, h->xn, B, k1, k2, nullptr, st);
  h->fin_resid = nullptr; h->fin_out = nullptr;
  return s;
}

/* The layer sub-block with the threshold form of the masks. */
prox_status_t prox_ffn_block_forward_threshold(prox_ffn_t* h, const float* x_res, const void* norm_w, double eps,
                                               int B, float tau_x, float tau_s, float* x_res_out, void* stream) {
  prox_status_t s = check_common(h, x_res, B);
  if (s != PROX_OK) return s;
  if (!norm_w || !x_res_out || !aligned16(x_res_out) || !aligned16(norm_w)) return PROX_ERR_INVALID_ARG;
  if (!(eps >= 0.0) || !(tau_x >= 0.f) || !(tau_s >= 0.f) || !(tau_x < INFINITY) || !(tau_s < INFINITY))
    return PROX_ERR_INVALID_ARG;
  if (!h->quantized) return PROX_ERR_NOT_QUANTIZED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int D = h->cfg.d_model, F = h->cfg.d_ff;
  if (B == 1) {
    const FusedPlan pl = plan_fused(h, D, F, true);
    if (pl.ok) {
      const float taus[2] = {tau_x, tau_s};
      h->sel_unordered = 0;
      return launch_fused(h, pl, nullptr, D, F, nullptr, h->sel, st, x_res, static_cast<const uint16_t*>(norm_w),
                          eps, x_res_out, taus);
    }
  }
  rmsnorm_kernel<<<B, 256, 0, st>>>(x_res, static_cast<const uint16_t*>(norm_w), rms_const(D, eps), D, h->xn);
  h->launches++;
  CK(cudaGetLastError());
  if ((s = prox_stage1_mask_threshold(h, h->xn, B, tau_x, tau_s, h->sel, h->cnt_s, nullptr, stream)) != PROX_OK) return s;
  h->fin_resid = x_res; h->fin_out = x_res_out;          // the last kernel adds the residual stream
  s = launch_stage2(h, h->xn, B, h->sel, F, h->cnt_s, F, nullptr, st);
  h->fin_resid = nullptr; h->fin_out = nullptr;
  return s;
}

/* Stacks of layers: top-k form (tau arrays NULL) or threshold form (one pair of thresholds per layer). */
static prox_status_t stack_forward(prox_ffn_t* const* layers, int n_layers, const void* norm_w, double eps,
                                   float* x_res, int B, int k1, int k2, const float* tau_x, const float* tau_s,
                                   float* trace, void* stream) {
  if (!layers || n_layers < 1 || !norm_w || !x_res) return PROX_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l) {
    if (!layers[l]) return PROX_ERR_INVALID_ARG;
    if (layers[l]->cfg.d_model != layers[0]->cfg.d_model) return PROX_ERR_INVALID_ARG;
  }
  if (B < 1 || B > layers[0]->cfg.max_batch) return PROX_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t D = (size_t)layers[0]->cfg.d_model;
  const size_t bytes = (size_t)B * D * sizeof(float);
  if (trace) CK(cudaMemcpyAsync(trace, x_res, bytes, cudaMemcpyDeviceToDevice, st));
  for (int l = 0; l < n_layers; ++l) {
    const uint16_t* nw = static_cast<const uint16_t*>(norm_w) + (size_t)l * D;
    const prox_status_t s = tau_x
        ? prox_ffn_block_forward_threshold(layers[l], x_res, nw, eps, B, tau_x[l], tau_s[l], x_res, stream)
        : prox_ffn_block_forward(layers[l], x_res, nw, eps, B, k1, k2, x_res, stream);
    if (s != PROX_OK) return s;
    if (trace) CK(cudaMemcpyAsync(trace + (size_t)(l + 1) * B * D, x_res, bytes, cudaMemcpyDeviceToDevice, st));
  }
  return PROX_OK;
}

prox_status_t prox_ffn_stack_forward_threshold(prox_ffn_t* const* layers, int n_layers, const void* norm_w,
                                               double eps, float* x_res, int B, const float* tau_x_host,
                                               const float* tau_s_host, float* trace, void* stream) {
  if (!tau_x_host || !tau_s_host) return PROX_ERR_INVALID_ARG;
  return stack_forward(layers, n_layers, norm_w, eps, x_res, B, 0, 0, tau_x_host, tau_s_host, trace, stream);
}

/* The FFN sub-blocks of consecutive layers applied to one residual stream. */
prox_status_t prox_ffn_stack_forward(prox_ffn_t* const* layers, int n_layers, const void* norm_w, double eps,
                                     float* x_res, int B, int k1, int k2, float* trace, void* stream) {
  return stack_forward(layers, n_layers, norm_w, eps, x_res, B, k1, k2, nullptr, nullptr, trace, stream);
}

// Ablation A3 of Sec. "Ablation Studies": Stage 1 as always, then the selected proxy values themselves
// enter the down projection (no exact gate/up).  With 16-bit proxies this is the input-sparse /
// state-sparse pattern of Sec. 2.2.
prox_status_t prox_ffn_forward_proxy_values(prox_ffn_t* h, const void* x, int B, int k1, int k2, void* y,
                                            void* stream) {
  prox_status_t s = check_common(h, x, B);
  if (s != PROX_OK) return s;
  if (!y || !aligned16(y)) return PROX_ERR_INVALID_ARG;
  if (k1 < 1 || k1 > h->cfg.d_model || k2 < 1 || k2 > h->cfg.d_ff) return PROX_ERR_INVALID_ARG;
  if (!h->quantized) return PROX_ERR_NOT_QUANTIZED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int D = h->cfg.d_model, F = h->cfg.d_ff;
  h->sel_unordered = 0;
  if ((s = launch_input_select(h, x, B, k1, 0.f, 0, h->idx_x, D, nullptr, st)) != PROX_OK) return s;
  if ((s = launch_proxy(h, x, B, h->idx_x, D, nullptr, k1, h->scores, st, h->svals)) != PROX_OK) return s;
  if ((s = launch_channel_select(h, h->scores, B, k2, 0.f, 0, h->sel, F, nullptr, st)) != PROX_OK) return s;
  {
    LaunchScope ls(h, kKGateUp, st);
    dim3 g((k2 + 255) / 256, B);
    gather_values_kernel<<<g, 256, 0, st>>>(h->svals, h->sel, F, k2, F, h->hbuf, F, h->dev_status);
  }
  CK(cudaGetLastError());
  return launch_down(h, B, h->sel, F, nullptr, k2, y, st);
}

prox_status_t prox_fused_kernel_info(prox_ffn_t* h, int k1, int k2, int32_t* info) {
  if (!h || !info) return PROX_ERR_INVALID_ARG;
  if (!h->quantized) return PROX_ERR_NOT_QUANTIZED;
  for (int i = 0; i < 8; ++i) info[i] = 0;
  const FusedPlan pl = plan_fused(h, k1, k2);
  info[0] = pl.ok ? 1 : 0;
  if (!pl.ok) return PROX_OK;
  const void* fn = h->bits == 4
      ? (pl.xch == 1 ? (const void*)prox_fused_kernel<4, 1> : pl.xch == 2 ? (const void*)prox_fused_kernel<4, 2> : (const void*)prox_fused_kernel<4, 4>)
      : (pl.xch == 1 ? (const void*)prox_fused_kernel<8, 1> : pl.xch == 2 ? (const void*)prox_fused_kernel<8, 2> : (const void*)prox_fused_kernel<8, 4>);
  cudaFuncAttributes fa;
  CK(cudaFuncGetAttributes(&fa, fn));
  CK(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.optin));
  int nb = 0;
  CK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, fn, kFusedThreads, pl.smem));
  info[1] = pl.grid; info[2] = pl.pstages; info[3] = (int)pl.smem; info[4] = pl.nslots;
  info[5] = fa.numRegs; info[6] = (int)fa.sharedSizeBytes; info[7] = nb;
  return PROX_OK;
}

prox_status_t prox_fused_trace(prox_ffn_t* h, int on, uint64_t* stamps_host, int max_blocks) {
  if (!h) return PROX_ERR_INVALID_ARG;
  const int G = h->sm_count;
  if (on && !h->trace) {
    CK(dev_alloc(&h->trace, (size_t)G * 32));
    CK(cudaMemset(h->trace, 0, (size_t)G * 32 * sizeof(unsigned long long)));
  }
  if (stamps_host && h->trace) {
    CK(cudaDeviceSynchronize());
    const int n = max_blocks < G ? max_blocks : G;
    CK(cudaMemcpy(stamps_host, h->trace, (size_t)n * 32 * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
  }
  if (!on && h->trace) { cudaFree(h->trace); h->trace = nullptr; }
  return PROX_OK;
}

// ---- offline threshold calibration (host side) ---------------------------------
struct prox_calib {
  int64_t cap, seen;
  uint64_t seed;
  std::vector<float> res;
  std::vector<char> stage;
};

static inline uint64_t splitmix64_at(uint64_t seed, uint64_t i) {
  uint64_t z = seed + (i + 1) * 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

prox_status_t prox_calib_create(int64_t capacity, uint64_t seed, prox_calib_t** out) {
  if (!out || capacity < 1 || capacity > (int64_t)1 << 28) return PROX_ERR_INVALID_ARG;
  prox_calib* c = new (std::nothrow) prox_calib();
  if (!c) return PROX_ERR_OOM;
  c->cap = capacity; c->seen = 0; c->seed = seed;
  *out = c;
  return PROX_OK;
}

void prox_calib_destroy(prox_calib_t* c) { delete c; }

prox_status_t prox_calib_add(prox_calib_t* c, const void* values_dev, int64_t n, int dtype, void* stream) {
  if (!c || n < 0 || (n > 0 && !values_dev) || (dtype != 0 && dtype != 1)) return PROX_ERR_INVALID_ARG;
  if (n == 0) return PROX_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t esz = dtype == 0 ? 2 : 4;
  try { c->stage.resize((size_t)n * esz); } catch (...) { return PROX_ERR_OOM; }
  CK(cudaMemcpyAsync(c->stage.data(), values_dev, (size_t)n * esz, cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  try {
    for (int64_t k = 0; k < n; ++k) {
      float v;
      if (dtype == 0) {
        const uint32_t bits = (uint32_t)reinterpret_cast<const uint16_t*>(c->stage.data())[k] << 16;
        std::memcpy(&v, &bits, 4);
      } else {
        v = reinterpret_cast<const float*>(c->stage.data())[k];
      }
      v = std::fabs(v);
      if (c->seen < c->cap) {
        c->res.push_back(v);
      } else {
        const uint64_t j = splitmix64_at(c->seed, (uint64_t)c->seen) % ((uint64_t)c->seen + 1);
        if (j < (uint64_t)c->cap) c->res[(size_t)j] = v;
      }
      c->seen++;
    }
  } catch (...) { return PROX_ERR_OOM; }
  return PROX_OK;
}

prox_status_t prox_calib_threshold(const prox_calib_t* c, double s, float* tau) {
  if (!c || !tau || !(s >= 0.0 && s <= 1.0)) return PROX_ERR_INVALID_ARG;
  if (c->res.empty()) return PROX_ERR_UNSUPPORTED;
  std::vector<float> a;
  try { a = c->res; } catch (...) { return PROX_ERR_OOM; }
  std::sort(a.begin(), a.end());
  const size_t n = a.size();
  const double pos = s * (double)(n - 1);
  const size_t lo = (size_t)std::floor(pos), hi = lo + 1 < n ? lo + 1 : n - 1;
  *tau = (float)((double)a[lo] + (pos - (double)lo) * ((double)a[hi] - (double)a[lo]));
  return PROX_OK;
}

prox_status_t prox_calib_histogram(const prox_calib_t* c, int64_t* counts_host, float* upper) {
  if (!c || !counts_host || !upper) return PROX_ERR_INVALID_ARG;
  if (c->res.empty()) return PROX_ERR_UNSUPPORTED;
  float hi = 0.f;
  for (float v : c->res) hi = v > hi ? v : hi;
  for (int b = 0; b < 4096; ++b) counts_host[b] = 0;
  for (float v : c->res) {
    int b = 4095;
    if (hi > 0.f) {
      const double q = std::floor((double)v / (double)hi * 4096.0);
      b = q < 4095.0 ? (int)q : 4095;
    }
    counts_host[b]++;
  }
  *upper = hi;
  return PROX_OK;
}

prox_status_t prox_calib_seen(const prox_calib_t* c, int64_t* seen, int64_t* held) {
  if (!c) return PROX_ERR_INVALID_ARG;
  if (seen) *seen = c->seen;
  if (held) *held = (int64_t)c->res.size();
  return PROX_OK;
}

prox_status_t prox_rmsnorm(prox_ffn_t* h, const float* x_res, const void* norm_w, double eps, int B, void* xn_out,
                           void* stream) {
  prox_status_t s = check_common(h, x_res, B);
  if (s != PROX_OK) return s;
  if (!norm_w || !xn_out || !aligned16(xn_out) || !aligned16(norm_w) || !(eps >= 0.0)) return PROX_ERR_INVALID_ARG;
  const int D = h->cfg.d_model;
  rmsnorm_kernel<<<B, 256, 0, static_cast<cudaStream_t>(stream)>>>(x_res, static_cast<const uint16_t*>(norm_w), rms_const(D, eps), D,
                                                                   static_cast<uint16_t*>(xn_out));
  h->launches++;
  CK(cudaGetLastError());
  return PROX_OK;
}

prox_status_t prox_ffn_set_fused(prox_ffn_t* h, int on) {
  if (!h) return PROX_ERR_INVALID_ARG;
  h->use_fused = on != 0;
  return PROX_OK;
}

prox_status_t prox_ffn_set_mask_policy(prox_ffn_t* h, int policy) {
  if (!h || (policy != 0 && policy != 1)) return PROX_ERR_INVALID_ARG;
  h->mask_policy = policy;
  return PROX_OK;
}

prox_status_t prox_ffn_set_union(prox_ffn_t* h, int on) {
  if (!h) return PROX_ERR_INVALID_ARG;
  h->use_union = on != 0;
  h->use_mma = on != 1;                 // 1 selects the CUDA-core union kernels, any other non-zero value the tensor-core ones
  return PROX_OK;
}

prox_status_t prox_ffn_last_mask(prox_ffn_t* h, int B, int k2, int32_t* sel_dev, void* stream) {
  if (!h || !sel_dev || B < 1 || B > h->cfg.max_batch || k2 < 1 || k2 > h->cfg.d_ff) return PROX_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (B == 1 && h->sel_unordered) {
    // the persistent kernel lists the kept channels in its own order; the score buffer is free between calls
    LaunchScope ls(h, kKChannel, st);
    mask_ascending_kernel<<<1, 1024, 0, st>>>(h->sel, k2, h->cfg.d_ff, reinterpret_cast<int*>(h->hbuf), sel_dev);
    CK(cudaGetLastError());
    return PROX_OK;
  }
  CK(cudaMemcpy2DAsync(sel_dev, (size_t)k2 * sizeof(int), h->sel, (size_t)h->cfg.d_ff * sizeof(int),
                       (size_t)k2 * sizeof(int), (size_t)B, cudaMemcpyDeviceToDevice, st));
  return PROX_OK;
}

prox_status_t prox_ffn_forward_host(prox_ffn_t* h, const void* x_host, int B, int k1, int k2,
                                    void* y_host, void* stream) {
  if (!h || !x_host || !y_host) return PROX_ERR_INVALID_ARG;
  if (B < 1 || B > h->cfg.max_batch) return PROX_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t D = h->cfg.d_model;
  const size_t ybytes = (size_t)B * D * (h->cfg.out_dtype ? 4 : 2);
  CK(cudaMemcpyAsync(h->x_stage, x_host, (size_t)B * D * 2, cudaMemcpyHostToDevice, st));
  // If y_host is pinned and mapped, the kernels write the result straight into it (one small
  // write over the bus by the block that rounds y) and the copy back is not needed.
  void* y_direct = nullptr;
  {
    cudaPointerAttributes pa;
    if (cudaPointerGetAttributes(&pa, y_host) == cudaSuccess && pa.type == cudaMemoryTypeHost && pa.devicePointer &&
        aligned16(pa.devicePointer))
      y_direct = pa.devicePointer;
    else
      (void)cudaGetLastError();
  }
  prox_status_t s = prox_ffn_forward(h, h->x_stage, B, k1, k2, y_direct ? y_direct : h->y_stage, stream);
  if (s != PROX_OK) return s;
  if (!y_direct) CK(cudaMemcpyAsync(y_host, h->y_stage, ybytes, cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  if (h->host_flag && *reinterpret_cast<volatile int*>(h->host_flag)) {
    // a bounded device-side wait ran out: y_host is undefined; put the shared counters back and say so
    CK(cudaMemsetAsync(h->dev_status, 0, sizeof(int), st));
    s = reset_shared_state(h, st);
    return s != PROX_OK ? s : PROX_ERR_TIMEOUT;
  }
  return PROX_OK;
}

// ---- threshold variant ------------------------------------------------------
namespace {
__global__ void count_accum_kernel(const int* cnt_x, const int* cnt_s, int B, unsigned long long* c) {
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    unsigned long long a = 0, s = 0;
    for (int b = 0; b < B; ++b) { a += (unsigned long long)cnt_x[b]; s += (unsigned long long)cnt_s[b]; }
    c[0] += (unsigned long long)B; c[1] += a; c[2] += s;
  }
}
}  // namespace

prox_status_t prox_stage1_mask_threshold(prox_ffn_t* h, const void* x, int B, float tau_x, float tau_s,
                                         int32_t* sel, int32_t* count, float* scores, void* stream) {
  prox_status_t s = check_common(h, x, B);
  if (s != PROX_OK) return s;
  if (!sel || !count) return PROX_ERR_INVALID_ARG;
  if (!(tau_x >= 0.f) || !(tau_s >= 0.f)) return PROX_ERR_INVALID_ARG;
  if (!h->quantized) return PROX_ERR_NOT_QUANTIZED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int D = h->cfg.d_model, F = h->cfg.d_ff;
  float* sc = scores ? scores : h->scores;
  if ((s = launch_input_select(h, x, B, 0, tau_x, 1, h->idx_x, D, h->cnt_x, st)) != PROX_OK) return s;
  if ((s = launch_proxy(h, x, B, h->idx_x, D, h->cnt_x, D, sc, st)) != PROX_OK) return s;
  if ((s = launch_channel_select(h, sc, B, 0, tau_s, 1, sel, F, count, st)) != PROX_OK) return s;
  count_accum_kernel<<<1, 32, 0, st>>>(h->cnt_x, count, B, h->counters);
  h->launches++;
  CK(cudaGetLastError());
  return PROX_OK;
}

prox_status_t prox_stage2_ffn_var(prox_ffn_t* h, const void* x, int B, const int32_t* sel,
                                  const int32_t* count, void* y, void* stream) {
  prox_status_t s = check_common(h, x, B);
  if (s != PROX_OK) return s;
  if (!sel || !count || !y || !aligned16(y)) return PROX_ERR_INVALID_ARG;
  if (!h->quantized) return PROX_ERR_NOT_QUANTIZED;
  return launch_stage2(h, x, B, sel, h->cfg.d_ff, count, h->cfg.d_ff, y, static_cast<cudaStream_t>(stream));
}

prox_status_t prox_ffn_forward_threshold(prox_ffn_t* h, const void* x, int B, float tau_x, float tau_s,
                                         void* y, void* stream) {
  if (!h) return PROX_ERR_INVALID_ARG;
  if (B == 1 && h->quantized && x && y && aligned16(x) && aligned16(y) && tau_x >= 0.f && tau_s >= 0.f &&
      tau_x < INFINITY && tau_s < INFINITY) {
    // one launch of the persistent kernel in its threshold form
    const FusedPlan pl = plan_fused(h, h->cfg.d_model, h->cfg.d_ff, true);
    if (pl.ok) {
      const float taus[2] = {tau_x, tau_s};
      h->sel_unordered = 0;
      return launch_fused(h, pl, x, h->cfg.d_model, h->cfg.d_ff, y, h->sel, static_cast<cudaStream_t>(stream),
                          nullptr, nullptr, 0.0, nullptr, taus);
    }
  }
  prox_status_t s = prox_stage1_mask_threshold(h, x, B, tau_x, tau_s, h->sel, h->cnt_s, nullptr, stream);
  if (s != PROX_OK) return s;
  return prox_stage2_ffn_var(h, x, B, h->sel, h->cnt_s, y, stream);
}

prox_status_t prox_runtime_sparsity(prox_ffn_t* h, double alpha, int64_t* tokens, double* s1_hat,
                                    double* s2_hat, double* e_hat, int reset) {
  if (!h) return PROX_ERR_INVALID_ARG;
  unsigned long long c[4] = {0, 0, 0, 0};
  CK(cudaDeviceSynchronize());
  CK(cudaMemcpy(c, h->counters, sizeof(c), cudaMemcpyDeviceToHost));
  if (reset) CK(cudaMemset(h->counters, 0, sizeof(c)));
  const double n = (double)c[0];
  const double s1 = n > 0 ? 1.0 - (double)c[1] / (n * h->cfg.d_model) : 0.0;
  const double s2 = n > 0 ? 1.0 - (double)c[2] / (n * h->cfg.d_ff) : 0.0;
  if (tokens) *tokens = (int64_t)c[0];
  if (s1_hat) *s1_hat = s1;
  if (s2_hat) *s2_hat = s2;
  if (e_hat) *e_hat = s2 - 2.0 * alpha * (1.0 - s1) / 3.0;
  return PROX_OK;
}

// ---- host helpers -----------------------------------------------------------
prox_status_t prox_allocate_budget(double e, double alpha, double s_ref, double s1_min, double s1_max,
                                   double* s1, double* s2) {
  if (!s1 || !s2) return PROX_ERR_INVALID_ARG;
  if (!(alpha > 0.0) || !(s1_min <= s1_max) || !std::isfinite(e) || !std::isfinite(s_ref))
    return PROX_ERR_INVALID_ARG;
  double b = s_ref;
  double a = 1.0 - (b - e) * 3.0 / (2.0 * alpha);
  if (a < s1_min || a > s1_max) {
    a = a < s1_min ? s1_min : s1_max;
    b = e + 2.0 * alpha * (1.0 - a) / 3.0;
  }
  *s1 = a;
  *s2 = b;
  return PROX_OK;
}

prox_status_t prox_sparsity_to_k(double s, int dim, int* k) {
  if (!k || dim < 1 || !std::isfinite(s)) return PROX_ERR_INVALID_ARG;
  double v = std::floor((1.0 - s) * (double)dim + 0.5);
  if (v < 1.0) v = 1.0;
  if (v > (double)dim) v = (double)dim;
  *k = (int)v;
  return PROX_OK;
}

prox_status_t prox_algorithmic_bytes(const prox_ffn_t* h, int rows_in, int rows_ch, int64_t* stage1,
                                     int64_t* gate_up, int64_t* down, int64_t* activations) {
  if (!h || rows_in < 0 || rows_ch < 0) return PROX_ERR_INVALID_ARG;
  if (!h->quantized) return PROX_ERR_NOT_QUANTIZED;
  const int64_t D = h->cfg.d_model, F = h->cfg.d_ff;
  const int64_t ngroups = D / h->group;
  if (stage1) *stage1 = (int64_t)rows_in * F * h->bits / 4 + (h->bits == 16 ? 0 : 2 * ngroups * F * 2);
  if (gate_up) *gate_up = 2 * (int64_t)rows_ch * D * 2;
  if (down) *down = (int64_t)rows_ch * D * 2;
  if (activations) *activations = 4 * D + 8 * F + 16 * (int64_t)rows_ch + (h->cfg.out_dtype ? 4 : 2) * D;
  return PROX_OK;
}

// ---- export / save / load ---------------------------------------------------
prox_status_t prox_proxy_export(prox_ffn_t* h, int which, int8_t* q_host, float* scale_host) {
  if (!h || !q_host || !scale_host || (which != 0 && which != 1)) return PROX_ERR_INVALID_ARG;
  if (!h->quantized) return PROX_ERR_NOT_QUANTIZED;
  if (h->bits == 16) return PROX_ERR_UNSUPPORTED;        // no integer codes to export
  CK(cudaDeviceSynchronize());
  const int D = h->cfg.d_model, F = h->cfg.d_ff, bits = h->bits;
  const int CH = ch_per_chunk(bits), nchunks = F / CH, ngroups = D / h->group;
  std::vector<uint32_t> P;
  try { P.resize(h->p_bytes / 4); } catch (...) { return PROX_ERR_OOM; }
  CK(cudaMemcpy(P.data(), h->P, h->p_bytes, cudaMemcpyDeviceToHost));
  const int per_word = bits == 4 ? 8 : 4;
  const uint32_t mask = bits == 4 ? 0xFu : 0xFFu;
  const int off = bits == 4 ? 8 : 128;
  for (int i = 0; i < D; ++i) {
    const uint32_t* row = P.data() + (size_t)i * nchunks * 4;
    for (int c = 0; c < nchunks; ++c)
      for (int half = 0; half < 2; ++half) {
        const uint32_t w = row[c * 4 + which * 2 + half];
        for (int m = 0; m < per_word; ++m) {
          const int j = c * CH + half * per_word + m;
          q_host[(size_t)j * D + i] = (int8_t)((int)((w >> (m * bits)) & mask) - off);
        }
      }
  }
  CK(cudaMemcpy(scale_host, h->s_plain + (size_t)which * F * ngroups, (size_t)F * ngroups * sizeof(float),
                cudaMemcpyDeviceToHost));
  return PROX_OK;
}

namespace {
struct PackHeader {
  char magic[8];
  int32_t version, d_model, d_ff, bits, group;
  uint64_t p_bytes, s_count, wdt_count;
};
const char kMagic[8] = {'P', 'R', 'O', 'X', 'P', 'A', 'C', 'K'};
}  // namespace

prox_status_t prox_pack_save(prox_ffn_t* h, const char* path) {
  if (!h || !path) return PROX_ERR_INVALID_ARG;
  if (!h->quantized) return PROX_ERR_NOT_QUANTIZED;
  CK(cudaDeviceSynchronize());
  const int D = h->cfg.d_model, F = h->cfg.d_ff, ngroups = D / h->group;
  PackHeader hd;
  std::memset(&hd, 0, sizeof(hd));
  std::memcpy(hd.magic, kMagic, 8);
  hd.version = 1; hd.d_model = D; hd.d_ff = F; hd.bits = h->bits; hd.group = h->group;
  hd.p_bytes = h->p_bytes; hd.s_count = h->s_count; hd.wdt_count = (uint64_t)F * D;
  std::vector<char> buf;
  const size_t sp_bytes = (size_t)2 * F * ngroups * sizeof(float);
  const size_t biggest = h->p_bytes > hd.wdt_count * 2 ? h->p_bytes : hd.wdt_count * 2;
  try { buf.resize(biggest > sp_bytes ? biggest : sp_bytes); } catch (...) { return PROX_ERR_OOM; }
  FILE* f = std::fopen(path, "wb");
  if (!f) return PROX_ERR_IO;
  bool ok = std::fwrite(&hd, sizeof(hd), 1, f) == 1;
  auto dump = [&](const void* dev, size_t bytes) {
    if (!ok) return;
    if (cudaMemcpy(buf.data(), dev, bytes, cudaMemcpyDeviceToHost) != cudaSuccess) { ok = false; return; }
    ok = std::fwrite(buf.data(), 1, bytes, f) == bytes;
  };
  dump(h->P, h->p_bytes);
  dump(h->S, h->s_count * sizeof(__half));
  dump(h->s_plain, sp_bytes);
  dump(h->wdt, hd.wdt_count * 2);
  ok = (std::fclose(f) == 0) && ok;
  return ok ? PROX_OK : PROX_ERR_IO;
}

prox_status_t prox_pack_load(prox_ffn_t* h, const char* path, void* stream) {
  if (!h || !path) return PROX_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  FILE* f = std::fopen(path, "rb");
  if (!f) return PROX_ERR_IO;
  PackHeader hd;
  if (std::fread(&hd, sizeof(hd), 1, f) != 1 || std::memcmp(hd.magic, kMagic, 8) != 0 || hd.version != 1) {
    std::fclose(f);
    return PROX_ERR_IO;
  }
  const int D = h->cfg.d_model, F = h->cfg.d_ff;
  const bool shape_ok = hd.d_model == D && hd.d_ff == F && (hd.bits == 4 || hd.bits == 8 || hd.bits == 16) &&
                        (hd.group == D || hd.group == 128);
  if (!shape_ok || (hd.bits == 16 && hd.group != D)) { std::fclose(f); return PROX_ERR_INVALID_ARG; }   // 16-bit proxies have no groups
  prox_status_t s = alloc_packed(h, hd.bits, hd.group);
  if (s != PROX_OK) { std::fclose(f); free_packed(h); return s; }
  const int ngroups = D / hd.group;
  const size_t sp_bytes = (size_t)2 * F * ngroups * sizeof(float);
  if (hd.p_bytes != h->p_bytes || hd.s_count != h->s_count || hd.wdt_count != (uint64_t)F * D) {
    std::fclose(f); free_packed(h);
    return PROX_ERR_IO;
  }
  std::vector<char> buf;
  const size_t biggest = h->p_bytes > (size_t)F * D * 2 ? h->p_bytes : (size_t)F * D * 2;
  try { buf.resize(biggest > sp_bytes ? biggest : sp_bytes); } catch (...) { std::fclose(f); free_packed(h); return PROX_ERR_OOM; }
  bool ok = true;
  cudaError_t ce = cudaSuccess;
  auto fill = [&](void* dev, size_t bytes) {
    if (!ok) return;
    if (std::fread(buf.data(), 1, bytes, f) != bytes) { ok = false; return; }
    ce = cudaMemcpyAsync(dev, buf.data(), bytes, cudaMemcpyHostToDevice, st);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
    if (ce != cudaSuccess) ok = false;
  };
  fill(h->P, h->p_bytes);
  fill(h->S, h->s_count * sizeof(__half));
  fill(h->s_plain, sp_bytes);
  fill(h->wdt, (size_t)F * D * 2);
  std::fclose(f);
  if (!ok) { free_packed(h); return ce != cudaSuccess ? map_cuda(ce) : PROX_ERR_IO; }
  h->quantized = true;
  return PROX_OK;
}

prox_status_t prox_last_device_status(prox_ffn_t* h, int32_t* code, void* stream) {
  if (!h || !code) return PROX_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CK(cudaMemcpyAsync(code, h->dev_status, sizeof(int), cudaMemcpyDeviceToHost, st));
  CK(cudaMemsetAsync(h->dev_status, 0, sizeof(int), st));
  CK(cudaStreamSynchronize(st));
  if (*code & kWaitExpired) {
    const prox_status_t s = reset_shared_state(h, st);
    return s != PROX_OK ? s : PROX_ERR_TIMEOUT;
  }
  return PROX_OK;
}

prox_status_t prox_debug_set_wait(prox_ffn_t* h, uint32_t spin_limit, uint32_t barrier_bias) {
  if (!h) return PROX_ERR_INVALID_ARG;
  h->spin_limit = spin_limit ? spin_limit : kSpinLimit;
  h->bar_bias = barrier_bias;
  return PROX_OK;
}

prox_status_t prox_ffn_last_stage1(prox_ffn_t* h, int k1, int32_t* idx_dev, float* scores_dev, void* stream) {
  if (!h || (!idx_dev && !scores_dev)) return PROX_ERR_INVALID_ARG;
  if (idx_dev && (k1 < 1 || k1 > h->cfg.d_model)) return PROX_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (idx_dev) CK(cudaMemcpyAsync(idx_dev, h->idx_x, (size_t)k1 * sizeof(int), cudaMemcpyDeviceToDevice, st));
  if (scores_dev) CK(cudaMemcpyAsync(scores_dev, h->scores, (size_t)h->cfg.d_ff * sizeof(float), cudaMemcpyDeviceToDevice, st));
  return PROX_OK;
}

prox_status_t prox_profile_enable(prox_ffn_t* h, int on) {
  if (!h) return PROX_ERR_INVALID_ARG;
  h->profiling = on != 0;
  return PROX_OK;
}

prox_status_t prox_profile_read(prox_ffn_t* h, int64_t* counts, double* ms) {
  if (!h || !counts || !ms) return PROX_ERR_INVALID_ARG;
  for (int k = 0; k < PROX_NUM_KERNEL_KINDS; ++k) { counts[k] = 0; ms[k] = 0.0; }
  prox_status_t st = PROX_OK;
  for (auto& r : *h->prof) {
    float t = 0.f;
    cudaError_t e = cudaEventSynchronize(r.b);
    if (e == cudaSuccess) e = cudaEventElapsedTime(&t, r.a, r.b);
    if (e == cudaSuccess && r.kind >= 0 && r.kind < PROX_NUM_KERNEL_KINDS) { counts[r.kind]++; ms[r.kind] += t; }
    else if (e != cudaSuccess) st = PROX_ERR_CUDA;
    cudaEventDestroy(r.a); cudaEventDestroy(r.b);
  }
  h->prof->clear();
  return st;
}

prox_status_t prox_launch_count(const prox_ffn_t* h, int64_t* launches) {
  if (!h || !launches) return PROX_ERR_INVALID_ARG;
  *launches = h->launches;
  return PROX_OK;
}

const char* prox_status_string(prox_status_t s) {
  switch (s) {
    case PROX_OK: return "ok";
    case PROX_ERR_INVALID_ARG: return "invalid argument";
    case PROX_ERR_UNSUPPORTED: return "unsupported shape or format";
    case PROX_ERR_NOT_QUANTIZED: return "proxy not quantized yet";
    case PROX_ERR_CUDA: return "CUDA runtime error";
    case PROX_ERR_OOM: return "out of memory";
    case PROX_ERR_TIMEOUT: return "device-side wait timed out";
    case PROX_ERR_IO: return "file I/O error";
  }
  return "unknown status";
}

const char* prox_last_cuda_error(void) {
  return g_last_cuda == cudaSuccess ? "" : cudaGetErrorString(g_last_cuda);
}

const char* prox_version(void) { return "libprox 0.1 (sm_100a)"; }

}  // extern "C"
