// prox_stage2_ffn_noalloc: Stage 2 of the path for callers that must not
// allocate device memory.  See include/prox.h for the contract.
#include "prox.h"

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

// The kernels are the ones the handle-based Stage 2 launches.  They are pulled
// into this translation unit with internal linkage so that the library does not
// end up with two copies of the same external symbol.
namespace {
#include "prox_kernels.cuh"
}  // namespace

namespace {

constexpr int kNoAllocMaxDModel = 16384;   // fp32 accumulator for y: 64 KB
constexpr int kNoAllocMaxK2 = 32768;       // one fp32 h value per kept channel: 128 KB
constexpr int kMaxDevices = 64;

// Scratch that lives in the library image: every GPU that loads libprox holds
// these 192 KB until the process exits.  Layout: [h values | y accumulator |
// one word in which the gate/up kernel notes out-of-range channel ids].
// In host code this name is only a handle for cudaGetSymbolAddress; it is never
// passed to a kernel directly.
static __device__ __align__(256) float g_noalloc_scratch[kNoAllocMaxK2 + kNoAllocMaxDModel + 64];

std::mutex g_setup_mutex;
float* g_scratch_dev[kMaxDevices];          // device address of the array, per device (null = not set up)
int g_sm_count[kMaxDevices];

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" prox_status_t prox_stage2_ffn_noalloc(const void* x_dev, const void* w_gate_dev,
                                                 const void* w_up_dev, const void* w_down_t_dev,
                                                 int d_model, int d_ff, const int32_t* sel_dev, int k2,
                                                 void* y_dev, int out_dtype, void* stream) {
  using namespace prox;
  if (!x_dev || !w_gate_dev || !w_up_dev || !w_down_t_dev || !sel_dev || !y_dev) return PROX_ERR_INVALID_ARG;
  if (!aligned16(x_dev) || !aligned16(w_gate_dev) || !aligned16(w_up_dev) || !aligned16(w_down_t_dev) ||
      !aligned16(y_dev))
    return PROX_ERR_INVALID_ARG;
  if (out_dtype != 0 && out_dtype != 1) return PROX_ERR_INVALID_ARG;
  if (d_model <= 0 || d_ff <= 0 || k2 < 1 || k2 > d_ff) return PROX_ERR_INVALID_ARG;
  if (d_model % 128 || d_ff % 64) return PROX_ERR_UNSUPPORTED;
  // The fixed scratch bounds the problem size; larger problems need the handle-based call.
  if (d_model > kNoAllocMaxDModel || k2 > kNoAllocMaxK2) return PROX_ERR_UNSUPPORTED;

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PROX_ERR_CUDA;
  float* scratch = nullptr;
  int sms = 0;
  {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_dev[dev]) {
      // First call on this device (which is current): resolve the device address of
      // the static array once.  This is set-up work, not something to do under
      // stream capture.
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) {
        (void)cudaGetLastError();
        return PROX_ERR_CUDA;
      }
      int n = 0;
      if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
        (void)cudaGetLastError();
        return PROX_ERR_CUDA;
      }
      g_sm_count[dev] = n;
      g_scratch_dev[dev] = static_cast<float*>(p);
    }
    scratch = g_scratch_dev[dev];
    sms = g_sm_count[dev];
  }
  float* hbuf = scratch;                          // [k2]
  float* yacc = scratch + kNoAllocMaxK2;          // [d_model]
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  // The array keeps whatever the previous call left; the accumulator must start at zero.
  if (cudaMemsetAsync(yacc, 0, (size_t)d_model * sizeof(float), st) != cudaSuccess) {
    (void)cudaGetLastError();
    return PROX_ERR_CUDA;
  }
  // Channel ids outside [0, d_ff) are skipped (they contribute nothing); the note the
  // kernel makes of them goes to a word of the scratch that nobody reads back.
  int* note = reinterpret_cast<int*>(scratch + kNoAllocMaxK2 + kNoAllocMaxDModel);
  const int wpb = kGateUpThreads / 32;
  dim3 g1((k2 + wpb - 1) / wpb, 1);
  gateup_kernel<<<g1, kGateUpThreads, (size_t)d_model * 2, st>>>(
      static_cast<const uint16_t*>(w_gate_dev), static_cast<const uint16_t*>(w_up_dev),
      static_cast<const uint16_t*>(x_dev), sel_dev, k2, nullptr, k2, d_model, d_ff, hbuf, k2, note);
  if (cudaGetLastError() != cudaSuccess) return PROX_ERR_CUDA;
  const int dtiles = (d_model + kDownThreads * 8 - 1) / (kDownThreads * 8);
  int nsplit = (2 * sms + dtiles - 1) / dtiles;
  if (nsplit > k2) nsplit = k2;
  if (nsplit < 1) nsplit = 1;
  dim3 g2(dtiles, nsplit, 1);
  down_kernel<<<g2, kDownThreads, 0, st>>>(static_cast<const uint16_t*>(w_down_t_dev), hbuf, k2, sel_dev, k2,
                                           nullptr, k2, d_model, d_ff, yacc);
  if (cudaGetLastError() != cudaSuccess) return PROX_ERR_CUDA;
  finalize_kernel<<<(d_model + 255) / 256, 256, 0, st>>>(yacc, y_dev, d_model, out_dtype);
  if (cudaGetLastError() != cudaSuccess) return PROX_ERR_CUDA;
  return PROX_OK;
}
