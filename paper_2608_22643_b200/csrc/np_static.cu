// np_predict_logits_noalloc: the predictor forward pass for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc (or anything that may): code running
// inside a memory-pool or arena owner that forbids foreign allocations, a real-time decode
// loop where an allocation's implicit device synchronisation would stall every stream, or a
// process whose device memory is fully budgeted up front.  np_init allocates the library's
// tables, so those callers cannot create a context at all.  This entry point needs none: the
// only scratch the predictor has (the hidden activations between its two layers, and a status
// word for the kernels' bounded waits) lives in a fixed device array that is part of the
// loaded library image.
#include <cstdio>
#include <mutex>

#include "np_internal.h"

namespace {

constexpr int kNoAllocMaxHidden = NP_NOALLOC_MAX_HIDDEN_FLOATS;  // B * H floats
constexpr int kStatusInts = 64;                                   // 256 bytes, keeps `hidden` aligned
constexpr int kMaxDevices = 64;

// Scratch shared by every call on a device; it keeps whatever the last call left in it.
// Layout: [0, kStatusInts) status words, then the hidden activations.
static __device__ __align__(256) float g_noalloc_scratch[kStatusInts + kNoAllocMaxHidden];

std::mutex g_mu;
float* g_scratch_addr[kMaxDevices];  // device address of g_noalloc_scratch, per device
int g_sm_count[kMaxDevices];
thread_local char g_err[256] = "";

int fail(int code, const char* msg) {
  snprintf(g_err, sizeof g_err, "%s", msg);
  return code;
}

}  // namespace

extern "C" {

const char* np_noalloc_last_error(void) { return g_err; }

int np_predict_logits_noalloc(const void* w1, const void* w2, const void* x_bf16, int32_t B, int32_t n_layers,
                              int32_t d_model, int32_t d_ffn, int32_t d_pred, float* logits_out, void* stream) {
  if (!w1 || !w2 || !x_bf16 || !logits_out) return fail(NP_E_INVAL, "a pointer argument is NULL");
  if (((uintptr_t)w1 | (uintptr_t)w2 | (uintptr_t)x_bf16 | (uintptr_t)logits_out) % 16)
    return fail(NP_E_INVAL, "w1, w2, x and logits_out must be 16-byte aligned");
  if (B < 1 || B > npi::kMaxBatch) return fail(NP_E_INVAL, "B must be in [1, 16]");
  if (n_layers < 1 || d_model < 8 || d_model % 8 || d_model > 16384 || d_ffn < 32 || d_ffn % 32 || d_pred < 8 ||
      d_pred % 8 || d_pred > 4096)
    return fail(NP_E_INVAL, "shape outside the library's limits (see np_config)");
  if ((long long)B * d_pred > kNoAllocMaxHidden) {
    snprintf(g_err, sizeof g_err,
             "B * d_pred = %lld exceeds the fixed scratch of %d floats (NP_NOALLOC_MAX_HIDDEN_FLOATS)",
             (long long)B * d_pred, kNoAllocMaxHidden);
    return NP_E_INVAL;
  }
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return fail(NP_E_CUDA, "cudaGetDevice failed");
  if (dev < 0 || dev >= kMaxDevices) return fail(NP_E_INVAL, "device ordinal above 63");
  float* scratch = nullptr;
  int sm_count = 0;
  {
    // first call on this device: resolve the array's device address.  The array's name is
    // only a host-side handle here; a kernel must be given the address the runtime reports
    // for the current device.
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_scratch_addr[dev]) {
      void* p = nullptr;
      cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
      if (e != cudaSuccess) {
        snprintf(g_err, sizeof g_err, "cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
        return NP_E_CUDA;
      }
      int n = 0;
      e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
      if (e != cudaSuccess) {
        snprintf(g_err, sizeof g_err, "cudaDeviceGetAttribute failed: %s", cudaGetErrorString(e));
        return NP_E_CUDA;
      }
      g_sm_count[dev] = n;
      g_scratch_addr[dev] = static_cast<float*>(p);
    }
    scratch = g_scratch_addr[dev];
    sm_count = g_sm_count[dev];
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int32_t* status = reinterpret_cast<int32_t*>(scratch);
  float* hidden = scratch + kStatusInts;
  npi::Dims d = {};
  d.L = n_layers;
  d.D = d_model;
  d.M = d_ffn;
  d.H = d_pred;
  d.W = d_ffn / 32;
  d.Bmax = B;
  // the status words start every call at zero (the array keeps the last call's contents), so
  // that np_noalloc_check reports only what this call's kernels recorded
  cudaError_t e = cudaMemsetAsync(status, 0, kStatusInts * sizeof(int32_t), s);
  if (e == cudaSuccess) e = npi::launch_pred_l1(d, w1, x_bf16, B, hidden, s);
  if (e == cudaSuccess) e = npi::launch_pred_l2(d, w2, hidden, B, logits_out, status, s, sm_count);
  if (e != cudaSuccess) {
    snprintf(g_err, sizeof g_err, "kernel launch failed: %s", cudaGetErrorString(e));
    return NP_E_CUDA;
  }
  return NP_OK;
}

int np_noalloc_check(void* stream) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return fail(NP_E_CUDA, "cudaGetDevice failed");
  if (dev < 0 || dev >= kMaxDevices) return fail(NP_E_INVAL, "device ordinal above 63");
  float* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lk(g_mu);
    scratch = g_scratch_addr[dev];
  }
  if (!scratch) return fail(NP_E_STATE, "np_predict_logits_noalloc has not run on this device");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int32_t word = 0;  // on the caller's stack: nothing is allocated
  cudaError_t e = cudaMemcpyAsync(&word, scratch, sizeof word, cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) {
    snprintf(g_err, sizeof g_err, "reading the status word failed: %s", cudaGetErrorString(e));
    return NP_E_CUDA;
  }
  if (word != 0) {
    snprintf(g_err, sizeof g_err,
             "the last np_predict_logits_noalloc on this device recorded status 0x%x (a bounded wait ran out): "
             "its logits are incomplete",
             (unsigned)word);
    return NP_E_DEVICE;
  }
  return NP_OK;
}

}  // extern "C"
