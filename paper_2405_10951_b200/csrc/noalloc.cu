// Linear-layer backward for callers that cannot allocate device memory.
//
// bsr_linear_backward splits the long reduction of the weight gradient over several CTAs and needs a
// float scratch buffer for the partial sums, which its caller normally allocates.  Some callers cannot:
// an on-device trainer whose memory was partitioned once at start-up and has no allocator left to ask,
// a plug-in inside a host application that owns every byte of device memory through its own pool, or a
// latency-critical loop in which cudaMalloc's implicit device-wide synchronisation is not acceptable.
// For them the scratch lives in a fixed array inside the library image.  Every GPU that loads the
// library holds these 16 MiB until the process exits.
#include <cstdio>
#include <mutex>

#include "../../include/bsr.h"
#include "common.cuh"
#include "kernels.h"

namespace {

constexpr size_t SCRATCH_FLOATS = BSR_STATIC_SCRATCH_BYTES / sizeof(float);
constexpr int MAX_DEVICES = 64;

// In host code this name is only a handle for the runtime, not an address a kernel may use:
// the device address is looked up with cudaGetSymbolAddress below.
static __device__ __align__(256) float g_static_scratch[SCRATCH_FLOATS];

std::mutex g_mutex;
float* g_scratch_ptr[MAX_DEVICES] = {nullptr};
int g_sm_count[MAX_DEVICES] = {0};
thread_local char g_noalloc_error[256] = "no error";

// Once per device, with that device current: resolve the array's device address.
int scratch_for_current_device(float** out, int* sms) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) {
    snprintf(g_noalloc_error, sizeof(g_noalloc_error), "no current CUDA device with an ordinal below %d", MAX_DEVICES);
    return -1;
  }
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_scratch_ptr[dev] == nullptr) {
    float* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress((void**)&p, g_static_scratch);
    if (e != cudaSuccess || p == nullptr) {
      snprintf(g_noalloc_error, sizeof(g_noalloc_error), "cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
      return -2;
    }
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
      snprintf(g_noalloc_error, sizeof(g_noalloc_error), "the device's multiprocessor count could not be read");
      return -3;
    }
    g_scratch_ptr[dev] = p;
    g_sm_count[dev] = n;
  }
  *out = g_scratch_ptr[dev];
  *sms = g_sm_count[dev];
  return 0;
}

}  // namespace

extern "C" {

const char* bsr_static_last_error(void) { return g_noalloc_error; }

int32_t bsr_linear_backward_static(const void* x, const void* w, const void* dy, void* dx, float* dw, int32_t m, int32_t n,
                                   int32_t k, void* stream) {
  using namespace bsr;
  if (x == nullptr || w == nullptr || dy == nullptr || dx == nullptr || dw == nullptr) {
    snprintf(g_noalloc_error, sizeof(g_noalloc_error), "null argument");
    return BSR_ERR_INVALID_ARG;
  }
  if (m < 8 || n < 8 || k < 8 || (m % 8) || (n % 8) || (k % 8)) {
    snprintf(g_noalloc_error, sizeof(g_noalloc_error), "m, n, k must be positive multiples of 8 (bf16 tensor-core path)");
    return BSR_ERR_INVALID_ARG;
  }
  if ((size_t)n * (size_t)k * 2 > SCRATCH_FLOATS) {
    snprintf(g_noalloc_error, sizeof(g_noalloc_error),
             "weight of %d x %d elements exceeds the built-in scratch: n * k must not exceed %zu", n, k, SCRATCH_FLOATS / 2);
    return BSR_ERR_WORKSPACE_TOO_SMALL;
  }
  float* scratch = nullptr;
  int sms = 0;
  if (scratch_for_current_device(&scratch, &sms) != 0) return BSR_ERR_CUDA;   // the message says which step failed
  Ctx c;
  c.stream = (cudaStream_t)stream;
  c.dtype = BSR_DTYPE_BF16;
  c.status = nullptr;
  c.sm_count = sms;
  c.use_tc = 1;
  GemmEpilogue none;
  // Every partial sum in the scratch is rewritten in full by the call that uses it, so nothing has to be
  // cleared between calls; what the previous call left there is never read.
  int rc = gemm_tc_strided(c, dy, n, 1, w, 1, k, dx, 0, m, k, n, none, nullptr, 0);               // dX = dY W
  if (rc == 0) rc = gemm_tc_strided(c, dy, 1, n, x, 1, k, dw, 1, n, k, m, none, scratch, SCRATCH_FLOATS);   // dW = dY^T X
  if (rc != 0) {
    snprintf(g_noalloc_error, sizeof(g_noalloc_error), "tcgen05 GEMM set-up failed (%d)", rc);
    return BSR_ERR_CUDA;
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    snprintf(g_noalloc_error, sizeof(g_noalloc_error), "launch failed: %s", cudaGetErrorString(e));
    return BSR_ERR_CUDA;
  }
  snprintf(g_noalloc_error, sizeof(g_noalloc_error), "no error");
  return BSR_OK;
}

}  // extern "C"
