// Host-side runtime pieces of libqtale: status codes, device status word,
// device properties.
#include <math.h>

#include "common.cuh"

namespace qtale {

// One status word per device image of the library.
__device__ int g_device_status = 0;

static int g_sm_count[64] = {0};

int sm_count() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return QTALE_SM_COUNT_FALLBACK;
  if (g_sm_count[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
      n = QTALE_SM_COUNT_FALLBACK;
    g_sm_count[dev] = n;
  }
  return g_sm_count[dev];
}

int launch_status(cudaError_t e) { return e == cudaSuccess ? QTALE_OK : QTALE_ERR_CUDA; }

int* device_status_ptr() {
  static int* ptrs[64] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  if (!ptrs[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_device_status) != cudaSuccess) return nullptr;
    ptrs[dev] = static_cast<int*>(p);
  }
  return ptrs[dev];
}

}  // namespace qtale

extern "C" {

const char* qtale_strerror(int status) {
  switch (status) {
    case QTALE_OK: return "ok";
    case QTALE_ERR_NULL: return "a required pointer is NULL";
    case QTALE_ERR_ALIGN: return "pointer or pitch is not 16-byte aligned";
    case QTALE_ERR_SHAPE: return "unsupported or inconsistent sizes";
    case QTALE_ERR_BITS: return "bits must be 3 or 4";
    case QTALE_ERR_GROUP: return "group must be 64 or 128";
    case QTALE_ERR_WORKSPACE: return "workspace too small";
    case QTALE_ERR_CAPACITY: return "count exceeds buffer capacity";
    case QTALE_ERR_TIMEOUT: return "a bounded device-side wait gave up";
    case QTALE_ERR_CUDA: return "a CUDA call failed";
    case QTALE_ERR_MODE: return "unknown mode, epilogue or phase";
    default: return "unknown status";
  }
}

int qtale_device_status(void* stream) {
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaStreamSynchronize(s) != cudaSuccess) return QTALE_ERR_CUDA;
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, qtale::g_device_status, sizeof(int)) != cudaSuccess)
    return QTALE_ERR_CUDA;
  if (v != 0) {
    int zero = 0;
    if (cudaMemcpyToSymbol(qtale::g_device_status, &zero, sizeof(int)) != cudaSuccess)
      return QTALE_ERR_CUDA;
  }
  return v;
}

int qtale_topk_count(double ratio, int n_valid) {
  double k = floor(ratio * (double)n_valid + 0.5);
  if (k < 0) k = 0;
  if (k > n_valid) k = n_valid;
  return (int)k;
}

}  // extern "C"
