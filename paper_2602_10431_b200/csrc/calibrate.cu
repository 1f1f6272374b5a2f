// Ratio-targeted threshold (Sec. 3.4, Eq. 9; App. A.1): the single global theta for which a
// requested share of the router scores of a calibration batch, pooled over all layers, lies at
// or above it.  The paper searches theta on a grid by task accuracy; this is the mechanical
// half of that search, the exact quantile, computed on the device: an MSB-first radix select
// (four passes of eight bits over the order-preserving integer image of the fp32 scores), each
// pass one launch whose CTAs histogram a slice of the scores and whose last CTA (ticket
// counter) picks the digit that holds the target rank.
#include "common.cuh"

namespace qtale {

constexpr int kCalThreads = 512;

// scratch words
constexpr int kCalTicket = 0;     // [4] one ticket per pass + [1] for the counting pass
constexpr int kCalValid = 8;      // valid scores (accumulated in pass 0)
constexpr int kCalPrefix = 9;     // digits chosen so far (high bits of the key)
constexpr int kCalRemain = 10;    // rank still to be located inside the prefix (1-based)
constexpr int kCalNone = 11;      // 1: k = 0, nothing executes
constexpr int kCalCount = 12;     // scores >= theta (counting pass)
constexpr int kCalHist = 16;      // 4 x 256 counters
constexpr int kCalWords = kCalHist + 4 * 256;

__device__ __forceinline__ uint32_t cal_key(float s) {
  const uint32_t b = __float_as_uint(s);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float cal_unkey(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

// pass = 0..3: histogram of digit `pass` among the valid scores whose higher digits equal the
// prefix; pass = 4: count of valid scores >= theta and the outputs.
__global__ void __launch_bounds__(kCalThreads)
    theta_pass_kernel(const float* __restrict__ scores, const uint8_t* __restrict__ valid, size_t n,
                      int pass, double ratio, uint32_t* ws, float* theta_out, int32_t* count_out) {
  __shared__ uint32_t s_hist[256];
  __shared__ int s_last;
  const int tid = threadIdx.x;
  for (int i = tid; i < 256; i += kCalThreads) s_hist[i] = 0;
  __syncthreads();
  const uint32_t prefix = pass > 0 ? ws[kCalPrefix] : 0u;
  const uint32_t none = pass > 0 ? ws[kCalNone] : 0u;
  const int shift = 24 - 8 * pass;
  const uint32_t mask = pass == 0 ? 0u : (pass >= 4 ? 0xFFFFFFFFu : 0xFFFFFFFFu << (shift + 8));
  uint32_t n_valid = 0, n_ge = 0;
  for (size_t i = blockIdx.x * (size_t)kCalThreads + tid; i < n; i += (size_t)gridDim.x * kCalThreads) {
    if (valid && !valid[i]) continue;
    const uint32_t key = cal_key(scores[i]);
    ++n_valid;
    if (pass < 4) {
      if ((key & mask) == prefix) atomicAdd(&s_hist[(key >> shift) & 0xFFu], 1u);
    } else {
      n_ge += key >= prefix ? 1u : 0u;
    }
  }
  __syncthreads();
  if (pass < 4) {
    for (int i = tid; i < 256; i += kCalThreads)
      if (s_hist[i]) atomicAdd(ws + kCalHist + pass * 256 + i, s_hist[i]);
  }
  n_valid = __reduce_add_sync(0xffffffffu, n_valid);
  n_ge = __reduce_add_sync(0xffffffffu, n_ge);
  if ((tid & 31) == 0) {
    if (pass == 0 && n_valid) atomicAdd(ws + kCalValid, n_valid);
    if (pass == 4 && n_ge) atomicAdd(ws + kCalCount, n_ge);
  }
  // the CTA that finishes last closes the pass
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = atomicAdd(ws + kCalTicket + pass, 1u) == gridDim.x - 1;
  __syncthreads();
  if (!s_last || tid != 0) return;
  __threadfence();
  if (pass == 4) {
    *theta_out = none ? 2.0f : cal_unkey(prefix);  // scores are probabilities: 2 is above all of them
    *count_out = none ? 0 : (int32_t)__ldcg(ws + kCalCount);
    return;
  }
  if (pass == 0) {
    const uint32_t nv = __ldcg(ws + kCalValid);
    double kd = floor(ratio * (double)nv + 0.5);
    kd = kd < 0.0 ? 0.0 : (kd > (double)nv ? (double)nv : kd);
    ws[kCalRemain] = (uint32_t)kd;
    ws[kCalNone] = kd < 1.0 ? 1u : 0u;
  }
  if (ws[kCalNone]) return;
  uint32_t rem = ws[kCalRemain];
  int digit = 0;
  for (int b = 255; b >= 0; --b) {
    const uint32_t c = __ldcg(ws + kCalHist + pass * 256 + b);
    if (rem <= c) { digit = b; break; }
    rem -= c;
  }
  ws[kCalPrefix] = prefix | ((uint32_t)digit << shift);
  ws[kCalRemain] = rem;
}

}  // namespace qtale

using namespace qtale;

extern "C" {

size_t qtale_theta_workspace_bytes(void) { return (size_t)kCalWords * sizeof(uint32_t); }

int qtale_theta_for_ratio(const float* scores, const uint8_t* valid, size_t n, double ratio,
                          float* theta_out, int32_t* count_out, void* ws, size_t ws_bytes,
                          void* stream) {
  if (!scores || !theta_out || !count_out || !ws) return QTALE_ERR_NULL;
  if (n < 1 || n > ((size_t)1 << 31) || !(ratio >= 0.0 && ratio <= 1.0)) return QTALE_ERR_SHAPE;
  if (ws_bytes < qtale_theta_workspace_bytes()) return QTALE_ERR_WORKSPACE;
  if (!aligned16(ws)) return QTALE_ERR_ALIGN;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(ws, 0, qtale_theta_workspace_bytes(), s) != cudaSuccess) return QTALE_ERR_CUDA;
  size_t want = (n + (size_t)kCalThreads * 8 - 1) / ((size_t)kCalThreads * 8);
  int grid = (int)(want < 1 ? 1 : (want > (size_t)sm_count() * 2 ? (size_t)sm_count() * 2 : want));
  for (int pass = 0; pass <= 4; ++pass) {
    theta_pass_kernel<<<grid, kCalThreads, 0, s>>>(scores, valid, n, pass, ratio,
                                                   static_cast<uint32_t*>(ws), theta_out, count_out);
    if (cudaGetLastError() != cudaSuccess) return QTALE_ERR_CUDA;
  }
  return QTALE_OK;
}

}  // extern "C"
