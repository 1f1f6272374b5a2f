// Router as a small MLP (Eq. 2: a lightweight MLP emits the two class logits; Eq. 9: the
// execute probability is their softmax).  u = W1 x + b1, a = max(u, 0), z = (w2[0] - w2[1]) . a
// + (b2[0] - b2[1]), p = 1 / (1 + exp(-z)).
//
// The hidden layer is a [T, d] x [d, h] contraction and runs on the tensor cores (warp MMA,
// bf16 x bf16 products are exact in fp32).  The decision that follows compares p with theta
// and must agree with an fp64 evaluation except within 1e-6 of theta, so the fp32 accumulators
// only ever hold 64 products: after every 64 input features they are added to fp64
// accumulators and cleared (error of the logit about 1e-7, of the probability below 1e-7).
// A CTA of two warps owns 32 token rows; x and W1 stream through a four-stage cp.async ring of
// 64-feature chunks (128-byte rows, 16-byte chunks XOR-swizzled by the row), several CTAs per
// SM keep enough of x in flight for the sweep to run near memory bandwidth.
#include "common.cuh"
#include "ptx.cuh"

namespace qtale {

using namespace ptx;

constexpr int kMlpRows = 32;     // token rows per CTA (16 per warp)
constexpr int kMlpThreads = 64;
constexpr int kMlpStages = 4;
constexpr int kMlpKC = 64;       // input features per stage
constexpr int kMlpMaxH = 64;     // hidden units (padded to a multiple of 8)

__device__ __forceinline__ void cp_async_16(void* smem, const void* gmem, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(smem)), "l"(gmem),
               "r"(src_bytes)
               : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

template <int NT>  // hidden units / 8
__global__ void __launch_bounds__(kMlpThreads)
    router_mlp_kernel(const __nv_bfloat16* __restrict__ x, int T, int d,
                      const __nv_bfloat16* __restrict__ w1, const float* __restrict__ b1,
                      const float* __restrict__ w2, int h, float b2_diff, float* __restrict__ scores) {
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int XB = kMlpRows * 128;   // bytes of an x stage
  constexpr int WB = NT * 8 * 128;     // bytes of a W1 stage
  unsigned char* sx = smem;
  unsigned char* sw = smem + kMlpStages * XB;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int row0 = blockIdx.x * kMlpRows;
  const int n_kc = (d + kMlpKC - 1) / kMlpKC;

  auto issue = [&](int kc) {
    const int s = kc % kMlpStages;
    const int k0 = kc * kMlpKC;
    for (int c = tid; c < kMlpRows * 8; c += kMlpThreads) {
      const int r = c >> 3, ch = c & 7;
      const int row = min(row0 + r, T - 1);
      const int k = k0 + ch * 8;
      cp_async_16(sx + s * XB + r * 128 + ((ch ^ (r & 7)) << 4), x + (size_t)row * d + min(k, d - 8),
                  k < d ? 16 : 0);
    }
    for (int c = tid; c < NT * 8 * 8; c += kMlpThreads) {
      const int r = c >> 3, ch = c & 7;
      const int k = k0 + ch * 8;
      cp_async_16(sw + s * WB + r * 128 + ((ch ^ (r & 7)) << 4),
                  w1 + (size_t)min(r, h - 1) * d + min(k, d - 8), (k < d && r < h) ? 16 : 0);
    }
  };

  float acc[NT][4];
  double acc64[NT][4];
#pragma unroll
  for (int j = 0; j < NT; ++j)
#pragma unroll
    for (int e = 0; e < 4; ++e) { acc[j][e] = 0.f; acc64[j][e] = 0.0; }

  for (int kc = 0; kc < kMlpStages - 1; ++kc) {
    if (kc < n_kc) issue(kc);
    cp_async_commit();
  }
  for (int kc = 0; kc < n_kc; ++kc) {
    cp_async_wait<kMlpStages - 2>();
    __syncthreads();  // stage kc has landed for every thread; stage kc - 1 is no longer read
    if (kc + kMlpStages - 1 < n_kc) issue(kc + kMlpStages - 1);
    cp_async_commit();
    const int s = kc % kMlpStages;
    const uint32_t xs = smem_u32(sx + s * XB), ws = smem_u32(sw + s * WB);
#pragma unroll
    for (int s16 = 0; s16 < kMlpKC / 16; ++s16) {
      const int mi = lane >> 3;
      uint32_t a[4];
      {
        const int r = warp * 16 + (mi & 1) * 8 + (lane & 7);
        const int ch = 2 * s16 + (mi >> 1);
        ldmatrix_x4(xs + r * 128 + ((ch ^ (r & 7)) << 4), a);
      }
#pragma unroll
      for (int j = 0; j < NT; j += 2) {
        uint32_t b[4];
        const int r = (j + (mi >> 1)) * 8 + (lane & 7);
        const int ch = 2 * s16 + (mi & 1);
        const int rc = min(r, NT * 8 - 1);  // odd NT: the second tile's lanes re-read the last row
        ldmatrix_x4(ws + rc * 128 + ((ch ^ (rc & 7)) << 4), b);
        mma_m16n8k16<false>(acc[j], a, b[0], b[1]);
        if (j + 1 < NT) mma_m16n8k16<false>(acc[j + 1], a, b[2], b[3]);
      }
    }
    // 64 products per fp32 accumulator: fold into fp64 and start over
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) { acc64[j][e] += (double)acc[j][e]; acc[j][e] = 0.f; }
  }
  cp_async_wait<0>();

  // hidden activation and output layer: this thread holds hidden units 8 j + 2 t, + 1 of rows g, g + 8
  const int g = lane >> 2, t = lane & 3;
  double z[2] = {0.0, 0.0};
#pragma unroll
  for (int j = 0; j < NT; ++j) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int col = j * 8 + 2 * t + (e & 1);
      if (col < h) {
        const double u = acc64[j][e] + (double)__ldg(b1 + col);
        const double a = u > 0.0 ? u : 0.0;
        z[e >> 1] += ((double)__ldg(w2 + col) - (double)__ldg(w2 + h + col)) * a;
      }
    }
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    z[r] += __shfl_xor_sync(0xffffffffu, z[r], 1);
    z[r] += __shfl_xor_sync(0xffffffffu, z[r], 2);
    const int row = row0 + warp * 16 + g + r * 8;
    if (t == 0 && row < T) scores[row] = (float)(1.0 / (1.0 + exp(-(z[r] + (double)b2_diff))));
  }
}

template <int NT>
static int launch_mlp(const void* x, int T, int d, const void* w1, const float* b1, const float* w2,
                      int h, float b2_diff, float* scores, cudaStream_t s) {
  const size_t smem = (size_t)kMlpStages * (kMlpRows * 128 + NT * 8 * 128);
  static bool configured[64] = {false};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return QTALE_ERR_CUDA;
  if (!configured[dev]) {
    if (cudaFuncSetAttribute(router_mlp_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)smem) != cudaSuccess)
      return QTALE_ERR_CUDA;
    configured[dev] = true;
  }
  router_mlp_kernel<NT><<<(T + kMlpRows - 1) / kMlpRows, kMlpThreads, smem, s>>>(
      static_cast<const __nv_bfloat16*>(x), T, d, static_cast<const __nv_bfloat16*>(w1), b1, w2, h,
      b2_diff, scores);
  return launch_status(cudaGetLastError());
}

int router_mlp_launch(const void* x, int T, int d, const void* w1, const float* b1, const float* w2,
                      int h, float b2_execute, float b2_bypass, float* scores, cudaStream_t s) {
  const float b2_diff = b2_execute - b2_bypass;
  const int nt = (h + 7) / 8;
  switch (nt) {
    case 1: return launch_mlp<1>(x, T, d, w1, b1, w2, h, b2_diff, scores, s);
    case 2: return launch_mlp<2>(x, T, d, w1, b1, w2, h, b2_diff, scores, s);
    case 3: case 4: return launch_mlp<4>(x, T, d, w1, b1, w2, h, b2_diff, scores, s);
    case 5: case 6: case 7: case 8: return launch_mlp<8>(x, T, d, w1, b1, w2, h, b2_diff, scores, s);
  }
  return QTALE_ERR_SHAPE;
}

}  // namespace qtale

using namespace qtale;

extern "C" {

int qtale_router_mlp_scores(const void* x, int T, int d, const void* w1, const float* b1,
                            const float* w2, int h, float b2_execute, float b2_bypass,
                            float* scores_out, void* stream) {
  if (!x || !w1 || !b1 || !w2 || !scores_out) return QTALE_ERR_NULL;
  if (T < 1 || d < 8 || d % 8 != 0 || h < 1 || h > kMlpMaxH) return QTALE_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(w1)) return QTALE_ERR_ALIGN;
  return router_mlp_launch(x, T, d, w1, b1, w2, h, b2_execute, b2_bypass, scores_out,
                           static_cast<cudaStream_t>(stream));
}

}  // extern "C"
