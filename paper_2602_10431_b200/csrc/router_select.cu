// Router score + execute decision + ordered compaction (Eq. 2, Eq. 9; App. B.2).
//
// One launch.  Phase A (all CTAs): z_t = w . x_t + b accumulated in fp64 over a
// bandwidth-bound sweep of x, p_t = 1 / (1 + exp(-z_t)) stored as fp32.  Phase
// B (the CTA that finishes last, found with a ticket counter): threshold or
// top-k decision on the fp32 scores and an ordered prefix-sum compaction into
// the ascending index list, the per-sequence offsets and the positions.
#include "common.cuh"

namespace qtale {

constexpr int kRouterThreads = 512;  // 16 warps
constexpr int kRowsPerWarp = 2;
constexpr int kSelectThreads = 1024;  // upper bound of the CTA size the selection code supports

struct RouterParams {
  const __nv_bfloat16* x;
  const float* w;
  const float* scores_override;
  const uint8_t* valid;
  const int32_t* cu_seqlens;
  const int32_t* pos0;
  float* scores;
  int32_t* idx;
  int32_t* n_exec;
  int32_t* cu_exec;
  int32_t* pos;
  unsigned int* ticket;
  int T, d, B, mode, k;
  float bias, theta;
};

__device__ __forceinline__ uint32_t score_key(float s) {
  uint32_t b = __float_as_uint(s);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// ---- phase B: decision + compaction, executed by one CTA of kSelectThreads ----
__device__ void select_and_compact(const RouterParams& p, uint32_t* sh_hist, int* sh_scan) {
  const int tid = threadIdx.x;
  const int nthr = blockDim.x;
  const int T = p.T;
  __shared__ uint32_t s_prefix, s_mask;
  __shared__ int s_remaining, s_need_eq, s_total;

  uint32_t tau = 0;  // key of the k-th largest score (top-k)
  int need_eq = 0;   // how many tokens with key == tau execute (lowest indices first)

  if (p.mode == QTALE_SELECT_TOPK) {
    // MSB-first radix select of the k-th largest key among valid tokens.
    if (tid == 0) {
      s_prefix = 0;
      s_mask = 0;
      s_remaining = p.k;
    }
    __syncthreads();
    for (int pass = 0; pass < 4 && p.k > 0; ++pass) {
      const int shift = 24 - 8 * pass;
      for (int i = tid; i < 256; i += nthr) sh_hist[i] = 0;
      __syncthreads();
      const uint32_t prefix = s_prefix, mask = s_mask;
      for (int t = tid; t < T; t += nthr) {
        if (p.valid && !p.valid[t]) continue;
        uint32_t key = score_key(__ldcg(p.scores + t));
        if ((key & mask) == prefix) {
          // scores cluster in a few buckets: one atomic per distinct bucket per warp
          const uint32_t bucket = (key >> shift) & 0xFF;
          const uint32_t peers = __match_any_sync(__activemask(), bucket);
          if ((int)(__ffs(peers) - 1) == (threadIdx.x & 31)) atomicAdd(&sh_hist[bucket], __popc(peers));
        }
      }
      __syncthreads();
      if (tid == 0) {
        int rem = s_remaining;
        int b = 255;
        for (; b > 0; --b) {
          int c = (int)sh_hist[b];
          if (c >= rem) break;
          rem -= c;
        }
        s_remaining = rem;  // rank of the target inside bucket b (1-based)
        s_prefix = prefix | ((uint32_t)b << shift);
        s_mask = mask | (0xFFu << shift);
      }
      __syncthreads();
    }
    tau = s_prefix;
    need_eq = (p.k > 0) ? s_remaining : 0;
  }

  // ordered compaction: each thread owns a contiguous chunk of tokens
  const int chunk = (T + nthr - 1) / nthr;
  const int t0 = min(T, tid * chunk), t1 = min(T, t0 + chunk);
  int n_sel = 0, n_eq = 0;
  for (int t = t0; t < t1; ++t) {
    const bool ok = !p.valid || p.valid[t];
    const float s = __ldcg(p.scores + t);
    if (p.mode == QTALE_SELECT_TOPK) {
      const uint32_t key = score_key(s);
      n_sel += (ok && p.k > 0 && key > tau);
      n_eq += (ok && p.k > 0 && key == tau);
    } else {
      n_sel += (ok && s >= p.theta);
    }
  }
  // block-wide exclusive scans of (n_sel, n_eq) with warp shuffles
  auto block_exclusive = [&](int v, int& total) -> int {
    const int lane = tid & 31, wid = tid >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int n = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += n;
    }
    __syncthreads();
    if (lane == 31) sh_scan[wid] = inc;
    __syncthreads();
    if (wid == 0) {
      int w = (lane < (nthr >> 5)) ? sh_scan[lane] : 0;
      int winc = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, winc, o);
        if (lane >= o) winc += n;
      }
      sh_scan[32 + lane] = winc - w;  // exclusive warp offsets
      if (lane == 31) s_total = winc;
    }
    __syncthreads();
    total = s_total;
    return inc - v + sh_scan[32 + wid];
  };
  int tot_eq = 0, tot_sel = 0;
  int eq_before = 0;
  if (p.mode == QTALE_SELECT_TOPK) eq_before = block_exclusive(n_eq, tot_eq);
  int sel_before = block_exclusive(n_sel, tot_sel);
  int out = sel_before;
  int total = tot_sel;
  if (p.mode == QTALE_SELECT_TOPK) {
    out += min(eq_before, need_eq);
    total += min(tot_eq, need_eq);
  }

  // sequence of the first token of the chunk: largest b with cu_seqlens[b] <= t0
  int b = 0;
  if (t0 < t1) {
    int lo = 0, hi = p.B;  // invariant: cu[lo] <= t0 < cu[hi] (cu[B] = T > t0)
    while (hi - lo > 1) {
      int mid = (lo + hi) >> 1;
      if (p.cu_seqlens[mid] <= t0) lo = mid; else hi = mid;
    }
    b = lo;
  }
  int e = eq_before;
  for (int t = t0; t < t1; ++t) {
    while (b + 1 < p.B && t >= p.cu_seqlens[b + 1]) ++b;
    const bool ok = !p.valid || p.valid[t];
    const float s = __ldcg(p.scores + t);
    bool take;
    if (p.mode == QTALE_SELECT_TOPK) {
      const uint32_t key = score_key(s);
      take = ok && p.k > 0 && key > tau;
      if (ok && p.k > 0 && key == tau) {
        take = e < need_eq;
        ++e;
      }
    } else {
      take = ok && s >= p.theta;
    }
    if (take) {
      p.idx[out] = t;
      p.pos[out] = t - p.cu_seqlens[b] + (p.pos0 ? p.pos0[b] : 0);
      ++out;
    }
  }
  __syncthreads();
  if (tid == 0) *p.n_exec = total;
  // cu_exec[b] = number of executed tokens with index < cu_seqlens[b]
  for (int q = tid; q <= p.B; q += nthr) {
    const int bound = p.cu_seqlens[q];
    int lo = 0, hi = total;
    while (lo < hi) {
      int mid = (lo + hi) >> 1;
      if (p.idx[mid] < bound) lo = mid + 1; else hi = mid;
    }
    p.cu_exec[q] = lo;
  }
}

// ---- the fused kernel -------------------------------------------------------
__global__ void __launch_bounds__(kRouterThreads)
    router_select_kernel(const RouterParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ uint32_t sh_hist[256];
  __shared__ int sh_scan[64];
  __shared__ int s_is_last;

  const int tid = threadIdx.x;
  if (p.scores_override == nullptr) {
    // phase A: router GEMV.  Router weights staged in shared memory as fp64,
    // laid out [iteration][element j of the lane's 8][lane] so that the 32
    // lanes of a warp read consecutive doubles.
    double* w_s = reinterpret_cast<double*>(smem_raw);
    const int d = p.d;
    const int n_it = (d + 255) / 256;
    for (int i = tid; i < n_it * 256; i += blockDim.x) {
      const int it = i >> 8, rem = i & 255, lane = rem >> 3, j = rem & 7;
      w_s[(it * 8 + j) * 32 + lane] = (i < d) ? (double)p.w[i] : 0.0;
    }
    __syncthreads();
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int warps_per_cta = blockDim.x >> 5;
    const int n_groups = (p.T + kRowsPerWarp - 1) / kRowsPerWarp;
    for (int g = blockIdx.x * warps_per_cta + warp; g < n_groups; g += gridDim.x * warps_per_cta) {
      const int r0 = g * kRowsPerWarp;
      double acc[kRowsPerWarp];
#pragma unroll
      for (int r = 0; r < kRowsPerWarp; ++r) acc[r] = 0.0;
      for (int it = 0; it < n_it; ++it) {
        const int col = it * 256 + lane * 8;
        uint4 v[kRowsPerWarp];
#pragma unroll
        for (int r = 0; r < kRowsPerWarp; ++r) {
          const int row = min(r0 + r, p.T - 1);
          v[r] = (col < d) ? ld_nc_16(p.x + (size_t)row * d + col) : make_uint4(0, 0, 0, 0);
        }
        double wv[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) wv[j] = w_s[(it * 8 + j) * 32 + lane];
#pragma unroll
        for (int r = 0; r < kRowsPerWarp; ++r) {
          const uint32_t u[4] = {v[r].x, v[r].y, v[r].z, v[r].w};
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            acc[r] = fma((double)bf16_lo(u[q]), wv[2 * q], acc[r]);
            acc[r] = fma((double)bf16_hi(u[q]), wv[2 * q + 1], acc[r]);
          }
        }
      }
#pragma unroll
      for (int r = 0; r < kRowsPerWarp; ++r) {
        const double z = warp_sum(acc[r]) + (double)p.bias;
        if (lane == 0 && r0 + r < p.T) p.scores[r0 + r] = (float)(1.0 / (1.0 + exp(-z)));
      }
    }
  } else {
    for (int t = blockIdx.x * blockDim.x + tid; t < p.T; t += gridDim.x * blockDim.x)
      p.scores[t] = p.scores_override[t];
  }

  // ticket: the CTA that arrives last runs the selection
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const unsigned int t = atomicAdd(p.ticket, 1u);
    s_is_last = (t == gridDim.x - 1);
  }
  __syncthreads();
  if (!s_is_last) return;
  __threadfence();
  select_and_compact(p, sh_hist, sh_scan);
  if (tid == 0) *p.ticket = 0;  // leave the counter ready for the next launch
}

// ---- bookkeeping for a caller-supplied index list ----------------------------
__global__ void index_bookkeeping_kernel(const int32_t* idx, int n, const int32_t* cu_seqlens,
                                         int B, const int32_t* pos0, int32_t* n_exec,
                                         int32_t* cu_exec, int32_t* pos) {
  const int gtid = blockIdx.x * blockDim.x + threadIdx.x;
  const int stride = gridDim.x * blockDim.x;
  if (gtid == 0) *n_exec = n;
  for (int q = gtid; q <= B; q += stride) {
    const int bound = cu_seqlens[q];
    int lo = 0, hi = n;
    while (lo < hi) {
      int mid = (lo + hi) >> 1;
      if (idx[mid] < bound) lo = mid + 1; else hi = mid;
    }
    cu_exec[q] = lo;
  }
  for (int i = gtid; i < n; i += stride) {
    const int t = idx[i];
    int lo = 0, hi = B;
    while (hi - lo > 1) {
      int mid = (lo + hi) >> 1;
      if (cu_seqlens[mid] <= t) lo = mid; else hi = mid;
    }
    pos[i] = t - cu_seqlens[lo] + (pos0 ? pos0[lo] : 0);
  }
}

}  // namespace qtale

using namespace qtale;

extern "C" {

size_t qtale_router_select_workspace_bytes(int T) {
  (void)T;
  return 256;  // ticket counter (kept zero between launches)
}

int qtale_router_select(const void* x, int T, int d, const float* w_router, float bias,
                        const float* scores_override, const uint8_t* valid,
                        const int32_t* cu_seqlens, int B, const int32_t* pos0, int mode,
                        float theta, int k, float* scores_out, int32_t* idx_out,
                        int32_t* n_exec_out, int32_t* cu_exec_out, int32_t* pos_out, void* ws,
                        size_t ws_bytes, void* stream) {
  if (!scores_out || !idx_out || !n_exec_out || !cu_exec_out || !pos_out || !cu_seqlens || !ws)
    return QTALE_ERR_NULL;
  if (!scores_override && (!x || !w_router)) return QTALE_ERR_NULL;
  if (T < 1 || T > (1 << 24) || B < 1 || B > T) return QTALE_ERR_SHAPE;
  if (!scores_override && (d < 8 || d % 8 != 0 || d > 16384)) return QTALE_ERR_SHAPE;
  if (mode != QTALE_SELECT_THRESHOLD && mode != QTALE_SELECT_TOPK) return QTALE_ERR_MODE;
  if (mode == QTALE_SELECT_TOPK && (k < 0 || k > T)) return QTALE_ERR_CAPACITY;
  if (!aligned16(x) || !aligned16(ws)) return QTALE_ERR_ALIGN;
  if (ws_bytes < qtale_router_select_workspace_bytes(T)) return QTALE_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);

  RouterParams p;
  p.x = static_cast<const __nv_bfloat16*>(x);
  p.w = w_router;
  p.scores_override = scores_override;
  p.valid = valid;
  p.cu_seqlens = cu_seqlens;
  p.pos0 = pos0;
  p.scores = scores_out;
  p.idx = idx_out;
  p.n_exec = n_exec_out;
  p.cu_exec = cu_exec_out;
  p.pos = pos_out;
  p.ticket = static_cast<unsigned int*>(ws);
  p.T = T; p.d = d; p.B = B; p.mode = mode; p.k = k;
  p.bias = bias; p.theta = theta;

  if (cudaMemsetAsync(ws, 0, sizeof(unsigned int), s) != cudaSuccess) return QTALE_ERR_CUDA;
  int grid;
  size_t smem = 0;
  if (scores_override) {
    grid = 1;
  } else {
    const int n_it = (d + 255) / 256;
    smem = (size_t)n_it * 256 * sizeof(double);
    const int warps = kRouterThreads / 32;
    const int n_groups = (T + kRowsPerWarp - 1) / kRowsPerWarp;
    grid = (n_groups + warps - 1) / warps;
    const int cap = sm_count() * 2;
    if (grid > cap) grid = cap;
    if (grid < 1) grid = 1;
    if (smem > 48 * 1024) {
      if (cudaFuncSetAttribute(router_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               (int)smem) != cudaSuccess)
        return QTALE_ERR_CUDA;
    }
  }
  router_select_kernel<<<grid, kRouterThreads, smem, s>>>(p);
  return launch_status(cudaGetLastError());
}

// ---- variant for callers that cannot allocate device memory -------------------
// The kernel's only scratch is its ticket counter; here it lives in a static
// device array that every GPU loading the library carries until exit.
#define QTALE_ROUTER_STATIC_SCRATCH_BYTES 256
static __device__ __align__(256) unsigned char g_router_static_scratch[QTALE_ROUTER_STATIC_SCRATCH_BYTES];

int qtale_router_select_static(const void* x, int T, int d, const float* w_router, float bias,
                               const float* scores_override, const uint8_t* valid,
                               const int32_t* cu_seqlens, int B, const int32_t* pos0, int mode,
                               float theta, int k, float* scores_out, int32_t* idx_out,
                               int32_t* n_exec_out, int32_t* cu_exec_out, int32_t* pos_out,
                               void* stream) {
  // In host code the array's name is only a handle; its device address has to be
  // asked for, once per device, with that device current.
  static void* scratch_of_device[64] = {nullptr};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return QTALE_ERR_CUDA;
  if (T >= 1 && qtale_router_select_workspace_bytes(T) > (size_t)QTALE_ROUTER_STATIC_SCRATCH_BYTES)
    return QTALE_ERR_CAPACITY;  // the built-in scratch is too small for this many tokens
  if (!scratch_of_device[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_router_static_scratch) != cudaSuccess || !ptr)
      return QTALE_ERR_CUDA;
    scratch_of_device[dev] = ptr;
  }
  // The shared entry point zeroes the ticket word (cudaMemsetAsync on the stream)
  // before the launch, so whatever the previous call left behind does not matter.
  return qtale_router_select(x, T, d, w_router, bias, scores_override, valid, cu_seqlens, B, pos0,
                             mode, theta, k, scores_out, idx_out, n_exec_out, cu_exec_out, pos_out,
                             scratch_of_device[dev], QTALE_ROUTER_STATIC_SCRATCH_BYTES, stream);
}

int qtale_index_bookkeeping(const int32_t* idx, int n, int T, const int32_t* cu_seqlens, int B,
                            const int32_t* pos0, int32_t* n_exec_out, int32_t* cu_exec_out,
                            int32_t* pos_out, void* stream) {
  if (!cu_seqlens || !n_exec_out || !cu_exec_out || !pos_out) return QTALE_ERR_NULL;
  if (n < 0 || n > T || B < 1) return QTALE_ERR_CAPACITY;
  if (n > 0 && !idx) return QTALE_ERR_NULL;
  const int threads = 256;
  int blocks = (max(n, B + 1) + threads - 1) / threads;
  if (blocks < 1) blocks = 1;
  if (blocks > 1024) blocks = 1024;
  index_bookkeeping_kernel<<<blocks, threads, 0, static_cast<cudaStream_t>(stream)>>>(
      idx, n, cu_seqlens, B, pos0, n_exec_out, cu_exec_out, pos_out);
  return launch_status(cudaGetLastError());
}

}  // extern "C"
