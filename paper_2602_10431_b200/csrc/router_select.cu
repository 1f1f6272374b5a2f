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
  __shared__ int s_remaining, s_total, s_bucket, s_new_remaining;

  uint32_t tau = 0;  // key of the k-th largest score (top-k)
  int need_eq = 0;   // how many tokens with key == tau execute (lowest indices first)

  if (p.mode == QTALE_SELECT_TOPK) {
    // MSB-first radix select of the k-th largest key among valid tokens.  Keys are read
    // in batches of kBatch independent loads per thread (token t = (batch*kBatch + j) * nthr
    // + tid); when a thread's share fits one batch it is read once and kept in registers.
    constexpr int kBatch = 16;
    constexpr uint32_t kInvalid = 0u;  // key 0 is below every real key (those have a set bit)
    if (tid == 0) {
      s_prefix = 0;
      s_mask = 0;
      s_remaining = p.k;
    }
    const int per = (T + nthr - 1) / nthr;
    const int n_batches = (per + kBatch - 1) / kBatch;
    uint32_t keys[kBatch];
    auto load_batch = [&](int bi) {
#pragma unroll
      for (int j = 0; j < kBatch; ++j) {
        const int t = (bi * kBatch + j) * nthr + tid;
        float sc = 0.f;
        bool ok = t < T;
        if (ok) sc = __ldcg(p.scores + t);
        if (ok && p.valid) ok = p.valid[t] != 0;
        keys[j] = ok ? score_key(sc) : kInvalid;
      }
    };
    if (n_batches == 1) load_batch(0);
    __syncthreads();
    for (int pass = 0; pass < 4 && p.k > 0; ++pass) {
      const int shift = 24 - 8 * pass;
      for (int i = tid; i < 256; i += nthr) sh_hist[i] = 0;
      if (tid == 0) {  // defaults if k exceeds the number of valid tokens: lowest bucket
        s_bucket = 0;
        s_new_remaining = s_remaining;
      }
      __syncthreads();
      const uint32_t prefix = s_prefix, mask = s_mask;
      for (int bi = 0; bi < n_batches; ++bi) {
        if (n_batches > 1) load_batch(bi);
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
          const uint32_t key = keys[j];
          const bool in = key != kInvalid && (key & mask) == prefix;
          // scores cluster in a few buckets: one atomic per distinct bucket per warp
          const uint32_t bucket = in ? ((key >> shift) & 0xFF) : 256u;
          const uint32_t peers = __match_any_sync(0xffffffffu, bucket);
          if (in && (int)(__ffs(peers) - 1) == (tid & 31)) atomicAdd(&sh_hist[bucket], __popc(peers));
        }
      }
      __syncthreads();
      // bucket holding the target: suffix sums over the 256 buckets, one bucket per thread
      {
        const int lane = tid & 31, wid = tid >> 5;
        int h = 0, inc = 0;
        if (tid < 256) {
          h = (int)sh_hist[255 - tid];  // descending bucket order
          inc = h;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const int n = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += n;
          }
          if (lane == 31) sh_scan[wid] = inc;
        }
        __syncthreads();
        if (tid < 256) {
          int before = 0;
          for (int w = 0; w < wid; ++w) before += sh_scan[w];
          inc += before;
          const int rem = s_remaining;
          if (inc >= rem && inc - h < rem) {  // exactly one thread (bucket counts are >= 0)
            s_bucket = 255 - tid;
            s_new_remaining = rem - (inc - h);
          }
        }
        __syncthreads();
        if (tid == 0) {
          s_remaining = s_new_remaining;  // rank of the target inside the bucket (1-based)
          s_prefix = prefix | ((uint32_t)s_bucket << shift);
          s_mask = mask | (0xFFu << shift);
        }
        __syncthreads();
      }
    }
    tau = s_prefix;
    need_eq = (p.k > 0) ? s_remaining : 0;
  }

  // ordered compaction: each thread owns a contiguous chunk of tokens, read in batches of
  // independent loads
  constexpr int kCB = 16;
  const int chunk = (T + nthr - 1) / nthr;
  const int t0 = min(T, tid * chunk), t1 = min(T, t0 + chunk);
  float cs[kCB];
  bool cv[kCB];
  auto load_chunk = [&](int base) {
#pragma unroll
    for (int j = 0; j < kCB; ++j) {
      const int t = base + j;
      cs[j] = 0.f;
      cv[j] = false;
      if (t < t1) {
        cs[j] = __ldcg(p.scores + t);
        cv[j] = !p.valid || p.valid[t];
      }
    }
  };
  int n_sel = 0, n_eq = 0;
  for (int base = t0; base < t1; base += kCB) {
    load_chunk(base);
#pragma unroll
    for (int j = 0; j < kCB; ++j) {
      if (p.mode == QTALE_SELECT_TOPK) {
        const uint32_t key = score_key(cs[j]);
        n_sel += (cv[j] && p.k > 0 && key > tau);
        n_eq += (cv[j] && p.k > 0 && key == tau);
      } else {
        n_sel += (cv[j] && cs[j] >= p.theta);
      }
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

  // Sequence bookkeeping of the chunk.  b = sequence of the current token; q = next entry of
  // cu_seqlens not yet passed.  The thread whose chunk contains token cu_seqlens[q] writes
  // cu_exec[q] = executed tokens before it; entries equal to T are written at the end.
  int b = 0, q = 0, seq_start = 0, seq_pos0 = 0, next_bound = T + 1;
  if (t0 < t1) {
    int lo = 0, hi = p.B;  // invariant: cu[lo] <= t0 < cu[hi] (cu[B] = T > t0)
    while (hi - lo > 1) {
      int mid = (lo + hi) >> 1;
      if (p.cu_seqlens[mid] <= t0) lo = mid; else hi = mid;
    }
    b = lo;
    q = b + 1;
    if (p.cu_seqlens[b] == t0) {  // boundaries sitting exactly on the chunk start are ours
      q = b;
      while (q > 0 && p.cu_seqlens[q - 1] == t0) --q;
    }
    seq_start = p.cu_seqlens[b];
    seq_pos0 = p.pos0 ? p.pos0[b] : 0;
    next_bound = p.cu_seqlens[q];
  }
  int e = eq_before;
  for (int base = t0; base < t1; base += kCB) {
    if (chunk > kCB || base != t0) load_chunk(base);  // a single batch is still in registers
#pragma unroll
    for (int j = 0; j < kCB; ++j) {
      const int t = base + j;
      if (t >= t1) break;
      while (t >= next_bound) {  // token t opens sequence q (or skips empty ones)
        p.cu_exec[q] = out;
        if (q < p.B) {
          b = q;
          seq_start = next_bound;
          seq_pos0 = p.pos0 ? p.pos0[b] : 0;
        }
        ++q;
        next_bound = q <= p.B ? p.cu_seqlens[q] : T + 1;
      }
      bool take;
      if (p.mode == QTALE_SELECT_TOPK) {
        const uint32_t key = score_key(cs[j]);
        take = cv[j] && p.k > 0 && key > tau;
        if (cv[j] && p.k > 0 && key == tau) {
          take = e < need_eq;
          ++e;
        }
      } else {
        take = cv[j] && cs[j] >= p.theta;
      }
      if (take) {
        p.idx[out] = t;
        p.pos[out] = t - seq_start + seq_pos0;
        ++out;
      }
    }
  }
  if (tid == 0) *p.n_exec = total;
  for (int qq = tid; qq <= p.B; qq += nthr)
    if (p.cu_seqlens[qq] >= T) p.cu_exec[qq] = total;
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
    // phase A: router GEMV.  Router weights staged in shared memory as fp32, laid out
    // [iteration][lane][8] so a lane's eight weights are two 16-byte loads.  Each 16-byte
    // load of x (8 bf16) is reduced with fp32 FMAs into a block sum, and the block sums
    // are accumulated in fp64: conversions and fp64 adds are one per 8 elements, which
    // keeps the sweep bandwidth bound, and the result stays within about 1e-8 of the
    // all-fp64 dot product.
    float* w_s = reinterpret_cast<float*>(smem_raw);
    const int d = p.d;
    const int n_it = (d + 255) / 256;
    for (int i = tid; i < n_it * 256; i += blockDim.x) w_s[i] = (i < d) ? p.w[i] : 0.f;
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
      constexpr int kUnroll = 4;  // 16-byte loads in flight per lane: kUnroll x rows per warp
      for (int it0 = 0; it0 < n_it; it0 += kUnroll) {
        uint4 v[kUnroll][kRowsPerWarp];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
          const int col = (it0 + u) * 256 + lane * 8;
#pragma unroll
          for (int r = 0; r < kRowsPerWarp; ++r) {
            const int row = min(r0 + r, p.T - 1);
            v[u][r] = (it0 + u < n_it && col < d) ? ld_nc_16(p.x + (size_t)row * d + col)
                                                  : make_uint4(0, 0, 0, 0);
          }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
          if (it0 + u >= n_it) break;
          const float4 wa = *reinterpret_cast<const float4*>(w_s + (it0 + u) * 256 + lane * 8);
          const float4 wb = *reinterpret_cast<const float4*>(w_s + (it0 + u) * 256 + lane * 8 + 4);
#pragma unroll
          for (int r = 0; r < kRowsPerWarp; ++r) {
            float blk = bf16_lo(v[u][r].x) * wa.x;
            blk = fmaf(bf16_hi(v[u][r].x), wa.y, blk);
            blk = fmaf(bf16_lo(v[u][r].y), wa.z, blk);
            blk = fmaf(bf16_hi(v[u][r].y), wa.w, blk);
            blk = fmaf(bf16_lo(v[u][r].z), wb.x, blk);
            blk = fmaf(bf16_hi(v[u][r].z), wb.y, blk);
            blk = fmaf(bf16_lo(v[u][r].w), wb.z, blk);
            blk = fmaf(bf16_hi(v[u][r].w), wb.w, blk);
            acc[r] += (double)blk;
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
    // copy of the supplied scores: enough CTAs that each thread moves a few elements
    grid = (T + kRouterThreads * 4 - 1) / (kRouterThreads * 4);
    if (grid > sm_count()) grid = sm_count();
    if (grid < 1) grid = 1;
  } else {
    const int n_it = (d + 255) / 256;
    smem = (size_t)n_it * 256 * sizeof(float);
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
