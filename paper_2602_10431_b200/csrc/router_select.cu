// Router score + execute decision + ordered compaction (Eq. 2, Eq. 9; App. B.2).
//
// One launch.  Phase A (all CTAs): z_t = w . x_t + b accumulated in fp64 over a
// bandwidth-bound sweep of x, p_t = 1 / (1 + exp(-z_t)) stored as fp32.  Phase
// B (the CTA that finishes last, found with a ticket counter): threshold or
// top-k decision on the fp32 scores and an ordered prefix-sum compaction into
// the ascending index list, the per-sequence offsets and the positions.
#include "router_select.cuh"

namespace qtale {

constexpr int kRouterThreads = 512;  // 16 warps
constexpr int kRowsPerWarp = 2;

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
  int* status;
  int T, d, B, mode, k;  // k < 0 (top-k): k = floor(ratio * valid tokens + 0.5), counted here
  double ratio;
  float bias, theta;
};

__device__ __forceinline__ uint32_t score_key(float s) {
  uint32_t b = __float_as_uint(s);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// ---- phase B: decision + compaction, executed by one CTA ----------------------
// Every sweep over the scores is warp-cooperative and coalesced: warp w owns the
// contiguous token segment [w * seg, (w + 1) * seg) and walks it 32 tokens at a
// time (token = segment start + 32 i + lane), so ballots give each selected
// token its rank in token order.  When a lane's share is at most kKeep scores
// they are read once and kept in registers for all sweeps.
constexpr int kKeep = 16;

__device__ void select_and_compact(const RouterParams& p, uint32_t* sh_hist, int* sh_scan) {
  const int tid = threadIdx.x;
  const int nthr = blockDim.x;
  const int lane = tid & 31, wid = tid >> 5, nwarps = nthr >> 5;
  const int T = p.T;
  __shared__ uint32_t s_prefix, s_mask;
  __shared__ int s_remaining, s_n_valid;

  // cu_seqlens must be 0 = cu[0] <= cu[1] <= ... <= cu[B] = T.  Anything else is reported in the
  // status word; tokens outside [cu[0], cu[B]) then never execute and every walk below stays
  // inside the B + 1 entries.
  const int t_begin = min(max(__ldg(p.cu_seqlens), 0), T);
  const int t_end = min(max(__ldg(p.cu_seqlens + p.B), t_begin), T);
  {
    bool bad = tid == 0 && (__ldg(p.cu_seqlens) != 0 || __ldg(p.cu_seqlens + p.B) != T);
    for (int q = tid; q < p.B; q += nthr) bad |= __ldg(p.cu_seqlens + q) > __ldg(p.cu_seqlens + q + 1);
    if (bad) report_device_error(p.status, QTALE_ERR_SHAPE);
  }

  const int seg = ((T + nwarps - 1) / nwarps + 31) & ~31;  // tokens per warp, multiple of 32
  const int w0 = min(T, wid * seg), w1 = min(T, w0 + seg);
  const int n_it = (w1 - w0 + 31) >> 5;                    // 32-token steps of this warp
  const bool keep = seg <= 32 * kKeep;                     // uniform over the CTA

  // score and validity of the token of step i (0 and false past the end)
  auto load_one = [&](int i, float& sc, bool& ok) {
    const int t = w0 + 32 * i + lane;
    ok = t < w1 && t >= t_begin && t < t_end;
    sc = 0.f;
    if (ok) {
      sc = __ldcg(p.scores + t);
      if (p.valid) ok = p.valid[t] != 0;
    }
  };
  float ksc[kKeep];
  uint32_t kok = 0;  // bit i: token of step i is valid
  if (keep) {
#pragma unroll
    for (int i = 0; i < kKeep; ++i) {
      bool ok;
      load_one(i, ksc[i], ok);
      kok |= (ok ? 1u : 0u) << i;
    }
  }

  uint32_t tau = 0;  // key of the k-th largest score (top-k)
  int need_eq = 0;   // how many tokens with key == tau execute (lowest indices first)

  int k_sel = p.k;
  if (p.mode == QTALE_SELECT_TOPK && p.k < 0) {
    // k for a requested ratio of the valid tokens (padding does not count)
    if (tid == 0) s_n_valid = 0;
    __syncthreads();
    int nv = 0;
    if (keep) {
      nv = __popc(kok);
    } else {
      for (int i = 0; i < n_it; ++i) {
        float sc;
        bool ok;
        load_one(i, sc, ok);
        nv += ok ? 1 : 0;
      }
    }
    nv = __reduce_add_sync(0xffffffffu, nv);
    if (lane == 0) atomicAdd(&s_n_valid, nv);
    __syncthreads();
    const int n_valid = s_n_valid;
    double kd = floor(p.ratio * (double)n_valid + 0.5);
    kd = kd < 0.0 ? 0.0 : (kd > (double)n_valid ? (double)n_valid : kd);
    k_sel = (int)kd;
  }

  if (p.mode == QTALE_SELECT_TOPK && k_sel > 0) {
    // MSB-first radix select (four 8-bit digits) of the k-th largest key among valid tokens
    if (tid == 0) {
      s_prefix = 0;
      s_mask = 0;
      s_remaining = k_sel;
    }
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      for (int i = tid; i < 256; i += nthr) sh_hist[i] = 0;
      __syncthreads();
      const uint32_t prefix = s_prefix, mask = s_mask;
      auto count_key = [&](float sc, bool ok) {
        const uint32_t key = score_key(sc);
        const bool in = ok && (key & mask) == prefix;
        const uint32_t bucket = (key >> shift) & 0xFFu;
        // scores cluster in few buckets of the leading digits: one atomic when the warp agrees
        const uint32_t members = __ballot_sync(0xffffffffu, in);
        if (members == 0) return;
        const int first = __ffs(members) - 1;
        const uint32_t b0 = __shfl_sync(0xffffffffu, bucket, first);
        if (__all_sync(0xffffffffu, !in || bucket == b0)) {
          if (lane == first) atomicAdd(&sh_hist[b0], (uint32_t)__popc(members));
        } else if (in) {
          atomicAdd(&sh_hist[bucket], 1u);
        }
      };
      if (keep) {
#pragma unroll
        for (int i = 0; i < kKeep; ++i) count_key(ksc[i], (kok >> i) & 1u);
      } else {
        for (int i0 = 0; i0 < n_it; i0 += 8) {
          float sc[8];
          bool ok[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) load_one(i0 + j, sc[j], ok[j]);
#pragma unroll
          for (int j = 0; j < 8; ++j) count_key(sc[j], ok[j]);
        }
      }
      __syncthreads();
      // bucket holding the target rank: warp 0 scans the 256 counts from the top, 8 per lane
      if (wid == 0) {
        int c[8], sum = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          c[j] = (int)sh_hist[255 - (lane * 8 + j)];
          sum += c[j];
        }
        int inc = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int n = __shfl_up_sync(0xffffffffu, inc, o);
          if (lane >= o) inc += n;
        }
        const int rem = s_remaining;
        int before = inc - sum;  // keys in buckets above this lane's eight
        int found = -1, new_rem = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (found < 0 && before + c[j] >= rem && before < rem) {
            found = 255 - (lane * 8 + j);
            new_rem = rem - before;
          }
          before += c[j];
        }
        const uint32_t owner = __ballot_sync(0xffffffffu, found >= 0);
        if (owner == 0) {
          // k exceeds the number of valid tokens: everything valid executes (lowest bucket)
          if (lane == 0) {
            s_prefix = prefix;
            s_mask = mask | (0xFFu << shift);
          }
        } else if (lane == __ffs(owner) - 1) {
          s_remaining = new_rem;  // rank of the target inside the bucket (1-based)
          s_prefix = prefix | ((uint32_t)found << shift);
          s_mask = mask | (0xFFu << shift);
        }
      }
      __syncthreads();
    }
    tau = s_prefix;
    need_eq = s_remaining;
  }

  const bool topk = p.mode == QTALE_SELECT_TOPK;
  const bool none = topk && k_sel <= 0;
  // (executes for sure, executes if among the first need_eq equal keys)
  auto classify = [&](float sc, bool ok, bool& sure, bool& eq) {
    if (topk) {
      const uint32_t key = score_key(sc);
      sure = ok && !none && key > tau;
      eq = ok && !none && key == tau;
    } else {
      sure = ok && sc >= p.theta;
      eq = false;
    }
  };

  // sweep 1: executed tokens and tied tokens of each warp's segment
  int n_sure = 0, n_eq = 0;
  if (keep) {
#pragma unroll
    for (int i = 0; i < kKeep; ++i) {
      bool sure, eq;
      classify(ksc[i], (kok >> i) & 1u, sure, eq);
      n_sure += __popc(__ballot_sync(0xffffffffu, sure));
      n_eq += __popc(__ballot_sync(0xffffffffu, eq));
    }
  } else {
    for (int i0 = 0; i0 < n_it; i0 += 8) {
      float sc[8];
      bool ok[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) load_one(i0 + j, sc[j], ok[j]);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        bool sure, eq;
        classify(sc[j], ok[j], sure, eq);
        n_sure += __popc(__ballot_sync(0xffffffffu, sure));
        n_eq += __popc(__ballot_sync(0xffffffffu, eq));
      }
    }
  }
  // exclusive scans over the warps (at most 32 of them): sh_scan[0..31] sure, [32..63] tied
  if (lane == 0) {
    sh_scan[wid] = n_sure;
    sh_scan[32 + wid] = n_eq;
  }
  __syncthreads();
  int eq_before = 0, sure_before = 0, tot_eq = 0, tot_sure = 0;
  for (int w = 0; w < nwarps; ++w) {
    const int a = sh_scan[w], b = sh_scan[32 + w];
    if (w < wid) {
      sure_before += a;
      eq_before += b;
    }
    tot_sure += a;
    tot_eq += b;
  }
  const int total = tot_sure + min(tot_eq, need_eq);
  int out = sure_before + min(eq_before, need_eq);

  // sweep 2: ordered write of idx / pos, and cu_exec at every sequence start.
  // b = sequence holding the lane's current token (largest b with cu_seqlens[b] <= t).
  int b = 0;
  {
    const int t = min(w0 + lane, T - 1);
    int lo = 0, hi = p.B;  // cu[lo] <= t < cu[hi]
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (__ldg(p.cu_seqlens + mid) <= t) lo = mid; else hi = mid;
    }
    b = lo;
  }
  int seq_start = __ldg(p.cu_seqlens + b), seq_end = __ldg(p.cu_seqlens + b + 1);
  const uint32_t lt = (1u << lane) - 1u;
  auto emit = [&](int i, float sc, bool ok) {
    const int t = w0 + 32 * i + lane;
    bool sure, eq;
    classify(sc, ok, sure, eq);
    const uint32_t m_eq = __ballot_sync(0xffffffffu, eq);
    const bool take = sure || (eq && eq_before + __popc(m_eq & lt) < need_eq);
    const uint32_t m_take = __ballot_sync(0xffffffffu, take);
    const int my_out = out + __popc(m_take & lt);
    if (t < w1) {
      while (t >= seq_end && b + 1 < p.B) {  // move to the sequence holding t (skips empty ones)
        ++b;
        seq_start = seq_end;
        seq_end = __ldg(p.cu_seqlens + b + 1);
      }
      if (t == seq_start) {  // first token of sequence b and of the empty sequences before it
        for (int q = b; q >= 0 && __ldg(p.cu_seqlens + q) == t; --q) p.cu_exec[q] = my_out;
      }
      if (take) {
        p.idx[my_out] = t;
        p.pos[my_out] = t - seq_start + (p.pos0 ? __ldg(p.pos0 + b) : 0);
      }
    }
    out += __popc(m_take);
    eq_before += __popc(m_eq);
  };
  if (keep) {
#pragma unroll
    for (int i = 0; i < kKeep; ++i) emit(i, ksc[i], (kok >> i) & 1u);
  } else {
    for (int i0 = 0; i0 < n_it; i0 += 8) {
      float sc[8];
      bool ok[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) load_one(i0 + j, sc[j], ok[j]);
#pragma unroll
      for (int j = 0; j < 8; ++j) emit(i0 + j, sc[j], ok[j]);
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
  return router_select_launch(x, T, d, w_router, bias, scores_override, valid, cu_seqlens, B, pos0,
                              mode, theta, k, -1.0, scores_out, idx_out, n_exec_out, cu_exec_out,
                              pos_out, ws, ws_bytes, static_cast<cudaStream_t>(stream));
}

}  // extern "C"

namespace qtale {

int router_select_launch(const void* x, int T, int d, const float* w_router, float bias,
                         const float* scores_override, const uint8_t* valid,
                         const int32_t* cu_seqlens, int B, const int32_t* pos0, int mode,
                         float theta, int k, double ratio, float* scores_out, int32_t* idx_out,
                         int32_t* n_exec_out, int32_t* cu_exec_out, int32_t* pos_out, void* ws,
                         size_t ws_bytes, cudaStream_t s) {
  if (!scores_out || !idx_out || !n_exec_out || !cu_exec_out || !pos_out || !cu_seqlens || !ws)
    return QTALE_ERR_NULL;
  if (!scores_override && (!x || !w_router)) return QTALE_ERR_NULL;
  if (T < 1 || T > (1 << 24) || B < 1 || B > T) return QTALE_ERR_SHAPE;
  if (!scores_override && (d < 8 || d % 8 != 0 || d > 16384)) return QTALE_ERR_SHAPE;
  if (mode != QTALE_SELECT_THRESHOLD && mode != QTALE_SELECT_TOPK) return QTALE_ERR_MODE;
  if (mode == QTALE_SELECT_TOPK && ratio < 0.0 && (k < 0 || k > T)) return QTALE_ERR_CAPACITY;
  if (!aligned16(x) || !aligned16(ws)) return QTALE_ERR_ALIGN;
  if (ws_bytes < qtale_router_select_workspace_bytes(T)) return QTALE_ERR_WORKSPACE;

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
  p.status = device_status_ptr();
  p.T = T; p.d = d; p.B = B; p.mode = mode;
  p.k = (mode == QTALE_SELECT_TOPK && ratio >= 0.0) ? -1 : k;
  p.ratio = ratio;
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

}  // namespace qtale

extern "C" {

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
