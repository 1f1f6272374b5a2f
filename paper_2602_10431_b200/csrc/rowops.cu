// Bandwidth-bound row kernels: gather (+RMSNorm) of executed tokens (App. B.2),
// residual scatter (Eq. 3), fp32 RMSNorm, rotary embedding, SwiGLU, KV-cache
// append, embedding gather.  All move 16 bytes per thread per access, keep a
// row's data in registers between the reduction and the write, and read the
// executed-token count from device memory.
#include <string.h>

#include "rowops.cuh"

namespace qtale {

constexpr int kRowThreads = 256;

// ---- gather (+ RMSNorm) ------------------------------------------------------
// One CTA of 128 threads per executed row: the row (d <= 128 * 8 * MAXC bf16) stays in
// registers between the sum of squares and the write, a thread holds MAXC 16-byte chunks.
// Many small CTAs per SM keep loads, reductions and stores of different rows overlapped.
constexpr int kGatherThreads = 128;
template <int MAXC, int ACT>
__global__ void __launch_bounds__(kGatherThreads)
    compact_kernel(const uint4* __restrict__ x, const int32_t* __restrict__ idx,
                   const int32_t* __restrict__ n_exec, int cap, int d,
                   const float* __restrict__ gamma, float eps, uint4* __restrict__ xc,
                   uint4* __restrict__ hn, const GatherExtras ex) {
  __shared__ float s_part[2][kGatherThreads / 32];
  const int tid = threadIdx.x;
  const int n = n_exec ? min(*n_exec, cap) : cap;
  const int chunks = d >> 3;  // 16-byte chunks per row
  // Riding along (the kernel is bandwidth bound, its arithmetic units idle):
  //  * the rotary table of the executed tokens, cs[i][j] = (cos, sin)(pos[i] * base^(-2j/hd)) in
  //    fp64 arithmetic, read by the epilogue of the QKV projection;
  //  * zeroes in the value columns of the `tail_rows` rows that follow the executed count: the
  //    attention kernel loads key / value tiles that start at any executed row, so a tile can
  //    reach that far past the count; masked keys get probability 0, but 0 x NaN is NaN in the
  //    P V product, so those rows must be finite whatever the workspace held before.
  double inv_freq = 0.0;
  if (ex.cs && tid < ex.half) inv_freq = pow((double)ex.rope_base, -(double)tid / (double)ex.half);
  if (ex.tail) {
    const int end = min(cap, n + ex.tail_rows);
    const int cpr = ex.tail_cols >> 3;  // 16-byte chunks per row to clear
    const int total = max(end - n, 0) * cpr;
    for (int e = blockIdx.x * kGatherThreads + tid; e < total; e += gridDim.x * kGatherThreads) {
      const int r = e / cpr, c = e % cpr;
      ex.tail[(size_t)(n + r) * (ex.tail_ld >> 3) + (ex.tail_col0 >> 3) + c] = make_uint4(0, 0, 0, 0);
    }
  }
  int par = 0;
  // the index of a CTA's next row is fetched one row ahead, so a row's loads do not wait for it
  int row = (int)blockIdx.x < n ? idx[blockIdx.x] : 0;
  for (int i = blockIdx.x; i < n; i += gridDim.x, par ^= 1) {
    const uint4* src = x + (size_t)row * chunks;
    if (i + (int)gridDim.x < n) row = idx[i + gridDim.x];
    if (ex.cs && tid < ex.half) {
      double sn, cn;
      sincos((double)ex.pos[i] * inv_freq, &sn, &cn);
      ex.cs[(size_t)i * ex.half + tid] = make_float2((float)cn, (float)sn);
    }
    uint4 v[MAXC];
#pragma unroll
    for (int c = 0; c < MAXC; ++c) {
      const int cc = c * kGatherThreads + tid;
      if (cc < chunks) v[c] = ld_nc_16(src + cc);
    }
    if (xc) {
#pragma unroll
      for (int c = 0; c < MAXC; ++c) {
        const int cc = c * kGatherThreads + tid;
        if (cc < chunks) st_16(xc + (size_t)i * chunks + cc, v[c]);
      }
    }
    if (hn) {
      float ss = 0.f;
#pragma unroll
      for (int c = 0; c < MAXC; ++c) {
        const int cc = c * kGatherThreads + tid;
        if (cc < chunks) {
          const uint32_t u[4] = {v[c].x, v[c].y, v[c].z, v[c].w};
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const float a = bf16_lo(u[q]), b = bf16_hi(u[q]);
            ss = fmaf(a, a, ss);
            ss = fmaf(b, b, ss);
          }
        }
      }
      ss = warp_sum(ss);
      // partial sums alternate between two slots, so one barrier per row is enough
      if ((tid & 31) == 0) s_part[par][tid >> 5] = ss;
      __syncthreads();
      float tot = 0.f;
#pragma unroll
      for (int w = 0; w < kGatherThreads / 32; ++w) tot += s_part[par][w];
      const float inv = rsqrtf(tot / (float)d + eps);
#pragma unroll
      for (int c = 0; c < MAXC; ++c) {
        const int cc = c * kGatherThreads + tid;
        if (cc < chunks) {
          const float4 g0 = *reinterpret_cast<const float4*>(gamma + cc * 8);
          const float4 g1 = *reinterpret_cast<const float4*>(gamma + cc * 8 + 4);
          uint4 o;
          o.x = Act16<ACT>::pack(bf16_lo(v[c].x) * inv * g0.x, bf16_hi(v[c].x) * inv * g0.y);
          o.y = Act16<ACT>::pack(bf16_lo(v[c].y) * inv * g0.z, bf16_hi(v[c].y) * inv * g0.w);
          o.z = Act16<ACT>::pack(bf16_lo(v[c].z) * inv * g1.x, bf16_hi(v[c].z) * inv * g1.y);
          o.w = Act16<ACT>::pack(bf16_lo(v[c].w) * inv * g1.z, bf16_hi(v[c].w) * inv * g1.w);
          st_16(hn + (size_t)i * chunks + cc, o);
        }
      }
    }
  }
}

// ---- residual scatter: x[idx[i]] = bf16(float(xc[i]) + f[i]) -------------------
__global__ void __launch_bounds__(kRowThreads)
    scatter_add_kernel(uint4* __restrict__ x, const uint4* __restrict__ xc,
                       const float4* __restrict__ f, const int32_t* __restrict__ idx,
                       const int32_t* __restrict__ n_exec, int cap, int d) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  const int n = min(*n_exec, cap);
  const int chunks = d >> 3;
  for (int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; i < n; i += warps) {
    uint4* dst = x + (size_t)idx[i] * chunks;
    for (int cc = lane; cc < chunks; cc += 32) {
      const uint4 a = ld_nc_16(xc + (size_t)i * chunks + cc);
      const float4 f0 = f[((size_t)i * chunks + cc) * 2];
      const float4 f1 = f[((size_t)i * chunks + cc) * 2 + 1];
      uint4 o;
      o.x = pack_bf16x2(bf16_lo(a.x) + f0.x, bf16_hi(a.x) + f0.y);
      o.y = pack_bf16x2(bf16_lo(a.y) + f0.z, bf16_hi(a.y) + f0.w);
      o.z = pack_bf16x2(bf16_lo(a.z) + f1.x, bf16_hi(a.z) + f1.y);
      o.w = pack_bf16x2(bf16_lo(a.w) + f1.z, bf16_hi(a.w) + f1.w);
      st_16(dst + cc, o);
    }
  }
}

// ---- RMSNorm of an fp32 tensor into bf16: one CTA per row ---------------------
template <int MAXC, int ACT>
__global__ void __launch_bounds__(kRowThreads)
    rmsnorm_f32_kernel(const float4* __restrict__ u, const int32_t* __restrict__ n_rows, int cap,
                       int d, const float* __restrict__ gamma, float eps, uint2* __restrict__ out) {
  __shared__ float s_part[kRowThreads / 32];
  __shared__ float s_inv;
  const int n = n_rows ? min(*n_rows, cap) : cap;
  const int chunks = d >> 2;  // float4 chunks per row
  for (int i = blockIdx.x; i < n; i += gridDim.x) {
    float4 v[MAXC];
    float ss = 0.f;
#pragma unroll
    for (int c = 0; c < MAXC; ++c) {
      const int cc = c * kRowThreads + threadIdx.x;
      if (cc < chunks) {
        v[c] = u[(size_t)i * chunks + cc];
        ss = fmaf(v[c].x, v[c].x, ss);
        ss = fmaf(v[c].y, v[c].y, ss);
        ss = fmaf(v[c].z, v[c].z, ss);
        ss = fmaf(v[c].w, v[c].w, ss);
      }
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x < 32) {
      float t = threadIdx.x < kRowThreads / 32 ? s_part[threadIdx.x] : 0.f;
      t = warp_sum(t);
      if (threadIdx.x == 0) s_inv = rsqrtf(t / (float)d + eps);
    }
    __syncthreads();
    const float inv = s_inv;
#pragma unroll
    for (int c = 0; c < MAXC; ++c) {
      const int cc = c * kRowThreads + threadIdx.x;
      if (cc < chunks) {
        const float4 g = *reinterpret_cast<const float4*>(gamma + cc * 4);
        uint2 o;
        o.x = Act16<ACT>::pack(v[c].x * inv * g.x, v[c].y * inv * g.y);
        o.y = Act16<ACT>::pack(v[c].z * inv * g.z, v[c].w * inv * g.w);
        out[(size_t)i * chunks + cc] = o;
      }
    }
    __syncthreads();
  }
}

// ---- rotary embedding on the q and k heads of the fused qkv tensor -------------
// qkv: [n, ld] bf16; heads 0 .. n_rot-1 (q heads then k heads) are rotated in place,
// pairing element j with j + hd/2.  Only used when the QKV weights are in the plain row
// layout; with the rotary layout the rotation happens in the projection's epilogue.
template <int ACT>
__global__ void __launch_bounds__(kRowThreads)
    rope_kernel(uint4* __restrict__ qkv, const int32_t* __restrict__ n_exec, int cap, int ld,
                int n_rot, int hd, const float2* __restrict__ cs) {
  const int n = min(*n_exec, cap);
  const int half = hd >> 1;
  const int cpr = half >> 3;  // 16-byte chunks per half head
  const size_t per_row = (size_t)n_rot * cpr;
  const size_t total = (size_t)n * per_row;
  const int ldc = ld >> 3;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < total;
       e += (size_t)gridDim.x * blockDim.x) {
    const int i = (int)(e / per_row);
    const int r = (int)(e % per_row);
    const int h = r / cpr, c = r % cpr;
    uint4* p0 = qkv + (size_t)i * ldc + (size_t)h * (hd >> 3) + c;
    uint4* p1 = p0 + cpr;
    const uint4 a = *p0, b = *p1;
    const float4* t = reinterpret_cast<const float4*>(cs + (size_t)i * half + c * 8);
    const float4 t0 = t[0], t1 = t[1], t2 = t[2], t3 = t[3];  // (c,s) x 8
    const uint32_t au[4] = {a.x, a.y, a.z, a.w}, bu[4] = {b.x, b.y, b.z, b.w};
    const float cv[8] = {t0.x, t0.z, t1.x, t1.z, t2.x, t2.z, t3.x, t3.z};
    const float sv[8] = {t0.y, t0.w, t1.y, t1.w, t2.y, t2.w, t3.y, t3.w};
    uint32_t ao[4], bo[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float a0 = Act16<ACT>::lo(au[q]), a1 = Act16<ACT>::hi(au[q]);
      const float b0 = Act16<ACT>::lo(bu[q]), b1 = Act16<ACT>::hi(bu[q]);
      ao[q] = Act16<ACT>::pack(a0 * cv[2 * q] - b0 * sv[2 * q], a1 * cv[2 * q + 1] - b1 * sv[2 * q + 1]);
      bo[q] = Act16<ACT>::pack(b0 * cv[2 * q] + a0 * sv[2 * q], b1 * cv[2 * q + 1] + a1 * sv[2 * q + 1]);
    }
    *p0 = make_uint4(ao[0], ao[1], ao[2], ao[3]);
    *p1 = make_uint4(bo[0], bo[1], bo[2], bo[3]);
  }
}

// ---- SwiGLU: act[i, j] = silu(gu[i, j]) * gu[i, F + j] --------------------------
template <int ACT>
__global__ void __launch_bounds__(kRowThreads)
    swiglu_kernel(const uint4* __restrict__ gu, const int32_t* __restrict__ n_exec, int cap, int F,
                  uint4* __restrict__ act) {
  const int n = min(*n_exec, cap);
  const int fc = F >> 3;
  const size_t total = (size_t)n * fc;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < total;
       e += (size_t)gridDim.x * blockDim.x) {
    const size_t i = e / fc, c = e % fc;
    const uint4 g = ld_nc_16(gu + i * 2 * fc + c);
    const uint4 u = ld_nc_16(gu + i * 2 * fc + fc + c);
    const uint32_t gg[4] = {g.x, g.y, g.z, g.w}, uu[4] = {u.x, u.y, u.z, u.w};
    uint32_t o[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float g0 = Act16<ACT>::lo(gg[q]), g1 = Act16<ACT>::hi(gg[q]);
      o[q] = Act16<ACT>::pack(g0 / (1.f + __expf(-g0)) * Act16<ACT>::lo(uu[q]),
                              g1 / (1.f + __expf(-g1)) * Act16<ACT>::hi(uu[q]));
    }
    st_16(act + e, make_uint4(o[0], o[1], o[2], o[3]));
  }
}

// ---- KV-cache append of the executed tokens' K (rotated) and V ------------------
__global__ void __launch_bounds__(kRowThreads)
    kv_append_kernel(const uint4* __restrict__ qkv, const int32_t* __restrict__ n_exec, int cap_rows,
                     int ld, int q_dim, int kv_dim, int hd, const int32_t* __restrict__ cu_exec, int B,
                     uint4* __restrict__ cache_k, uint4* __restrict__ cache_v,
                     const int32_t* __restrict__ kv_len, int cap) {
  const int n = min(*n_exec, cap_rows);
  const int kc = kv_dim >> 3;
  const int ldc = ld >> 3;
  const size_t total = (size_t)n * kc;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < total;
       e += (size_t)gridDim.x * blockDim.x) {
    const int i = (int)(e / kc), c = (int)(e % kc);
    int lo = 0, hi = B;  // sequence of executed token i: cu_exec[lo] <= i < cu_exec[hi]
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (cu_exec[mid] <= i) lo = mid; else hi = mid;
    }
    const int slot = kv_len[lo] + (i - cu_exec[lo]);
    if (slot >= cap) continue;  // cache full: kv_len_update_kernel records QTALE_ERR_CAPACITY
    // cache layout [B, Hkv, cap, hd]
    const int hc = hd >> 3, head = c / hc, within = c % hc;
    const size_t dst = (((size_t)lo * (kv_dim / hd) + head) * cap + slot) * hc + within;
    cache_k[dst] = qkv[(size_t)i * ldc + (q_dim >> 3) + c];
    cache_v[dst] = qkv[(size_t)i * ldc + ((q_dim + kv_dim) >> 3) + c];
  }
}

// The lengths live on the device, so a full cache can only be detected here: the rows that did
// not fit are dropped, the length stays at the capacity and the status word reports it.
__global__ void kv_len_update_kernel(int32_t* kv_len, const int32_t* cu_exec, int B, int cap,
                                     int* status) {
  for (int b = blockIdx.x * blockDim.x + threadIdx.x; b < B; b += gridDim.x * blockDim.x) {
    const int want = kv_len[b] + cu_exec[b + 1] - cu_exec[b];
    if (want > cap) report_device_error(status, QTALE_ERR_CAPACITY);
    kv_len[b] = min(cap, want);
  }
}

// ---- embedding gather ------------------------------------------------------------
__global__ void __launch_bounds__(kRowThreads)
    embed_kernel(const uint4* __restrict__ embed, const int32_t* __restrict__ ids, int T, int d,
                 int vocab, uint4* __restrict__ out) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  const int chunks = d >> 3;
  for (int t = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; t < T; t += warps) {
    int id = ids[t];
    id = id < 0 ? 0 : (id >= vocab ? vocab - 1 : id);
    for (int cc = lane; cc < chunks; cc += 32)
      st_16(out + (size_t)t * chunks + cc, ld_nc_16(embed + (size_t)id * chunks + cc));
  }
}

// ---- decode-loop helpers ------------------------------------------------------------
// cu[b] = b for b = 0 .. B: one new token per sequence
__global__ void iota_kernel(int32_t* __restrict__ cu, int n) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) cu[i] = i;
}
// the next token of a sequence sits one position further (finished sequences stay where they are)
__global__ void advance_pos_kernel(int32_t* __restrict__ pos, const uint8_t* __restrict__ valid, int B) {
  for (int b = blockIdx.x * blockDim.x + threadIdx.x; b < B; b += gridDim.x * blockDim.x)
    if (!valid || valid[b]) pos[b] += 1;
}
// greedy choice: index of the largest logit of each row, the lowest index among equal ones
__global__ void __launch_bounds__(kRowThreads)
    argmax_rows_kernel(const float* __restrict__ logits, int V, int32_t* __restrict__ out) {
  __shared__ float s_v[kRowThreads / 32];
  __shared__ int s_i[kRowThreads / 32];
  const float* row = logits + (size_t)blockIdx.x * V;
  float best = -INFINITY;
  int bi = 0x7FFFFFFF;
  for (int j = threadIdx.x; j < V; j += kRowThreads) {
    const float v = row[j];
    if (v > best || (v == best && j < bi)) { best = v; bi = j; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, best, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
  }
  if ((threadIdx.x & 31) == 0) { s_v[threadIdx.x >> 5] = best; s_i[threadIdx.x >> 5] = bi; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < kRowThreads / 32; ++w)
      if (s_v[w] > best || (s_v[w] == best && s_i[w] < bi)) { best = s_v[w]; bi = s_i[w]; }
    out[blockIdx.x] = bi == 0x7FFFFFFF ? 0 : bi;
  }
}

// ---- host launchers ----------------------------------------------------------------

static int row_grid(int per_sm) { return sm_count() * per_sm; }

template <int ACT>
static int launch_compact_t(const void* x, const int32_t* idx, const int32_t* n_exec, int cap,
                            int d, const float* gamma, float eps, void* xc, void* hn,
                            const GatherExtras& ex, cudaStream_t s) {
  const int chunks = d / 8;
  const int grid = min(cap, row_grid(16));
  auto X = static_cast<const uint4*>(x);
  auto XC = static_cast<uint4*>(xc);
  auto HN = static_cast<uint4*>(hn);
#define QTALE_COMPACT(C)                                                                         \
  compact_kernel<C, ACT><<<grid, kGatherThreads, 0, s>>>(X, idx, n_exec, cap, d, gamma, eps, XC, HN, ex)
  if (chunks <= kGatherThreads * 1) QTALE_COMPACT(1);
  else if (chunks <= kGatherThreads * 2) QTALE_COMPACT(2);
  else if (chunks <= kGatherThreads * 4) QTALE_COMPACT(4);
  else if (chunks <= kGatherThreads * 5) QTALE_COMPACT(5);
  else if (chunks <= kGatherThreads * 8) QTALE_COMPACT(8);
  else if (chunks <= kGatherThreads * 16) QTALE_COMPACT(16);
  else return QTALE_ERR_SHAPE;
#undef QTALE_COMPACT
  return launch_status(cudaGetLastError());
}

int launch_compact(const void* x, const int32_t* idx, const int32_t* n_exec, int cap, int d,
                   const float* gamma, float eps, int act, void* xc, void* hn, cudaStream_t s,
                   const GatherExtras* extras) {
  GatherExtras ex;
  memset(&ex, 0, sizeof(ex));
  if (extras) ex = *extras;
  if (ex.cs && (ex.half > kGatherThreads || ex.half < 1)) return QTALE_ERR_SHAPE;
  return act == QTALE_ACT_F16 ? launch_compact_t<1>(x, idx, n_exec, cap, d, gamma, eps, xc, hn, ex, s)
                              : launch_compact_t<0>(x, idx, n_exec, cap, d, gamma, eps, xc, hn, ex, s);
}

int launch_scatter_add(void* x, const void* xc, const float* f, const int32_t* idx,
                       const int32_t* n_exec, int cap, int d, cudaStream_t s) {
  scatter_add_kernel<<<row_grid(8), kRowThreads, 0, s>>>(
      static_cast<uint4*>(x), static_cast<const uint4*>(xc), reinterpret_cast<const float4*>(f),
      idx, n_exec, cap, d);
  return launch_status(cudaGetLastError());
}

template <int ACT>
static int launch_rmsnorm_f32_t(const float* u, const int32_t* n_rows, int cap, int d,
                                const float* gamma, float eps, void* out, cudaStream_t s) {
  const int chunks = d / 4;
  const int grid = min(cap, row_grid(8));
  auto U = reinterpret_cast<const float4*>(u);
  auto O = static_cast<uint2*>(out);
  if (chunks <= kRowThreads * 1)
    rmsnorm_f32_kernel<1, ACT><<<grid, kRowThreads, 0, s>>>(U, n_rows, cap, d, gamma, eps, O);
  else if (chunks <= kRowThreads * 4)
    rmsnorm_f32_kernel<4, ACT><<<grid, kRowThreads, 0, s>>>(U, n_rows, cap, d, gamma, eps, O);
  else if (chunks <= kRowThreads * 8)
    rmsnorm_f32_kernel<8, ACT><<<grid, kRowThreads, 0, s>>>(U, n_rows, cap, d, gamma, eps, O);
  else
    return QTALE_ERR_SHAPE;
  return launch_status(cudaGetLastError());
}

int launch_rmsnorm_f32(const float* u, const int32_t* n_rows, int cap, int d, const float* gamma,
                       float eps, int act, void* out, cudaStream_t s) {
  return act == QTALE_ACT_F16 ? launch_rmsnorm_f32_t<1>(u, n_rows, cap, d, gamma, eps, out, s)
                              : launch_rmsnorm_f32_t<0>(u, n_rows, cap, d, gamma, eps, out, s);
}

int launch_rope(void* qkv, const int32_t* n_exec, int cap, int ld, int n_rot, int hd,
                const float* cs, int act, cudaStream_t s) {
  if (act == QTALE_ACT_F16)
    rope_kernel<1><<<row_grid(8), kRowThreads, 0, s>>>(static_cast<uint4*>(qkv), n_exec, cap, ld,
                                                       n_rot, hd, reinterpret_cast<const float2*>(cs));
  else
    rope_kernel<0><<<row_grid(8), kRowThreads, 0, s>>>(static_cast<uint4*>(qkv), n_exec, cap, ld,
                                                       n_rot, hd, reinterpret_cast<const float2*>(cs));
  return launch_status(cudaGetLastError());
}

int launch_swiglu(const void* gu, const int32_t* n_exec, int cap, int F, void* act, int act_dtype,
                  cudaStream_t s) {
  if (act_dtype == QTALE_ACT_F16)
    swiglu_kernel<1><<<row_grid(8), kRowThreads, 0, s>>>(static_cast<const uint4*>(gu), n_exec, cap,
                                                         F, static_cast<uint4*>(act));
  else
    swiglu_kernel<0><<<row_grid(8), kRowThreads, 0, s>>>(static_cast<const uint4*>(gu), n_exec, cap,
                                                         F, static_cast<uint4*>(act));
  return launch_status(cudaGetLastError());
}

int launch_kv_append(const void* qkv, const int32_t* n_exec, int cap_rows, int ld, int q_dim,
                     int kv_dim, int hd, const int32_t* cu_exec, int B, void* cache_k, void* cache_v,
                     int32_t* kv_len, int cap, cudaStream_t s) {
  kv_append_kernel<<<row_grid(4), kRowThreads, 0, s>>>(
      static_cast<const uint4*>(qkv), n_exec, cap_rows, ld, q_dim, kv_dim, hd, cu_exec, B,
      static_cast<uint4*>(cache_k), static_cast<uint4*>(cache_v), kv_len, cap);
  if (cudaGetLastError() != cudaSuccess) return QTALE_ERR_CUDA;
  kv_len_update_kernel<<<(B + 255) / 256, 256, 0, s>>>(kv_len, cu_exec, B, cap, device_status_ptr());
  return launch_status(cudaGetLastError());
}

int launch_iota(int32_t* cu, int n, cudaStream_t s) {
  iota_kernel<<<(n + 255) / 256, 256, 0, s>>>(cu, n);
  return launch_status(cudaGetLastError());
}

int launch_advance_pos(int32_t* pos, const uint8_t* valid, int B, cudaStream_t s) {
  advance_pos_kernel<<<(B + 255) / 256, 256, 0, s>>>(pos, valid, B);
  return launch_status(cudaGetLastError());
}

int launch_argmax_rows(const float* logits, int rows, int V, int32_t* out, cudaStream_t s) {
  argmax_rows_kernel<<<rows, kRowThreads, 0, s>>>(logits, V, out);
  return launch_status(cudaGetLastError());
}

int launch_embed(const void* embed, const int32_t* ids, int T, int d, int vocab, void* out,
                 cudaStream_t s) {
  embed_kernel<<<row_grid(8), kRowThreads, 0, s>>>(static_cast<const uint4*>(embed), ids, T, d,
                                                   vocab, static_cast<uint4*>(out));
  return launch_status(cudaGetLastError());
}

}  // namespace qtale

using namespace qtale;

extern "C" {

int qtale_compact(const void* x, const int32_t* idx, const int32_t* n_exec, int T, int d,
                  const float* rms_gamma, float eps, int act_dtype, void* xc_out, void* hn_out,
                  void* stream) {
  if (act_dtype != QTALE_ACT_BF16 && act_dtype != QTALE_ACT_F16) return QTALE_ERR_MODE;
  if (!x || !idx || !n_exec) return QTALE_ERR_NULL;
  if (!xc_out && !hn_out) return QTALE_ERR_NULL;
  if (hn_out && !rms_gamma) return QTALE_ERR_NULL;
  if (T < 1 || d < 8 || d % 8 != 0) return QTALE_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(xc_out) || !aligned16(hn_out) || !aligned16(rms_gamma))
    return QTALE_ERR_ALIGN;
  return launch_compact(x, idx, n_exec, T, d, rms_gamma, eps, act_dtype, xc_out, hn_out,
                        static_cast<cudaStream_t>(stream));
}

int qtale_scatter_add(void* x_inout, const void* xc, const float* f, const int32_t* idx,
                      const int32_t* n_exec, int T, int d, void* stream) {
  if (!x_inout || !xc || !f || !idx || !n_exec) return QTALE_ERR_NULL;
  if (T < 1 || d < 8 || d % 8 != 0) return QTALE_ERR_SHAPE;
  if (!aligned16(x_inout) || !aligned16(xc) || !aligned16(f)) return QTALE_ERR_ALIGN;
  return launch_scatter_add(x_inout, xc, f, idx, n_exec, T, d, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
