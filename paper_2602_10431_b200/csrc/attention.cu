// Attention over the executed tokens only (Eq. 3: a bypassed token never
// evaluates f_l, so it has no query, key or value at this layer).
//
// Decode (the prefill kernel lives in attention_tc.cu): one query per executed sequence against that sequence's cache of
// executed-token keys / values (bandwidth bound: half a warp per key row).
#include "attention.cuh"

namespace qtale {

// ---------------------------------------------------------------------------
// decode: one new token per executed sequence, keys / values from the cache
// ---------------------------------------------------------------------------
constexpr int kDecThreads = 128;

template <int HD, int REP, int ACT>
__global__ void __launch_bounds__(kDecThreads)
    attn_decode_kernel(const __nv_bfloat16* __restrict__ qkv, int ld,
                       const int32_t* __restrict__ idx, const int32_t* __restrict__ n_exec,
                       const __nv_bfloat16* __restrict__ cache_k,
                       const __nv_bfloat16* __restrict__ cache_v,
                       const int32_t* __restrict__ kv_len, int cap, int Hkv,
                       __nv_bfloat16* __restrict__ out, int ldo, float scale_log2) {
  constexpr int LPK = HD / 8;            // lanes per key row (16 bytes each)
  constexpr int KPW = 32 / LPK;          // keys per warp step
  constexpr int GROUPS = (kDecThreads / 32) * KPW;
  __shared__ float s_m[GROUPS][REP], s_l[GROUPS][REP];
  __shared__ float s_acc[GROUPS][REP][HD];

  const int i = blockIdx.x;  // executed sequence slot
  if (i >= *n_exec) return;
  const int hk = blockIdx.y;
  const int b = idx[i];
  const int n_keys = min(kv_len[b], cap);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int sub = lane % LPK;            // which 8 columns of the head
  const int grp = warp * KPW + lane / LPK;

  float q[REP][8];
#pragma unroll
  for (int r = 0; r < REP; ++r) {
    const uint4 v = *reinterpret_cast<const uint4*>(qkv + (size_t)i * ld + (size_t)(hk * REP + r) * HD + sub * 8);
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      q[r][2 * e] = Act16<ACT>::lo(u[e]) * scale_log2;
      q[r][2 * e + 1] = Act16<ACT>::hi(u[e]) * scale_log2;
    }
  }
  float m[REP], l[REP], acc[REP][8];
#pragma unroll
  for (int r = 0; r < REP; ++r) {
    m[r] = -INFINITY; l[r] = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[r][e] = 0.f;
  }
  // cache layout [B, Hkv, cap, HD]: the keys of this (sequence, head) are one contiguous stream
  const size_t row_stride = HD;
  const __nv_bfloat16* kb = cache_k + (((size_t)b * Hkv + hk) * cap) * HD + sub * 8;
  const __nv_bfloat16* vb = cache_v + (((size_t)b * Hkv + hk) * cap) * HD + sub * 8;
  constexpr int UNROLL = 4;
  // the trip count is the same for every lane (the shuffles below name the whole warp); keys
  // past the end are masked by `ok`
  for (int kbase = 0; kbase < n_keys; kbase += GROUPS * UNROLL) {
    const int k0 = kbase + grp;
    uint4 kv[UNROLL], vv[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const int key = k0 + u * GROUPS;
      if (key < n_keys) {
        kv[u] = ld_nc_16(kb + (size_t)key * row_stride);
        vv[u] = ld_nc_16(vb + (size_t)key * row_stride);
      } else {
        kv[u] = make_uint4(0, 0, 0, 0);
        vv[u] = make_uint4(0, 0, 0, 0);
      }
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const int key = k0 + u * GROUPS;
      const bool ok = key < n_keys;  // uniform inside a key group
      const uint32_t ku[4] = {kv[u].x, kv[u].y, kv[u].z, kv[u].w};
      const uint32_t vu[4] = {vv[u].x, vv[u].y, vv[u].z, vv[u].w};
      float kf[8], vf[8];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        kf[2 * e] = ok ? Act16<ACT>::lo(ku[e]) : 0.f; kf[2 * e + 1] = ok ? Act16<ACT>::hi(ku[e]) : 0.f;
        vf[2 * e] = ok ? Act16<ACT>::lo(vu[e]) : 0.f; vf[2 * e + 1] = ok ? Act16<ACT>::hi(vu[e]) : 0.f;
      }
#pragma unroll
      for (int r = 0; r < REP; ++r) {
        float sc = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) sc = fmaf(q[r][e], kf[e], sc);
#pragma unroll
        for (int off = LPK / 2; off > 0; off >>= 1) sc += __shfl_xor_sync(0xffffffffu, sc, off);
        if (ok) {
          const float mn = fmaxf(m[r], sc);
          const float corr = exp2f(m[r] - mn);
          const float p = exp2f(sc - mn);
          m[r] = mn;
          l[r] = l[r] * corr + p;
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[r][e] = fmaf(p, vf[e], acc[r][e] * corr);
        }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < REP; ++r) {
    if (sub == 0) { s_m[grp][r] = m[r]; s_l[grp][r] = l[r]; }
#pragma unroll
    for (int e = 0; e < 8; ++e) s_acc[grp][r][sub * 8 + e] = acc[r][e];
  }
  __syncthreads();
  for (int e = threadIdx.x; e < REP * HD; e += kDecThreads) {
    const int r = e / HD, c = e % HD;
    float mx = -INFINITY;
    for (int gI = 0; gI < GROUPS; ++gI) mx = fmaxf(mx, s_m[gI][r]);
    float num = 0.f, den = 0.f;
    for (int gI = 0; gI < GROUPS; ++gI) {
      const float w = (s_m[gI][r] == -INFINITY) ? 0.f : exp2f(s_m[gI][r] - mx);
      num += w * s_acc[gI][r][c];
      den += w * s_l[gI][r];
    }
    reinterpret_cast<unsigned short*>(out)[(size_t)i * ldo + (size_t)(hk * REP + r) * HD + c] =
        Act16<ACT>::one(den > 0.f ? num / den : 0.f);
  }
}

// ---------------------------------------------------------------------------
// host launchers
// ---------------------------------------------------------------------------
template <int HD, int ACT>
static int launch_decode_hd(const void* qkv, int ld, int H, int Hkv, const int32_t* idx,
                            const int32_t* n_exec, int B_cap, const void* ck, const void* cv,
                            const int32_t* kv_len, int cap, void* out, int ldo, cudaStream_t s) {
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)HD);
  dim3 grid(B_cap, Hkv);
  auto Q = static_cast<const __nv_bfloat16*>(qkv);
  auto K = static_cast<const __nv_bfloat16*>(ck);
  auto V = static_cast<const __nv_bfloat16*>(cv);
  auto O = static_cast<__nv_bfloat16*>(out);
  const int rep = H / Hkv;
#define QTALE_DEC(R)                                                                              \
  attn_decode_kernel<HD, R, ACT><<<grid, kDecThreads, 0, s>>>(Q, ld, idx, n_exec, K, V, kv_len, cap,   \
                                                         Hkv, O, ldo, scale_log2)
  if (rep == 1) QTALE_DEC(1);
  else if (rep == 2) QTALE_DEC(2);
  else if (rep == 4) QTALE_DEC(4);
  else if (rep == 8) QTALE_DEC(8);
  else return QTALE_ERR_SHAPE;
#undef QTALE_DEC
  return launch_status(cudaGetLastError());
}

int launch_attn_decode(const void* qkv, int ld, int H, int Hkv, int hd, int act, const int32_t* idx,
                       const int32_t* n_exec, int B_cap, const void* cache_k, const void* cache_v,
                       const int32_t* kv_len, int cap, void* out, int ldo, cudaStream_t s) {
#define QTALE_DC(HD_, ACT_)                                                                       \
  launch_decode_hd<HD_, ACT_>(qkv, ld, H, Hkv, idx, n_exec, B_cap, cache_k, cache_v, kv_len, cap, \
                              out, ldo, s)
  if (hd == 128) return act == QTALE_ACT_F16 ? QTALE_DC(128, 1) : QTALE_DC(128, 0);
  if (hd == 64) return act == QTALE_ACT_F16 ? QTALE_DC(64, 1) : QTALE_DC(64, 0);
#undef QTALE_DC
  return QTALE_ERR_SHAPE;
}

}  // namespace qtale
