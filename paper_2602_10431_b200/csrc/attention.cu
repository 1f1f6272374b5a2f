// Attention over the executed tokens only (Eq. 3: a bypassed token never
// evaluates f_l, so it has no query, key or value at this layer).
//
// Prefill: executed tokens of a sequence are contiguous and in ascending
// position order in the compact tensor, so causal attention among them is
// ordinary variable-length causal attention over the per-sequence executed
// counts (cu_exec, read on the device).  Flash-style streaming softmax with
// warp-level bf16 MMAs, K/V tiles staged in swizzled shared memory.
//
// Decode: one query per executed sequence against that sequence's cache of
// executed-token keys / values (bandwidth bound: half a warp per key row).
#include "attention.cuh"

namespace qtale {

// ---------------------------------------------------------------------------
// small PTX helpers
// ---------------------------------------------------------------------------
__device__ __forceinline__ void cp_async_16(void* smem, const void* gmem, bool valid) {
  const uint32_t s = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(s), "l"(gmem), "r"(sz)
               : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const void* smem) {
  const uint32_t s = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(s));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], const void* smem) {
  const uint32_t s = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(s));
}
template <int ACT>
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0,
                                          uint32_t b1) {
  if (ACT == 1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
  } else {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
  }
}

// ---------------------------------------------------------------------------
// prefill
// ---------------------------------------------------------------------------
constexpr int kBQ = 128;  // query rows per CTA (16 per warp, 8 warps)
constexpr int kBK = 64;   // keys per tile
constexpr int kAttnThreads = 256;

// byte offset of 16-byte chunk c of row r in a tile with HD bf16 per row
template <int HD>
__device__ __forceinline__ int sw_off(int r, int c) {
  return r * (HD * 2) + (((c & ~7) | ((c ^ r) & 7)) << 4);
}

template <int HD, int ROWS>
__device__ __forceinline__ void load_tile(unsigned char* smem, const __nv_bfloat16* base, int ld,
                                          int row0, int n_rows_valid) {
  constexpr int CPR = HD / 8;  // chunks per row
  for (int e = threadIdx.x; e < ROWS * CPR; e += kAttnThreads) {
    const int r = e / CPR, c = e % CPR;
    const bool ok = r < n_rows_valid;
    const __nv_bfloat16* src = base + (size_t)(row0 + (ok ? r : 0)) * ld + c * 8;
    cp_async_16(smem + sw_off<HD>(r, c), src, ok);
  }
}

template <int HD, int ACT>
__global__ void __launch_bounds__(kAttnThreads)
    attn_prefill_kernel(const __nv_bfloat16* __restrict__ qkv, int ld, int k_off, int v_off,
                        const int32_t* __restrict__ cu_exec, int B, int rep,
                        __nv_bfloat16* __restrict__ out, int ldo, float scale_log2) {
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int TILE_BYTES = kBK * HD * 2;
  constexpr int Q_BYTES = kBQ * HD * 2;
  unsigned char* sQ = smem;
  unsigned char* sK = smem + Q_BYTES;                    // two buffers
  unsigned char* sV = smem + Q_BYTES + 2 * TILE_BYTES;   // two buffers

  // locate (sequence, query tile) of this CTA; heavy (late) tiles are scheduled first
  int b = -1, qt = 0;
  {
    int tile = blockIdx.x;
    for (int s = B - 1; s >= 0; --s) {
      const int len = cu_exec[s + 1] - cu_exec[s];
      const int nt = (len + kBQ - 1) / kBQ;
      if (tile < nt) { b = s; qt = nt - 1 - tile; break; }
      tile -= nt;
    }
  }
  if (b < 0) return;
  const int h = blockIdx.y;
  const int hk = h / rep;
  const int seq0 = cu_exec[b];
  const int len = cu_exec[b + 1] - seq0;
  const int q0 = qt * kBQ;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;

  const __nv_bfloat16* qbase = qkv + (size_t)h * HD;
  const __nv_bfloat16* kbase = qkv + k_off + (size_t)hk * HD;
  const __nv_bfloat16* vbase = qkv + v_off + (size_t)hk * HD;

  load_tile<HD, kBQ>(sQ, qbase, ld, seq0 + q0, min(kBQ, len - q0));
  cp_async_commit();
  // causal: key tiles that hold a key <= the last query row of this CTA
  const int n_kt = min((len + kBK - 1) / kBK, (q0 + kBQ) / kBK);
  load_tile<HD, kBK>(sK, kbase, ld, seq0, min(kBK, len));
  load_tile<HD, kBK>(sV, vbase, ld, seq0, min(kBK, len));
  cp_async_commit();

  cp_async_wait<1>();
  __syncthreads();
  // Q fragments of this warp's 16 rows
  uint32_t qf[HD / 16][4];
#pragma unroll
  for (int ks = 0; ks < HD / 16; ++ks) {
    const int mat = lane >> 3;
    const int r = warp * 16 + (mat & 1) * 8 + (lane & 7);
    const int c = ks * 2 + (mat >> 1);
    ldsm_x4(qf[ks], sQ + sw_off<HD>(r, c));
  }

  float o[HD / 8][4];
#pragma unroll
  for (int i = 0; i < HD / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m_run[2] = {-INFINITY, -INFINITY};
  float l_run[2] = {0.f, 0.f};

  for (int kt = 0; kt < n_kt; ++kt) {
    const int buf = kt & 1;
    if (kt + 1 < n_kt) {
      const int k0n = (kt + 1) * kBK;
      load_tile<HD, kBK>(sK + (buf ^ 1) * TILE_BYTES, kbase, ld, seq0 + k0n, min(kBK, len - k0n));
      load_tile<HD, kBK>(sV + (buf ^ 1) * TILE_BYTES, vbase, ld, seq0 + k0n, min(kBK, len - k0n));
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    const unsigned char* k_s = sK + buf * TILE_BYTES;
    const unsigned char* v_s = sV + buf * TILE_BYTES;
    const int k0 = kt * kBK;
    const int warp_row0 = q0 + warp * 16;
    // a key tile entirely above this warp's rows contributes nothing (warp-uniform skip)
    if (k0 <= warp_row0 + 15) {

    // S = Q K^T for this warp's 16 rows x 64 keys
    float s[kBK / 8][4];
#pragma unroll
    for (int i = 0; i < kBK / 8; ++i) { s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < HD / 16; ++ks) {
#pragma unroll
      for (int np = 0; np < kBK / 16; ++np) {
        uint32_t kf[4];
        const int mat = lane >> 3;
        const int r = np * 16 + (mat >> 1) * 8 + (lane & 7);
        const int c = ks * 2 + (mat & 1);
        ldsm_x4(kf, k_s + sw_off<HD>(r, c));
        mma_16816<ACT>(s[2 * np], qf[ks], kf[0], kf[1]);
        mma_16816<ACT>(s[2 * np + 1], qf[ks], kf[2], kf[3]);
      }
    }
    // scale, causal / length mask (only tiles that reach past this warp's first row or the
    // end of the sequence need it)
    const bool diag = (k0 + kBK - 1 > warp_row0) || (k0 + kBK > len);
    const int row_a = warp_row0 + g, row_b = row_a + 8;
#pragma unroll
    for (int i = 0; i < kBK / 8; ++i) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int key = k0 + i * 8 + 2 * t + (e & 1);
        const int row = (e < 2) ? row_a : row_b;
        float v = s[i][e] * scale_log2;
        if (diag && (key > row || key >= len)) v = -INFINITY;
        s[i][e] = v;
      }
    }
    // online softmax (base 2)
    float mx[2] = {m_run[0], m_run[1]};
#pragma unroll
    for (int i = 0; i < kBK / 8; ++i) {
      mx[0] = fmaxf(mx[0], fmaxf(s[i][0], s[i][1]));
      mx[1] = fmaxf(mx[1], fmaxf(s[i][2], s[i][3]));
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
    }
    float corr[2], msafe[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      msafe[r] = (mx[r] == -INFINITY) ? 0.f : mx[r];
      corr[r] = exp2f(m_run[r] - msafe[r]);
      m_run[r] = mx[r];
      l_run[r] *= corr[r];
    }
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) {
      o[i][0] *= corr[0]; o[i][1] *= corr[0];
      o[i][2] *= corr[1]; o[i][3] *= corr[1];
    }
    uint32_t pf[kBK / 16][4];
#pragma unroll
    for (int i = 0; i < kBK / 8; ++i) {
      const float p0 = exp2f(s[i][0] - msafe[0]), p1 = exp2f(s[i][1] - msafe[0]);
      const float p2 = exp2f(s[i][2] - msafe[1]), p3 = exp2f(s[i][3] - msafe[1]);
      l_run[0] += p0 + p1;
      l_run[1] += p2 + p3;
      pf[i >> 1][(i & 1) * 2 + 0] = Act16<ACT>::pack(p0, p1);
      pf[i >> 1][(i & 1) * 2 + 1] = Act16<ACT>::pack(p2, p3);
    }
    // O += P V
#pragma unroll
    for (int kk = 0; kk < kBK / 16; ++kk) {
#pragma unroll
      for (int np = 0; np < HD / 16; ++np) {
        uint32_t vf[4];
        const int mat = lane >> 3;
        const int r = kk * 16 + (mat & 1) * 8 + (lane & 7);
        const int c = np * 2 + (mat >> 1);
        ldsm_x4_trans(vf, v_s + sw_off<HD>(r, c));
        mma_16816<ACT>(o[2 * np], pf[kk], vf[0], vf[1]);
        mma_16816<ACT>(o[2 * np + 1], pf[kk], vf[2], vf[3]);
      }
    }
    }
    __syncthreads();  // all warps done with this buffer before it is refilled
  }

  // finalise: divide by the row sums (reduced over the 4 lanes sharing a row)
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
  }
  const float inv0 = l_run[0] > 0.f ? 1.f / l_run[0] : 0.f;
  const float inv1 = l_run[1] > 0.f ? 1.f / l_run[1] : 0.f;
  const int ra = q0 + warp * 16 + g, rb = ra + 8;
#pragma unroll
  for (int i = 0; i < HD / 8; ++i) {
    const int col = h * HD + i * 8 + 2 * t;
    if (ra < len)
      *reinterpret_cast<uint32_t*>(out + (size_t)(seq0 + ra) * ldo + col) =
          Act16<ACT>::pack(o[i][0] * inv0, o[i][1] * inv0);
    if (rb < len)
      *reinterpret_cast<uint32_t*>(out + (size_t)(seq0 + rb) * ldo + col) =
          Act16<ACT>::pack(o[i][2] * inv1, o[i][3] * inv1);
  }
}

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
  const size_t row_stride = (size_t)Hkv * HD;
  const __nv_bfloat16* kb = cache_k + ((size_t)b * cap) * row_stride + (size_t)hk * HD + sub * 8;
  const __nv_bfloat16* vb = cache_v + ((size_t)b * cap) * row_stride + (size_t)hk * HD + sub * 8;
  constexpr int UNROLL = 4;
  for (int k0 = grp; k0 < n_keys; k0 += GROUPS * UNROLL) {
    uint4 kv[UNROLL], vv[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const int key = k0 + u * GROUPS;
      if (key < n_keys) {
        kv[u] = ld_nc_16(kb + (size_t)key * row_stride);
        vv[u] = ld_nc_16(vb + (size_t)key * row_stride);
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
static int launch_prefill_hd(const void* qkv, int ld, int k_off, int v_off, const int32_t* cu_exec,
                             int B, int H, int Hkv, int T_cap, void* out, int ldo, cudaStream_t s) {
  const size_t smem = (size_t)(kBQ + 4 * kBK) * HD * 2;
  static bool configured[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    if (cudaFuncSetAttribute(attn_prefill_kernel<HD, ACT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)smem) != cudaSuccess)
      return QTALE_ERR_CUDA;
    configured[dev] = true;
  }
  const int max_tiles = (T_cap + kBQ - 1) / kBQ + B;
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)HD);
  dim3 grid(max_tiles, H);
  attn_prefill_kernel<HD, ACT><<<grid, kAttnThreads, smem, s>>>(
      static_cast<const __nv_bfloat16*>(qkv), ld, k_off, v_off, cu_exec, B, H / Hkv,
      static_cast<__nv_bfloat16*>(out), ldo, scale_log2);
  return launch_status(cudaGetLastError());
}

int launch_attn_prefill(const void* qkv, int ld, int H, int Hkv, int hd, int act,
                        const int32_t* cu_exec, int B, int T_cap, void* out, int ldo,
                        cudaStream_t s) {
  const int k_off = H * hd, v_off = (H + Hkv) * hd;
#define QTALE_PF(HD_, ACT_) \
  launch_prefill_hd<HD_, ACT_>(qkv, ld, k_off, v_off, cu_exec, B, H, Hkv, T_cap, out, ldo, s)
  if (hd == 128) return act == QTALE_ACT_F16 ? QTALE_PF(128, 1) : QTALE_PF(128, 0);
  if (hd == 64) return act == QTALE_ACT_F16 ? QTALE_PF(64, 1) : QTALE_PF(64, 0);
#undef QTALE_PF
  return QTALE_ERR_SHAPE;
}

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
