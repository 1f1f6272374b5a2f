// Weight-only quantised GEMM on the tcgen05 tensor cores (Sec. 4.1: 4-bit /
// 3-bit integer weights with per-group parameters; the layer's four linears).
//
// The product is computed transposed, D[n, m] = sum_k W[n, k] * A[m, k]:
//   * the 128 weight rows of a tile are the MMA's M dimension; the packed codes
//     are fetched by a bulk TMA copy, turned into bf16 in registers
//     ((code - zero) * scale exactly in fp32, one rounding) and written with
//     tcgen05.st into tensor memory, from where the MMA reads its A operand;
//   * up to 256 tokens are the N dimension; their activations arrive by a tiled
//     TMA load into 128-byte-swizzled shared memory (the B operand);
//   * the fp32 accumulator D (128 lanes x TN columns) lives in tensor memory and
//     is drained by four epilogue warps, one TMEM lane quadrant each.
// The grid is persistent (one CTA per SM) and reads the number of executed
// tokens from device memory, so no launch parameter depends on the routing.
//
// Warp roles (320 threads): warp 0 TMA producer, warp 1 MMA issuer and TMEM
// allocator, warps 2-5 dequantisers, warps 6-9 epilogue.
#include <cuda.h>

#include <string.h>

#include "common.cuh"
#include "ptx.cuh"
#include "wq_gemm.cuh"

namespace qtale {

using namespace ptx;

constexpr int kGemmThreads = 320;
constexpr int kTileRows = 128;          // weight rows per tile (MMA M)
constexpr int kKB = 64;                 // K elements per pipeline stage (128 B of bf16)
constexpr uint32_t kSpinLimit = 1u << 24;
constexpr int kTmemCols = 512;
constexpr int kTmemAColBase = 256;      // A-operand stages start here; D uses [0, TN)
constexpr int kAColsPerStage = kKB / 2; // two bf16 per 32-bit column

template <int TN, int BITS>
struct GemmCfg {
  static constexpr int kXBytes = TN * 128;
  static constexpr int kWBytes = BITS == 16 ? kTileRows * 128 : kTileRows * kKB * BITS / 8;
  static constexpr int kSzBytes = BITS == 16 ? 0 : kTileRows * 4;
  static constexpr int kStageBytes = (kXBytes + kWBytes + kSzBytes + 1023) / 1024 * 1024;
  static constexpr int kMaxStages = (224 * 1024) / kStageBytes;
  static constexpr int kStages = kMaxStages > 8 ? 8 : kMaxStages;
  static constexpr size_t kSmemBytes = (size_t)kStages * kStageBytes + 1024;
  static_assert(kStages >= 2, "pipeline needs at least two stages");
  static_assert(kTmemAColBase + kStages * kAColsPerStage <= kTmemCols, "TMEM budget");
};

struct GemmParams {
  const uint8_t* packed;   // repacked blob (codes, then scale/zero words)
  size_t sz_offset;        // byte offset of the scale/zero region
  int n_tiles;             // 128-row tiles
  int nkb;                 // 64-wide K blocks
  int kb_per_group;        // group / 64
  int N, F, row_mode;      // logical rows; F = N / 2 for SWIGLU row mode
  const int32_t* m_dev;    // executed-token count (device) or NULL
  int M_cap;
  int epilogue;
  void* y;
  int ldy;
  const int32_t* idx;
  const void* resid;
  int ld_resid;
  void* dst;
  int ld_dst;
  int* status;
};

struct __align__(8) GemmShared {
  uint64_t full[8];
  uint64_t empty[8];
  uint64_t a_full[8];
  uint64_t d_full;
  uint64_t d_empty;
  uint32_t tmem_base;
  volatile int abort_flag;
};

// Bounded wait: gives up after kSpinLimit polls, records a timeout and raises
// the CTA-wide abort flag so that every role leaves its loop.
__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, GemmShared* sh,
                                              int* status) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 255u) == 255u && sh->abort_flag) return false;
  }
  sh->abort_flag = 1;
  report_device_error(status, QTALE_ERR_TIMEOUT);
  return false;
}

// logical output feature of lane L of tile nt (-1: padding row)
__device__ __forceinline__ int tile_row_to_n(const GemmParams& p, int nt, int L) {
  if (p.row_mode == QTALE_WQ_ROWS_SWIGLU) {
    const int q = L >> 5, r = L & 31;
    const int j = nt * 64 + q * 16 + (r & 15);
    if (j >= p.F) return -1;
    return (r < 16) ? j : p.F + j;
  }
  const int n = nt * kTileRows + L;
  return n < p.N ? n : -1;
}

// Eight codes sitting in the 4-bit slots of `t` -> four bf16x2 registers.
// Slot i holds the code in its low QBITS bits.  The code is moved into a float
// mantissa next to 2^23, so (float - (2^23 + zero * 16^i)) * (scale / 16^i) is
// exactly (code - zero) * scale.
template <uint32_t QMASK, int ACT>
__device__ __forceinline__ void dequant8(uint32_t t, const float (&C)[5], const float (&S)[5],
                                         uint32_t* out) {
  constexpr uint32_t MAGIC = 0x4B000000u;  // 2^23
  const uint32_t hi = t >> 12;
  float v[8];
#pragma unroll
  for (int i = 0; i < 5; ++i)
    v[i] = (__uint_as_float((t & (QMASK << (4 * i))) | MAGIC) - C[i]) * S[i];
#pragma unroll
  for (int i = 5; i < 8; ++i)
    v[i] = (__uint_as_float((hi & (QMASK << (4 * (i - 3)))) | MAGIC) - C[i - 3]) * S[i - 3];
#pragma unroll
  for (int q = 0; q < 4; ++q) out[q] = Act16<ACT>::pack(v[2 * q], v[2 * q + 1]);
}

template <int TN, int BITS, int ACT>
__global__ void __launch_bounds__(kGemmThreads, 1)
    wq_gemm_kernel(const __grid_constant__ CUtensorMap tmap_x,
                   const __grid_constant__ CUtensorMap tmap_w, const GemmParams p) {
  using Cfg = GemmCfg<TN, BITS>;
  constexpr int S = Cfg::kStages;
  extern __shared__ unsigned char smem_dyn[];
  __shared__ GemmShared sh;
  unsigned char* stage_base = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(&sh.full[s], 1);
      mbar_init(&sh.empty[s], 1);
      mbar_init(&sh.a_full[s], 4);
    }
    mbar_init(&sh.d_full, 1);
    mbar_init(&sh.d_empty, 4);
    sh.abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(&sh.tmem_base, kTmemCols);
    tmem_relinquish();
  }
  if (warp == 0 && lane == 0) {
    prefetch_tmap(&tmap_x);
    if (BITS == 16) prefetch_tmap(&tmap_w);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sh.tmem_base;

  int M = p.M_cap;
  if (p.m_dev) M = min(M, *p.m_dev);
  M = max(M, 0);
  const int n_mt = (M + TN - 1) / TN;
  const int total_tiles = n_mt * p.n_tiles;
  const int nkb = p.nkb;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        const int nt = tile / n_mt, mt = tile % n_mt;
        for (int kb = 0; kb < nkb; ++kb) {
          if (!wait_or_abort(&sh.empty[s], ph ^ 1u, &sh, p.status)) goto producer_done;
          unsigned char* st = stage_base + (size_t)s * Cfg::kStageBytes;
          const bool with_sz = BITS != 16 && (kb % p.kb_per_group) == 0;
          mbar_arrive_expect_tx(&sh.full[s],
                                Cfg::kXBytes + Cfg::kWBytes + (with_sz ? Cfg::kSzBytes : 0));
          tma_load_2d(st, &tmap_x, &sh.full[s], kb * kKB, mt * TN);
          if (BITS == 16) {
            tma_load_2d(st + Cfg::kXBytes, &tmap_w, &sh.full[s], kb * kKB, nt * kTileRows);
          } else {
            bulk_load(st + Cfg::kXBytes, p.packed + ((size_t)nt * nkb + kb) * Cfg::kWBytes,
                      Cfg::kWBytes, &sh.full[s]);
            if (with_sz)
              bulk_load(st + Cfg::kXBytes + Cfg::kWBytes,
                        p.packed + p.sz_offset +
                            ((size_t)nt * (nkb / p.kb_per_group) + kb / p.kb_per_group) *
                                Cfg::kSzBytes,
                        Cfg::kSzBytes, &sh.full[s]);
          }
          if (++s == S) { s = 0; ph ^= 1u; }
        }
      }
    producer_done:;
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer --------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_16bit_f32(kTileRows, TN, ACT == 1);
      int s = 0;
      uint32_t ph = 0, dph = 0;
      for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        if (!wait_or_abort(&sh.d_empty, dph ^ 1u, &sh, p.status)) goto mma_done;
        tc_fence_after();
        for (int kb = 0; kb < nkb; ++kb) {
          if (!wait_or_abort(&sh.full[s], ph, &sh, p.status)) goto mma_done;
          if (BITS != 16) {
            if (!wait_or_abort(&sh.a_full[s], ph, &sh, p.status)) goto mma_done;
          }
          tc_fence_after();
          unsigned char* st = stage_base + (size_t)s * Cfg::kStageBytes;
          const uint64_t b_desc = smem_desc_sw128(smem_u32(st));
#pragma unroll
          for (int j = 0; j < kKB / 16; ++j) {
            const uint32_t acc = (kb | j) != 0 ? 1u : 0u;
            if (BITS == 16) {
              const uint64_t a_desc = smem_desc_sw128(smem_u32(st + Cfg::kXBytes));
              mma_ss(tmem_base, a_desc + 2u * j, b_desc + 2u * j, idesc, acc);
            } else {
              mma_ts(tmem_base, tmem_base + kTmemAColBase + s * kAColsPerStage + j * 8,
                     b_desc + 2u * j, idesc, acc);
            }
          }
          mma_commit(&sh.empty[s]);  // frees the smem stage and the TMEM A slot
          if (++s == S) { s = 0; ph ^= 1u; }
        }
        mma_commit(&sh.d_full);
        dph ^= 1u;
      }
    mma_done:;
    }
  } else if (warp < 6) {
    // ------------------------------- dequantisers --------------------------------
    if (BITS != 16) {
      const int quad = warp & 3;
      const int L = quad * 32 + lane;
      int s = 0;
      uint32_t ph = 0;
      float C[5], Sc[5];
#pragma unroll
      for (int i = 0; i < 5; ++i) { C[i] = 0.f; Sc[i] = 0.f; }
      for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        for (int kb = 0; kb < nkb; ++kb) {
          if (!wait_or_abort(&sh.full[s], ph, &sh, p.status)) goto dequant_done;
          const unsigned char* st = stage_base + (size_t)s * Cfg::kStageBytes + Cfg::kXBytes;
          if ((kb % p.kb_per_group) == 0) {
            const uint32_t sz = reinterpret_cast<const uint32_t*>(st + Cfg::kWBytes)[L];
            const float scale = __half2float(__ushort_as_half((unsigned short)(sz & 0xFFFFu)));
            const float zero = __half2float(__ushort_as_half((unsigned short)(sz >> 16)));
#pragma unroll
            for (int i = 0; i < 5; ++i) {
              C[i] = 8388608.f + zero * (float)(1 << (4 * i));
              Sc[i] = scale * (1.f / (float)(1 << (4 * i)));
            }
          }
          const uint32_t a_taddr =
              tmem_base + ((uint32_t)(quad * 32) << 16) + kTmemAColBase + s * kAColsPerStage;
          if (BITS == 4) {
#pragma unroll
            for (int part = 0; part < 2; ++part) {
              const uint4 w = reinterpret_cast<const uint4*>(st)[part * kTileRows + L];
              uint32_t r[16];
              dequant8<0xFu, ACT>(w.x, C, Sc, r + 0);
              dequant8<0xFu, ACT>(w.y, C, Sc, r + 4);
              dequant8<0xFu, ACT>(w.z, C, Sc, r + 8);
              dequant8<0xFu, ACT>(w.w, C, Sc, r + 12);
              tmem_st_x16(a_taddr + part * 16, r);
            }
          } else {
            // 3-bit: low two bits of 16 codes per word (plane A), high bit of 32 codes
            // per word (plane B).  A nibble-style word with the code in the low 3 bits
            // of each 4-bit slot is assembled with one bitwise select.
            const uint4 a = reinterpret_cast<const uint4*>(st)[L];
            const uint2 b = reinterpret_cast<const uint2*>(st + kTileRows * 16)[L];
            const uint32_t aw[4] = {a.x, a.y, a.z, a.w};
            const uint32_t bw[2] = {b.x, b.y};
#pragma unroll
            for (int part = 0; part < 2; ++part) {
              uint32_t r[16];
#pragma unroll
              for (int uu = 0; uu < 4; ++uu) {
                const int u = part * 4 + uu;
                const uint32_t a2 = (u & 1) ? (aw[u >> 1] >> 2) : aw[u >> 1];
                const int rr = u & 3;
                const uint32_t b1 = rr == 0 ? (bw[u >> 2] << 2)
                                  : rr == 1 ? (bw[u >> 2] << 1)
                                  : rr == 2 ? bw[u >> 2] : (bw[u >> 2] >> 1);
                const uint32_t t = (a2 & 0x33333333u) | (b1 & 0xCCCCCCCCu);
                dequant8<0x7u, ACT>(t, C, Sc, r + 4 * uu);
              }
              tmem_st_x16(a_taddr + part * 16, r);
            }
          }
          tmem_wait_st();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sh.a_full[s]);
          if (++s == S) { s = 0; ph ^= 1u; }
        }
      }
    dequant_done:;
    }
  } else {
    // --------------------------------- epilogue -----------------------------------
    const int quad = warp & 3;
    const int L = quad * 32 + lane;
    uint32_t dph = 0;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
      const int nt = tile / n_mt, mt = tile % n_mt;
      if (!wait_or_abort(&sh.d_full, dph, &sh, p.status)) break;
      tc_fence_after();
      const int n = tile_row_to_n(p, nt, L);
      const int m_base = mt * TN;
#pragma unroll 1
      for (int c0 = 0; c0 < TN; c0 += 32) {
        const int m0 = m_base + c0;
        if (m0 >= M) break;
        const int n_cols = min(32, M - m0);  // warp-uniform
        uint32_t r[32];
        tmem_ld_x32(tmem_base + ((uint32_t)(quad * 32) << 16) + c0, r);
        if (p.epilogue == QTALE_EPI_RESID_F32 || p.epilogue == QTALE_EPI_RESID_SCATTER) {
          // all residual reads of the chunk are issued before the first store so that
          // their latencies overlap (one row index per column, fetched by one lane)
          const int my_row = (lane < n_cols) ? __ldg(p.idx + m0 + lane) : 0;
          float res[32];
          if (p.epilogue == QTALE_EPI_RESID_F32) {
            const unsigned short* rp = static_cast<const unsigned short*>(p.resid);
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              const int row = __shfl_sync(0xffffffffu, my_row, c);
              res[c] = (c < n_cols && n >= 0)
                           ? bf16_bits_to_float(__ldg(rp + (size_t)row * p.ld_resid + n)) : 0.f;
            }
            tmem_wait_ld();
            if (n >= 0) {
              float* y = static_cast<float*>(p.y);
#pragma unroll
              for (int c = 0; c < 32; ++c)
                if (c < n_cols) y[(size_t)(m0 + c) * p.ldy + n] = res[c] + __uint_as_float(r[c]);
            }
          } else {
            const float* rp = static_cast<const float*>(p.resid);
#pragma unroll
            for (int c = 0; c < 32; ++c)
              res[c] = (c < n_cols && n >= 0) ? __ldg(rp + (size_t)(m0 + c) * p.ld_resid + n) : 0.f;
            tmem_wait_ld();
            __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(p.dst);
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              const int row = __shfl_sync(0xffffffffu, my_row, c);
              if (c < n_cols && n >= 0)
                dst[(size_t)row * p.ld_dst + n] = __float2bfloat16_rn(res[c] + __uint_as_float(r[c]));
            }
          }
        } else if (p.epilogue == QTALE_EPI_SWIGLU) {
          tmem_wait_ld();
          // lanes 0-15 hold gate rows, lanes 16-31 the matching up rows
          float other[16];
#pragma unroll
          for (int i = 0; i < 16; ++i)
            other[i] = __shfl_xor_sync(0xffffffffu,
                                       __uint_as_float((lane < 16) ? r[16 + i] : r[i]), 16);
          const int j = nt * 64 + quad * 16 + (lane & 15);
          if (j < p.F) {
            unsigned short* y = static_cast<unsigned short*>(p.y);
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const int c = (lane < 16) ? i : 16 + i;
              const float g = (lane < 16) ? __uint_as_float(r[c]) : other[i];
              const float u = (lane < 16) ? other[i] : __uint_as_float(r[c]);
              if (c < n_cols)
                y[(size_t)(m0 + c) * p.ldy + j] = Act16<ACT>::one(g / (1.f + __expf(-g)) * u);
            }
          }
        } else {
          tmem_wait_ld();
          if (n >= 0) {
            if (p.epilogue == QTALE_EPI_STORE_16) {
              unsigned short* y = static_cast<unsigned short*>(p.y);
#pragma unroll
              for (int c = 0; c < 32; ++c)
                if (c < n_cols) y[(size_t)(m0 + c) * p.ldy + n] = Act16<ACT>::one(__uint_as_float(r[c]));
            } else {  // QTALE_EPI_STORE_F32
              float* y = static_cast<float*>(p.y);
#pragma unroll
              for (int c = 0; c < 32; ++c)
                if (c < n_cols) y[(size_t)(m0 + c) * p.ldy + n] = __uint_as_float(r[c]);
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.d_empty);
      dph ^= 1u;
    }
  }

  // teardown: every thread arrives here, also after an abort
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) ==
            cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// Tensor map over a row-major 16-bit (bf16 or fp16) matrix [rows, cols] with pitch `ld` elements;
// box = 64 columns x box_rows rows, 128-byte swizzle, zero fill out of bounds.
static int make_tmap_16(CUtensorMap* m, const void* base, int rows, int cols, int ld,
                        int box_rows, int act) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return QTALE_ERR_CUDA;
  cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t gstr[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)kKB, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(m, act == QTALE_ACT_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstr, box,
                  estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? QTALE_OK : QTALE_ERR_CUDA;
}

template <int TN, int BITS, int ACT>
static int launch_gemm(const CUtensorMap& tx, const CUtensorMap& tw, const GemmParams& p,
                       cudaStream_t s) {
  using Cfg = GemmCfg<TN, BITS>;
  static bool configured[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    if (cudaFuncSetAttribute(wq_gemm_kernel<TN, BITS, ACT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)Cfg::kSmemBytes) != cudaSuccess)
      return QTALE_ERR_CUDA;
    configured[dev] = true;
  }
  const int max_tiles = ((p.M_cap + TN - 1) / TN) * p.n_tiles;
  int grid = sm_count();
  if (grid > max_tiles) grid = max_tiles;
  if (grid < 1) grid = 1;
  wq_gemm_kernel<TN, BITS, ACT><<<grid, kGemmThreads, Cfg::kSmemBytes, s>>>(tx, tw, p);
  return launch_status(cudaGetLastError());
}

template <int BITS, int ACT>
static int dispatch_tn(const CUtensorMap& tx, const CUtensorMap& tw, const GemmParams& p, int tn,
                       cudaStream_t s) {
  if (tn == 64) return launch_gemm<64, BITS, ACT>(tx, tw, p, s);
  if (tn == 128) return launch_gemm<128, BITS, ACT>(tx, tw, p, s);
  return launch_gemm<256, BITS, ACT>(tx, tw, p, s);
}

static int pick_tn(int M_cap) { return M_cap <= 64 ? 64 : (M_cap <= 128 ? 128 : 256); }

size_t wq_blob_bytes(int N, int K, int bits, int group, int row_mode, WqGeometry* g) {
  WqGeometry q;
  q.K_pad = (K + group - 1) / group * group;
  q.nkb = q.K_pad / kKB;
  q.ng = q.K_pad / group;
  q.n_tiles = row_mode == QTALE_WQ_ROWS_SWIGLU ? ((N / 2) + 63) / 64 : (N + kTileRows - 1) / kTileRows;
  q.block_bytes = kTileRows * kKB * bits / 8;
  q.sz_offset = (size_t)q.n_tiles * q.nkb * q.block_bytes;
  q.total = q.sz_offset + (size_t)q.n_tiles * q.ng * kTileRows * 4;
  if (g) *g = q;
  return q.total;
}

int wq_gemm_launch(const void* a, int lda, const int32_t* m_dev, int M_cap,
                   const qtale_wq_weight* w, int act, int epilogue, const qtale_epilogue_args* epi,
                   void* y, int ldy, cudaStream_t s) {
  WqGeometry g;
  wq_blob_bytes(w->N, w->K, w->bits, w->group, w->row_mode, &g);
  GemmParams p;
  memset(&p, 0, sizeof(p));
  p.packed = static_cast<const uint8_t*>(w->packed);
  p.sz_offset = g.sz_offset;
  p.n_tiles = g.n_tiles;
  p.nkb = g.nkb;
  p.kb_per_group = w->group / kKB;
  p.N = w->N;
  p.F = w->N / 2;
  p.row_mode = w->row_mode;
  p.m_dev = m_dev;
  p.M_cap = M_cap;
  p.epilogue = epilogue;
  p.y = y;
  p.ldy = ldy;
  if (epi) {
    p.idx = epi->idx;
    p.resid = epi->resid;
    p.ld_resid = epi->ld_resid;
    p.dst = epi->dst;
    p.ld_dst = epi->ld_dst;
  }
  p.status = device_status_ptr();
  const int tn = pick_tn(M_cap);
  CUtensorMap tx, tw;
  memset(&tw, 0, sizeof(tw));
  int rc = make_tmap_16(&tx, a, M_cap, w->K, lda, tn, act);
  if (rc != QTALE_OK) return rc;
  if (act == QTALE_ACT_F16)
    return w->bits == 4 ? dispatch_tn<4, 1>(tx, tw, p, tn, s) : dispatch_tn<3, 1>(tx, tw, p, tn, s);
  return w->bits == 4 ? dispatch_tn<4, 0>(tx, tw, p, tn, s) : dispatch_tn<3, 0>(tx, tw, p, tn, s);
}

int bf16_gemm_launch(const void* a, int lda, const int32_t* m_dev, int M_cap, const void* w_bf16,
                     int N, int K, int ldw, float* y, int ldy, cudaStream_t s) {
  GemmParams p;
  memset(&p, 0, sizeof(p));
  p.n_tiles = (N + kTileRows - 1) / kTileRows;
  p.nkb = (K + kKB - 1) / kKB;
  p.kb_per_group = 1;
  p.N = N;
  p.row_mode = QTALE_WQ_ROWS_PLAIN;
  p.m_dev = m_dev;
  p.M_cap = M_cap;
  p.epilogue = QTALE_EPI_STORE_F32;
  p.y = y;
  p.ldy = ldy;
  p.status = device_status_ptr();
  const int tn = pick_tn(M_cap);
  CUtensorMap tx, tw;
  int rc = make_tmap_16(&tx, a, M_cap, K, lda, tn, QTALE_ACT_BF16);
  if (rc != QTALE_OK) return rc;
  rc = make_tmap_16(&tw, w_bf16, N, K, ldw, kTileRows, QTALE_ACT_BF16);
  if (rc != QTALE_OK) return rc;
  return dispatch_tn<16, 0>(tx, tw, p, tn, s);
}

// ---- offline repack (host) -------------------------------------------------------

static inline unsigned canon_code(const uint8_t* row, int k, int bits) {
  if (bits == 4) return (k & 1) ? (row[k >> 1] >> 4) : (row[k >> 1] & 0xF);
  const int bit = 3 * k;
  unsigned v = row[bit >> 3];
  if ((bit & 7) > 5) v |= (unsigned)row[(bit >> 3) + 1] << 8;
  return (v >> (bit & 7)) & 7u;
}

static inline float half_to_float_host(uint16_t h) {
  return __half2float(__ushort_as_half(h));
}

}  // namespace qtale

using namespace qtale;

extern "C" {

int qtale_wq_repack(const uint8_t* codes, const uint16_t* scales, const uint16_t* zeros, int N,
                    int K, int bits, int group, int row_mode, void* packed_out, size_t* bytes) {
  if (!bytes) return QTALE_ERR_NULL;
  if (bits != 3 && bits != 4) return QTALE_ERR_BITS;
  if (group != 64 && group != 128) return QTALE_ERR_GROUP;
  if (N < 1 || K < 1) return QTALE_ERR_SHAPE;
  if (row_mode != QTALE_WQ_ROWS_PLAIN && row_mode != QTALE_WQ_ROWS_SWIGLU) return QTALE_ERR_MODE;
  if (row_mode == QTALE_WQ_ROWS_SWIGLU && (N % 2) != 0) return QTALE_ERR_SHAPE;
  WqGeometry g;
  const size_t total = wq_blob_bytes(N, K, bits, group, row_mode, &g);
  if (!packed_out) {
    *bytes = total;
    return QTALE_OK;
  }
  if (*bytes < total) return QTALE_ERR_CAPACITY;
  if (!codes || !scales || !zeros) return QTALE_ERR_NULL;
  *bytes = total;
  uint8_t* out = static_cast<uint8_t*>(packed_out);
  memset(out, 0, total);
  const int row_bytes = bits == 4 ? (K + 1) / 2 : (3 * K + 7) / 8;
  const int ng_in = (K + group - 1) / group;
  const int F = N / 2;
  for (int nt = 0; nt < g.n_tiles; ++nt) {
    for (int L = 0; L < kTileRows; ++L) {
      int n;
      if (row_mode == QTALE_WQ_ROWS_SWIGLU) {
        const int q = L >> 5, r = L & 31;
        const int j = nt * 64 + q * 16 + (r & 15);
        n = (j < F) ? ((r < 16) ? j : F + j) : -1;
      } else {
        n = nt * kTileRows + L;
        if (n >= N) n = -1;
      }
      uint32_t* sz = reinterpret_cast<uint32_t*>(out + g.sz_offset) + (size_t)nt * g.ng * kTileRows;
      for (int gi = 0; gi < g.ng; ++gi) {
        uint32_t v = 0;  // padding rows: scale 0, zero 0
        if (n >= 0 && gi < ng_in)
          v = (uint32_t)scales[(size_t)n * ng_in + gi] | ((uint32_t)zeros[(size_t)n * ng_in + gi] << 16);
        sz[(size_t)gi * kTileRows + L] = v;
      }
      if (n < 0) continue;
      const uint8_t* row = codes + (size_t)n * row_bytes;
      for (int kb = 0; kb < g.nkb; ++kb) {
        uint8_t* blk = out + ((size_t)nt * g.nkb + kb) * g.block_bytes;
        unsigned q[64];
        for (int i = 0; i < 64; ++i) {
          const int k = kb * 64 + i;
          if (k < K) {
            q[i] = canon_code(row, k, bits);
          } else {  // K padding: code == zero-point, i.e. weight 0
            const int gi = k / group;
            const float z = gi < ng_in ? half_to_float_host(zeros[(size_t)n * ng_in + gi]) : 0.f;
            q[i] = (unsigned)z;
          }
        }
        if (bits == 4) {
          // [part][lane][4 words]; word j of part p: k = 32p + 8j + i in nibble i
          for (int part = 0; part < 2; ++part) {
            uint32_t* wdst = reinterpret_cast<uint32_t*>(blk) + ((size_t)part * kTileRows + L) * 4;
            for (int j = 0; j < 4; ++j) {
              uint32_t wv = 0;
              for (int i = 0; i < 8; ++i) wv |= (q[32 * part + 8 * j + i] & 0xFu) << (4 * i);
              wdst[j] = wv;
            }
          }
        } else {
          // plane A: [lane][4 words], 2-bit field f of word w2 <- code k = 8(2 w2 + f%2) + f/2
          // plane B: [lane][2 words], bit 4i + u%4 of word u/4 <- high bit of code 8u + i
          uint32_t* a = reinterpret_cast<uint32_t*>(blk) + (size_t)L * 4;
          uint32_t* b = reinterpret_cast<uint32_t*>(blk + kTileRows * 16) + (size_t)L * 2;
          for (int w2 = 0; w2 < 4; ++w2) {
            uint32_t wv = 0;
            for (int f = 0; f < 16; ++f) wv |= (q[8 * (2 * w2 + (f & 1)) + (f >> 1)] & 3u) << (2 * f);
            a[w2] = wv;
          }
          uint32_t b0 = 0, b1 = 0;
          for (int u = 0; u < 8; ++u)
            for (int i = 0; i < 8; ++i) {
              const uint32_t hb = (q[8 * u + i] >> 2) & 1u;
              if (u < 4) b0 |= hb << (4 * i + (u & 3)); else b1 |= hb << (4 * i + (u & 3));
            }
          b[0] = b0;
          b[1] = b1;
        }
      }
    }
  }
  return QTALE_OK;
}

int qtale_wq_gemm(const void* a, int lda, const int32_t* m_dev, int M_cap, const qtale_wq_weight* w,
                  int act_dtype, int epilogue, const qtale_epilogue_args* epi, void* y, int ldy,
                  void* stream) {
  if (!a || !w || !w->packed) return QTALE_ERR_NULL;
  if (act_dtype != QTALE_ACT_BF16 && act_dtype != QTALE_ACT_F16) return QTALE_ERR_MODE;
  if (w->bits != 3 && w->bits != 4) return QTALE_ERR_BITS;
  if (w->group != 64 && w->group != 128) return QTALE_ERR_GROUP;
  if (M_cap < 1 || w->N < 1 || w->K < 1 || lda < w->K) return QTALE_ERR_SHAPE;
  if (epilogue < QTALE_EPI_STORE_16 || epilogue > QTALE_EPI_SWIGLU) return QTALE_ERR_MODE;
  if (epilogue == QTALE_EPI_SWIGLU && w->row_mode != QTALE_WQ_ROWS_SWIGLU) return QTALE_ERR_MODE;
  if (epilogue == QTALE_EPI_RESID_F32 || epilogue == QTALE_EPI_RESID_SCATTER) {
    if (!epi || !epi->idx || !epi->resid) return QTALE_ERR_NULL;
    if (epilogue == QTALE_EPI_RESID_SCATTER && !epi->dst) return QTALE_ERR_NULL;
  }
  if (epilogue != QTALE_EPI_RESID_SCATTER && !y) return QTALE_ERR_NULL;
  if (!aligned16(a) || !aligned16(w->packed) || (lda * 2) % 16 != 0) return QTALE_ERR_ALIGN;
  return wq_gemm_launch(a, lda, m_dev, M_cap, w, act_dtype, epilogue, epi, y, ldy,
                        static_cast<cudaStream_t>(stream));
}

}  // extern "C"
