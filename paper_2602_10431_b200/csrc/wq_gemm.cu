// Weight-only quantised GEMM on the tcgen05 tensor cores (Sec. 4.1: 4-bit /
// 3-bit integer weights with per-group parameters; the layer's four linears).
//
// The product is computed transposed, D[n, m] = sum_k W[n, k] * A[m, k].  One CTA
// tile is 256 weight rows (two MMA row tiles of 128) x up to 192 tokens:
//   * the packed codes of both row tiles arrive by bulk TMA copies in a ring of
//     their own, are turned into the 16-bit activation format in registers
//     ((code - zero) * scale exactly in fp32, one rounding) and written with
//     tcgen05.st into a ring of tensor-memory slots, from where the MMAs read
//     their A operand;
//   * the tokens' activations arrive by tiled TMA loads into a ring of
//     128-byte-swizzled shared-memory stages (the B operand).  Both row tiles use
//     the same stage, which halves the L2 -> SM traffic per flop; with one row
//     tile per stage the loop is bound by L2 bandwidth (about 72 B/clk/SM), not
//     by the tensor cores;
//   * two fp32 accumulators (128 lanes x TN columns, one per row tile) live in
//     tensor memory and are drained through a transposing shared-memory tile so
//     that every global access of the epilogue is 16 bytes per lane.
// The rings (weights, dequantised A slots, activations) are independent, so the
// dequantisers run ahead of the activation loads instead of lengthening their
// round trip.  The grid is persistent (one CTA per SM) and reads the number of
// executed tokens from device memory: no launch parameter depends on the routing.
//
// Warp roles (640 threads): warps 0 and 2 TMA producers (even / odd K blocks,
// activations and weights), warps 1 and 3 MMA issuers (one per row tile; warp 1
// also allocates tensor memory), warps 4-19 dequantisers and, at the end of a
// tile, epilogue.  The sixteen form four sets of four warps (one TMEM lane
// quadrant each): set (g, h) owns row tile g and the K blocks whose running
// number has parity h, so that one set's "wait for the free slot, store to
// tensor memory, wait for the store" never delays the arithmetic of the next
// block: a single set per row tile needs about 1300 cycles per K block, the
// MMAs of a block 768.  In the epilogue set (g, h) drains every other 16-column
// chunk of accumulator g.
#include <cuda.h>

#include <string.h>

#include "common.cuh"
#include "ptx.cuh"
#include "wq_gemm.cuh"

namespace qtale {

using namespace ptx;

constexpr int kGemmThreads = 640;
constexpr int kPairThreads = 640;
constexpr int kPairFirstDq = 4;    // first dequantiser warp of the CTA-pair kernel
constexpr int kDequantWarps = 16;
constexpr int kTileRows = 128;           // weight rows per tile (MMA M)
constexpr int kKB = 64;                  // K elements per pipeline step (128 B of 16-bit data)
constexpr uint32_t kWaitSliceNs = 20000;  // longest hardware suspension of one barrier test
constexpr uint32_t kWaitSlices = 1u << 16;  // tests before a wait gives up (about a second)
constexpr int kTmemCols = 512;
constexpr int kAColsPerSlot = kKB / 2;   // two 16-bit values per 32-bit TMEM column
constexpr int kEpiCols = 16;             // tokens per epilogue chunk
constexpr int kEpiRowWords = 36;         // padded row (32 fp32 + 4) of the epilogue staging tile
constexpr int kEpiWarpBytes = kEpiCols * kEpiRowWords * 4;
constexpr size_t kSplitTileBytes = (size_t)2 * 128 * 64 * 4;  // one fp32 partial tile: 256 rows x 64 tokens

template <int TN, int BITS>
struct GemmCfg {
  static constexpr int kRowTiles = BITS == 16 ? 1 : 2;    // 128-row weight tiles per CTA tile
  static constexpr int kXBytes = TN * 128;
  // with 16-bit weights the weight tile travels with the activations (both from TMA)
  static constexpr int kXStageBytes = kXBytes + (BITS == 16 ? kTileRows * 128 : 0);
  static constexpr int kXStages = BITS == 16 ? 4 : (TN >= 192 ? 6 : 8);
  static constexpr int kWCodeBytes = BITS == 16 ? 0 : kTileRows * kKB * BITS / 8;
  static constexpr int kSzBytes = BITS == 16 ? 0 : kTileRows * 4;
  static constexpr int kWTileBytes = kWCodeBytes + kSzBytes;       // one row tile, one K block
  static constexpr int kWStageBytes = kRowTiles * kWTileBytes;
  static constexpr int kWStages = BITS == 16 ? 0 : 4;
  static constexpr int kDCols = TN;                                // columns of one accumulator
  static constexpr int kAColBase = kRowTiles * kDCols;             // A slots follow the accumulators
  static constexpr int kAEntriesMax = (kTmemCols - kAColBase) / (kRowTiles * kAColsPerSlot);
  static constexpr int kAEntries = kAEntriesMax > 4 ? 4 : kAEntriesMax;  // K blocks of A in flight
  static constexpr size_t kEpiOffset = (size_t)kXStages * kXStageBytes + (size_t)kWStages * kWStageBytes;
  static constexpr size_t kSmemBytes = kEpiOffset + kDequantWarps * kEpiWarpBytes + 1024;
  static_assert(kXStageBytes % 1024 == 0, "swizzled stages must stay 1024-byte aligned");
  static_assert(BITS == 16 || kWTileBytes % 16 == 0, "bulk copies need 16-byte granularity");
  static_assert(BITS == 16 || kAEntries >= 2, "TMEM budget");
  static_assert(BITS == 16 || (kAEntries % 2 == 0 && kWStages % 2 == 0),
                "a ring slot must always meet the same parity of the running K block number");
  static_assert(kSmemBytes <= 232448 - 512, "shared memory budget");
};

// Activation tensor maps for token tiles of 32, 64, ... , 192 rows (index w / 32 - 1).
struct TmapSet {
  CUtensorMap m[6];
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
  const float2* rope_cs;   // ROPE epilogue: (cos, sin) [M_cap, rope_hd / 2]
  int rope_hd;             // head dim of the rotary layout (ROPE row modes), else 0
  int rope_limit;          // output features below this are rotated (query and key heads)
  int split_k;             // single-CTA kernel: K slices per output tile (1: none)
  float* partial;          // split_k > 1: fp32 partial tiles [tile][slice][256 rows][TN tokens]
  int* tickets;            // split_k > 1: one counter per output tile, zero at launch
  int* status;
};

struct __align__(8) GemmShared {
  uint64_t full_x[8], empty_x[8];  // activation ring
  uint64_t full_w[8], empty_w[8];  // packed-weight ring
  uint64_t a_full[2][4], a_empty[2][4];  // dequantised A slots in tensor memory, per row tile
  uint64_t d_full[2], d_empty[2];        // the accumulators, per row tile
  uint32_t tmem_base;
  volatile int abort_flag;
  uint64_t part_bar;  // split K: all warps have written their part of the partial tile
};

// Bounded wait: gives up after kWaitSlices suspended tests, records a timeout and raises
// the CTA-wide abort flag so that every role leaves its loop.
__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, GemmShared* sh,
                                              int* status) {
  if (mbar_try_wait(bar, parity)) return true;
  for (uint32_t it = 0; it < kWaitSlices; ++it) {
    if (mbar_try_wait_suspend(bar, parity, kWaitSliceNs)) return true;
    if (sh->abort_flag) return false;
  }
  sh->abort_flag = 1;
  report_device_error(status, QTALE_ERR_TIMEOUT);
  return false;
}

// logical output feature of lane L of tile nt (-1: padding row)
// feature (inside a tile's block of heads) of element e of the rotary row layout: head e / half,
// offset e % half, with half = rope_hd / 2 a power of two (no integer division in the epilogues)
__device__ __forceinline__ int rope_first_half_feature(int e, int rope_hd) {
  const int half = rope_hd >> 1;
  return ((e & ~(half - 1)) << 1) + (e & (half - 1));
}

__device__ __forceinline__ int tile_row_to_n(const GemmParams& p, int nt, int L) {
  if (p.row_mode == QTALE_WQ_ROWS_SWIGLU) {
    const int q = L >> 5, r = L & 31;
    const int j = nt * 64 + q * 16 + (r & 15);
    if (j >= p.F) return -1;
    return (r < 16) ? j : p.F + j;
  }
  if (p.rope_hd) {
    // rotary layout: a lane quadrant holds 16 features of the first half of a head (lanes 0-15)
    // and their partners half a head further (lanes 16-31)
    const int q = L >> 5, r = L & 31, half = p.rope_hd >> 1;
    const int e = q * 16 + (r & 15);
    const int n = nt * kTileRows + rope_first_half_feature(e, p.rope_hd) + (r < 16 ? 0 : half);
    return n < p.N ? n : -1;
  }
  const int n = nt * kTileRows + L;
  return n < p.N ? n : -1;
}

// Eight codes sitting in the 4-bit slots of `t` -> four packed 16-bit pairs.
// Slot i holds, in its low QBITS bits, the code of input feature 2i (i < 4) or
// 2(i-4)+1 (i >= 4) of the word's eight features, so slots i and i+4 form the
// pair that shares a 32-bit TMEM column.
//
// Generic path (bf16 output): the code is moved into a float mantissa next to
// 2^23, so (float - (2^23 + zero * 16^i)) * (scale / 16^i) is exactly
// (code - zero) * scale in fp32, rounded once.
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
  for (int q = 0; q < 4; ++q) out[q] = Act16<ACT>::pack(v[q], v[q + 4]);
}

// fp16 path: two codes at a time in packed half arithmetic.  0x6400 | code is the
// half 1024 + code (1024 + 16 code for a code in bits 4-7); subtracting 1024 + zero
// (or one fused multiply-add by 1/16 and -(64 + zero)) leaves the exact integer
// code - zero, and the product with the fp16 scale is rounded once: the same value
// as rounding the exact fp32 product.
__device__ __forceinline__ uint32_t h2_sub(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("sub.rn.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}
__device__ __forceinline__ uint32_t h2_mul(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}
__device__ __forceinline__ uint32_t h2_fma(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t r;
  asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
  return r;
}
template <uint32_t QMASK>
__device__ __forceinline__ void dequant8_f16(uint32_t t, uint32_t z_lo, uint32_t z_hi,
                                             uint32_t scale2, uint32_t* out) {
  constexpr uint32_t MAGIC = 0x64006400u;        // (1024, 1024)
  constexpr uint32_t M0 = QMASK * 0x00010001u;   // codes in bits 0-3 of each half
  constexpr uint32_t M1 = M0 << 4;               // codes in bits 4-7 of each half
  constexpr uint32_t SIXTEENTH = 0x2C002C00u;    // (1/16, 1/16)
  const uint32_t t8 = t >> 8;
  out[0] = h2_mul(h2_sub((t & M0) | MAGIC, z_lo), scale2);               // slots 0, 4
  out[1] = h2_mul(h2_fma((t & M1) | MAGIC, SIXTEENTH, z_hi), scale2);    // slots 1, 5
  out[2] = h2_mul(h2_sub((t8 & M0) | MAGIC, z_lo), scale2);              // slots 2, 6
  out[3] = h2_mul(h2_fma((t8 & M1) | MAGIC, SIXTEENTH, z_hi), scale2);   // slots 3, 7
}

struct Ring {
  int s = 0;
  uint32_t ph = 0;
  __device__ __forceinline__ void advance(int n) {
    if (++s == n) { s = 0; ph ^= 1u; }
  }
};

// ---- epilogue of one 16-column chunk, run by one warp on its 32 weight rows ----
// `stage` holds the chunk transposed: stage[m * kEpiRowWords + lane_n] = D[lane_n, m].
// Each lane then owns 8 consecutive output features of one token row, so global
// accesses are 16 bytes per lane and 64 or 128 contiguous bytes per row.
//
// What an epilogue reads from global memory (residual rows, rotary table, token indices) is
// fetched by epilogue_fetch into an EpiOperands, separately from epilogue_chunk which uses it,
// so that a kernel can issue the loads before it waits for the accumulator columns.  (Fetching
// one whole chunk ahead measured the same: the epilogue is bound by instruction issue.)
constexpr int kRowGroups = kEpiCols / 8;
struct EpiOperands {
  uint4 q[4];            // ROPE: (cos, sin) x 8; RESID_F32: bf16 rows of both row groups (q[0], q[1]);
                         // RESID_SCATTER: fp32 rows, two 16-byte halves per row group
  int tok[kRowGroups];   // token index of the lane's row in each row group (RESID epilogues)
};

// EPI template argument of the epilogue helpers: the epilogue if the kernel is compiled for one
// (the CTA-pair kernel: the unused branches and their registers disappear), -1 to read p.epilogue
template <int EPI>
__device__ __forceinline__ int epilogue_kind(const GemmParams& p) {
  return EPI >= 0 ? EPI : p.epilogue;
}
template <int EPI>
__device__ __forceinline__ bool epilogue_gathers(const GemmParams& p) {
  return epilogue_kind<EPI>(p) == QTALE_EPI_RESID_F32 || epilogue_kind<EPI>(p) == QTALE_EPI_RESID_SCATTER;
}
// first output feature of the lane's eight in the plain / residual epilogues (-1: padding)
__device__ __forceinline__ int epilogue_n0(const GemmParams& p, int lane, int nt, int quad) {
  return tile_row_to_n(p, nt, quad * 32 + (lane & 3) * 8);
}
// token indices of the lane's rows of the chunk starting at m0 (RESID epilogues)
template <int EPI>
__device__ __forceinline__ void epilogue_fetch_tok(const GemmParams& p, int lane, int m0, int M,
                                                   EpiOperands& o) {
  if (!epilogue_gathers<EPI>(p)) return;  // uniform over the warp: the shuffles below need all lanes
  int my_row = 0;
  if (lane < kEpiCols && m0 + lane < M) my_row = __ldg(p.idx + m0 + lane);
#pragma unroll
  for (int i = 0; i < kRowGroups; ++i) o.tok[i] = __shfl_sync(0xffffffffu, my_row, i * 8 + (lane >> 2));
}
// the operands themselves (o.tok must be there already)
template <int EPI>
__device__ __forceinline__ void epilogue_fetch(const GemmParams& p, int lane, int nt, int quad, int m0,
                                               int M, EpiOperands& o) {
  const int epi = epilogue_kind<EPI>(p);
  if (epi == QTALE_EPI_ROPE) {
    const int half = p.rope_hd >> 1;
    const int e0 = quad * 16 + (lane & 1) * 8;
    const int f_lo = nt * kTileRows + rope_first_half_feature(e0, p.rope_hd);
    const int m = m0 + (lane >> 1);
    if (f_lo < p.N && f_lo < p.rope_limit && m < M) {
      const uint4* t = reinterpret_cast<const uint4*>(p.rope_cs + (size_t)m * half + (e0 & (half - 1)));
#pragma unroll
      for (int e = 0; e < 4; ++e) o.q[e] = __ldg(t + e);  // (c, s) x 8
    }
    return;
  }
  if (!epilogue_gathers<EPI>(p)) return;
  const int n0 = epilogue_n0(p, lane, nt, quad);
  if (n0 < 0) return;
#pragma unroll
  for (int i = 0; i < kRowGroups; ++i) {
    const int m = m0 + i * 8 + (lane >> 2);
    if (m >= M) continue;
    if (epi == QTALE_EPI_RESID_F32) {
      o.q[i] = ld_nc_16(static_cast<const unsigned short*>(p.resid) + (size_t)o.tok[i] * p.ld_resid + n0);
    } else {
      const uint4* r = reinterpret_cast<const uint4*>(static_cast<const float*>(p.resid) +
                                                      (size_t)m * p.ld_resid + n0);
      o.q[2 * i] = __ldg(r);
      o.q[2 * i + 1] = __ldg(r + 1);
    }
  }
}

template <int ACT, int EPI>
__device__ __forceinline__ void epilogue_chunk(const GemmParams& p, const float* stage, int lane,
                                               int nt, int quad, int m0, int M, const EpiOperands& o) {
  const int epi = epilogue_kind<EPI>(p);
  if (epi == QTALE_EPI_SWIGLU) {
    // lanes n = 0..15 of the chunk are gate rows, n = 16..31 the matching up rows
    const int jc = (lane & 1) * 8;
    const int j0 = nt * 64 + quad * 16 + jc;
    if (j0 >= p.F) return;
    const int row = lane >> 1;
    const int m = m0 + row;
    if (m >= M) return;
    const float4 g0 = *reinterpret_cast<const float4*>(stage + row * kEpiRowWords + jc);
    const float4 g1 = *reinterpret_cast<const float4*>(stage + row * kEpiRowWords + jc + 4);
    const float4 u0 = *reinterpret_cast<const float4*>(stage + row * kEpiRowWords + 16 + jc);
    const float4 u1 = *reinterpret_cast<const float4*>(stage + row * kEpiRowWords + 16 + jc + 4);
    const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
    const float u[8] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
    uint32_t w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e)
      // SiLU(g) u with the approximate reciprocal (2 ulp, far below the 16-bit rounding that
      // follows): the exact division is a dozen instructions per value in an epilogue that is
      // bound by instruction issue
      w[e] = Act16<ACT>::pack(__fdividef(g[2 * e], 1.f + __expf(-g[2 * e])) * u[2 * e],
                              __fdividef(g[2 * e + 1], 1.f + __expf(-g[2 * e + 1])) * u[2 * e + 1]);
    st_16(static_cast<unsigned short*>(p.y) + (size_t)m * p.ldy + j0, make_uint4(w[0], w[1], w[2], w[3]));
    return;
  }
  if (epi == QTALE_EPI_ROPE) {
    // lanes n = 0..15 of the chunk hold features of the first half of a head, n = 16..31 their
    // partners: (x1, x2) -> (x1 cos - x2 sin, x2 cos + x1 sin) at the token's position, formed
    // from the fp32 accumulators and rounded once; value heads are stored as they are
    const int jc = (lane & 1) * 8;
    const int half = p.rope_hd >> 1;
    const int e0 = quad * 16 + jc;
    const int f_lo = nt * kTileRows + rope_first_half_feature(e0, p.rope_hd);
    const int row = lane >> 1;
    const int m = m0 + row;
    if (f_lo >= p.N || m >= M) return;
    const float4 a0 = *reinterpret_cast<const float4*>(stage + row * kEpiRowWords + jc);
    const float4 a1 = *reinterpret_cast<const float4*>(stage + row * kEpiRowWords + jc + 4);
    const float4 b0 = *reinterpret_cast<const float4*>(stage + row * kEpiRowWords + 16 + jc);
    const float4 b1 = *reinterpret_cast<const float4*>(stage + row * kEpiRowWords + 16 + jc + 4);
    float x1[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
    float x2[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
    if (f_lo < p.rope_limit) {
      const uint32_t t[16] = {o.q[0].x, o.q[0].y, o.q[0].z, o.q[0].w, o.q[1].x, o.q[1].y, o.q[1].z, o.q[1].w,
                              o.q[2].x, o.q[2].y, o.q[2].z, o.q[2].w, o.q[3].x, o.q[3].y, o.q[3].z, o.q[3].w};
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float c = __uint_as_float(t[2 * e]), sn = __uint_as_float(t[2 * e + 1]);
        const float u = x1[e], v = x2[e];
        x1[e] = u * c - v * sn;
        x2[e] = v * c + u * sn;
      }
    }
    unsigned short* y = static_cast<unsigned short*>(p.y) + (size_t)m * p.ldy + f_lo;
    st_16(y, make_uint4(Act16<ACT>::pack(x1[0], x1[1]), Act16<ACT>::pack(x1[2], x1[3]),
                        Act16<ACT>::pack(x1[4], x1[5]), Act16<ACT>::pack(x1[6], x1[7])));
    st_16(y + half, make_uint4(Act16<ACT>::pack(x2[0], x2[1]), Act16<ACT>::pack(x2[2], x2[3]),
                               Act16<ACT>::pack(x2[4], x2[5]), Act16<ACT>::pack(x2[6], x2[7])));
    return;
  }
  const int nc = (lane & 3) * 8;
  const int n0 = epilogue_n0(p, lane, nt, quad);  // 8 consecutive features, all valid or none
  if (n0 < 0) return;
#pragma unroll
  for (int i = 0; i < kRowGroups; ++i) {
    const int row = i * 8 + (lane >> 2);
    const int m = m0 + row;
    if (m >= M) continue;
    const float4 a0 = *reinterpret_cast<const float4*>(stage + row * kEpiRowWords + nc);
    const float4 a1 = *reinterpret_cast<const float4*>(stage + row * kEpiRowWords + nc + 4);
    float v[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
    if (epi == QTALE_EPI_STORE_16) {
      st_16(static_cast<unsigned short*>(p.y) + (size_t)m * p.ldy + n0,
            make_uint4(Act16<ACT>::pack(v[0], v[1]), Act16<ACT>::pack(v[2], v[3]),
                       Act16<ACT>::pack(v[4], v[5]), Act16<ACT>::pack(v[6], v[7])));
    } else if (epi == QTALE_EPI_STORE_F32 || epi == QTALE_EPI_RESID_F32) {
      if (epi == QTALE_EPI_RESID_F32) {
        const uint32_t w[4] = {o.q[i].x, o.q[i].y, o.q[i].z, o.q[i].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          v[2 * e] += bf16_lo(w[e]);
          v[2 * e + 1] += bf16_hi(w[e]);
        }
      }
      float* y = static_cast<float*>(p.y) + (size_t)m * p.ldy + n0;
      st_16(y, make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]),
                          __float_as_uint(v[3])));
      st_16(y + 4, make_uint4(__float_as_uint(v[4]), __float_as_uint(v[5]), __float_as_uint(v[6]),
                              __float_as_uint(v[7])));
    } else {  // QTALE_EPI_RESID_SCATTER: x[idx[m]] = bf16(u + acc)   (Eq. 3)
      const uint4 r0 = o.q[2 * i], r1 = o.q[2 * i + 1];
      const float r[8] = {__uint_as_float(r0.x), __uint_as_float(r0.y), __uint_as_float(r0.z),
                          __uint_as_float(r0.w), __uint_as_float(r1.x), __uint_as_float(r1.y),
                          __uint_as_float(r1.z), __uint_as_float(r1.w)};
      st_16(static_cast<unsigned short*>(p.dst) + (size_t)o.tok[i] * p.ld_dst + n0,
            make_uint4(pack_bf16x2(v[0] + r[0], v[1] + r[1]), pack_bf16x2(v[2] + r[2], v[3] + r[3]),
                       pack_bf16x2(v[4] + r[4], v[5] + r[5]), pack_bf16x2(v[6] + r[6], v[7] + r[7])));
    }
  }
}

// Split K: sum of the S partial tiles' 16 columns of one row (slice order, so the result does not
// depend on timing), written transposed into the warp's staging tile.  Four slices (sixteen
// 16-byte loads) are requested at a time.
__device__ __forceinline__ void splitk_sum_to_stage(const float* part, int S, size_t slice_stride,
                                                 float* stage, int lane) {
  float acc[kEpiCols];
#pragma unroll
  for (int c = 0; c < kEpiCols; ++c) acc[c] = 0.f;
  constexpr int kBatch = 4;
#pragma unroll 1
  for (int sl0 = 0; sl0 < S; sl0 += kBatch) {
    float4 v[kBatch][kEpiCols / 4];
#pragma unroll
    for (int b = 0; b < kBatch; ++b) {
      const float4* src = reinterpret_cast<const float4*>(part + (size_t)min(sl0 + b, S - 1) * slice_stride);
#pragma unroll
      for (int q4 = 0; q4 < kEpiCols / 4; ++q4) v[b][q4] = __ldcg(src + q4);
    }
#pragma unroll
    for (int b = 0; b < kBatch; ++b) {
      if (sl0 + b < S) {
#pragma unroll
        for (int q4 = 0; q4 < kEpiCols / 4; ++q4) {
          acc[4 * q4] += v[b][q4].x; acc[4 * q4 + 1] += v[b][q4].y;
          acc[4 * q4 + 2] += v[b][q4].z; acc[4 * q4 + 3] += v[b][q4].w;
        }
      }
    }
  }
#pragma unroll
  for (int c = 0; c < kEpiCols; ++c) stage[c * kEpiRowWords + lane] = acc[c];
}

template <int TN, int BITS, int ACT, bool SPLIT>
__global__ void __launch_bounds__(kGemmThreads, 1)
    wq_gemm_kernel(const __grid_constant__ TmapSet tmaps_x,
                   const __grid_constant__ CUtensorMap tmap_w, const GemmParams p) {
  using Cfg = GemmCfg<TN, BITS>;
  constexpr int SX = Cfg::kXStages;
  constexpr int SW = Cfg::kWStages;
  constexpr int SA = Cfg::kAEntries;
  constexpr int RT = Cfg::kRowTiles;  // weight row tiles (of 128) sharing one activation tile
  extern __shared__ unsigned char smem_dyn[];
  __shared__ GemmShared sh;
  unsigned char* x_base = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
  unsigned char* w_base = x_base + (size_t)SX * Cfg::kXStageBytes;
  float* epi_base = reinterpret_cast<float*>(x_base + Cfg::kEpiOffset);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < 8; ++s) {
      mbar_init(&sh.full_x[s], 1);
      mbar_init(&sh.empty_x[s], 2);  // released by both MMA issuers
      mbar_init(&sh.full_w[s], 1);
      mbar_init(&sh.empty_w[s], 8);
    }
    for (int r = 0; r < 2; ++r) {
      for (int s = 0; s < 4; ++s) {
        mbar_init(&sh.a_full[r][s], 4);
        mbar_init(&sh.a_empty[r][s], 1);
      }
      mbar_init(&sh.d_full[r], 1);
      mbar_init(&sh.d_empty[r], 8);
    }
    mbar_init(&sh.part_bar, kDequantWarps);
    sh.abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(&sh.tmem_base, kTmemCols);
    tmem_relinquish();
  }
  if (warp == 0 && lane == 0) {
    if (BITS == 16) prefetch_tmap(&tmap_w);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sh.tmem_base;

  int M = p.M_cap;
  if (p.m_dev) M = min(M, *p.m_dev);
  M = max(M, 0);
  const int n_rp = (p.n_tiles + RT - 1) / RT;  // groups of RT row tiles
  const int nkb = p.nkb;
  // Token-tile width: the multiple of 32 (at most TN) that minimises
  // (waves of the persistent grid) x (columns per tile + fixed per-tile cost), so
  // that a tile count just above a multiple of the grid does not cost a whole wave.
  int TW = TN;
  {
    // per-tile time in columns of MMA work: the K loop costs max(w, 128) per block (below
    // about 128 tokens the dequantisers, not the MMAs, set the pace) plus epilogue / restart
    const int fixed = 1408 / max(nkb, 1);
    long best = -1;
    for (int w = TN; w >= 32; w -= 32) {
      const long tiles = (long)((M + w - 1) / w) * n_rp;
      const long cost = ((tiles + gridDim.x - 1) / gridDim.x) * (max(w, 128) + fixed);
      if (best < 0 || cost < best) { best = cost; TW = w; }
    }
  }
  if (SPLIT) TW = TN;  // partial tiles are laid out for one full-width token tile
  const CUtensorMap* tmap_x = &tmaps_x.m[TW / 32 - 1];
  // tile index = mt * n_rp + rp: CTAs running at the same time share a few token tiles and
  // sweep the (small, L2-resident) packed weights, so activations stream from HBM once
  const int n_mt = (M + TW - 1) / TW;
  // Split K (token counts of a decode step): a tile is (token tile, K slice, row-tile group);
  // every slice leaves an fp32 partial tile in global memory and counts itself in; when a CTA
  // has done all its tiles it sums its share of each output tile it took part in.
  const int S = SPLIT ? max(p.split_k, 1) : 1;
  const int total_tiles = n_mt * n_rp * S;
  auto tile_coords = [&](int tile, int& rp, int& mt, int& ks, int& kb0, int& kb1) {
    rp = tile % n_rp;
    const int q = tile / n_rp;
    ks = q % S;
    mt = q / S;
    kb0 = (int)((long)ks * nkb / S);
    kb1 = (int)((long)(ks + 1) * nkb / S);
  };
  const uint32_t x_stage_tx = (uint32_t)TW * 128u + (BITS == 16 ? kTileRows * 128 : 0);

  if (warp == 0 || warp == 2) {
    // ------- TMA producers: warp 0 serves even, warp 2 odd K blocks (activations + weights) -------
    if (lane == 0) {
      const int parity = warp >> 1;
      Ring rx, rw;
      int count = 0;
      for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        int rp, mt, ks, kb0, kb1;
        tile_coords(tile, rp, mt, ks, kb0, kb1);
        for (int kb = kb0; kb < kb1; ++kb, ++count) {
          if ((count & 1) == parity) {
            if (BITS != 16) {
              // one contiguous chunk per (row-tile pair, K block): both tiles' codes, each
              // followed by the scale / zero words of its group
              if (!wait_or_abort(&sh.empty_w[rw.s], rw.ph ^ 1u, &sh, p.status)) goto x_done;
              mbar_arrive_expect_tx(&sh.full_w[rw.s], Cfg::kWStageBytes);
              bulk_load(w_base + (size_t)rw.s * Cfg::kWStageBytes,
                        p.packed + ((size_t)rp * nkb + kb) * Cfg::kWStageBytes, Cfg::kWStageBytes,
                        &sh.full_w[rw.s]);
            }
            if (!wait_or_abort(&sh.empty_x[rx.s], rx.ph ^ 1u, &sh, p.status)) goto x_done;
            unsigned char* st = x_base + (size_t)rx.s * Cfg::kXStageBytes;
            mbar_arrive_expect_tx(&sh.full_x[rx.s], x_stage_tx);
            tma_load_2d(st, tmap_x, &sh.full_x[rx.s], kb * kKB, mt * TW);
            if (BITS == 16)
              tma_load_2d(st + Cfg::kXBytes, &tmap_w, &sh.full_x[rx.s], kb * kKB, rp * kTileRows);
          }
          rx.advance(SX);
          rw.advance(SW);
        }
      }
    x_done:;
    }
  } else if (warp == 1 || warp == 3) {
    // ---- MMA issuers: warp 1 drives row tile 0, warp 3 row tile 1; they share the activation
    // ---- stages and are otherwise independent (own A slots, own accumulator).  The tensor
    // ---- core's queue is only a few MMAs deep, so the waits, fence and commits of one issuer
    // ---- are covered by the MMAs of the other.
    if (lane == 0) {
      const int r = warp >> 1;
      const uint32_t idesc = idesc_16bit_f32(kTileRows, TW, ACT == 1);
      const uint32_t d_tmem = tmem_base + r * Cfg::kDCols;
      Ring rx, ra;
      uint32_t dph = 0;
      for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        int rp, mt_, ks_, kb0, kb1;
        tile_coords(tile, rp, mt_, ks_, kb0, kb1);
        const bool has_tile = r < RT && rp * RT + r < p.n_tiles;
        // the accumulator is free once the previous tile has been drained
        if (!wait_or_abort(&sh.d_empty[r], dph ^ 1u, &sh, p.status)) goto mma_done;
        tc_fence_after();
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!wait_or_abort(&sh.full_x[rx.s], rx.ph, &sh, p.status)) goto mma_done;
          if (BITS != 16) {
            if (!wait_or_abort(&sh.a_full[r][ra.s], ra.ph, &sh, p.status)) goto mma_done;
          }
          if (has_tile) {
            tc_fence_after();
            unsigned char* st = x_base + (size_t)rx.s * Cfg::kXStageBytes;
            const uint64_t b_desc = smem_desc_sw128(smem_u32(st));
#pragma unroll
            for (int j = 0; j < kKB / 16; ++j) {
              const uint32_t acc = (kb != kb0 || j != 0) ? 1u : 0u;
              if (BITS == 16) {
                const uint64_t a_desc = smem_desc_sw128(smem_u32(st + Cfg::kXBytes));
                mma_ss(d_tmem, a_desc + 2u * j, b_desc + 2u * j, idesc, acc);
              } else {
                mma_ts(d_tmem,
                       tmem_base + Cfg::kAColBase + (ra.s * RT + r) * kAColsPerSlot + j * 8,
                       b_desc + 2u * j, idesc, acc);
              }
            }
            mma_commit(&sh.empty_x[rx.s]);                      // one of the two releases of the stage
            if (BITS != 16) mma_commit(&sh.a_empty[r][ra.s]);   // frees this row tile's A slot
          } else {
            // nothing to multiply for this row tile: keep the handshakes in step
            mbar_arrive(&sh.empty_x[rx.s]);
            if (BITS != 16) mbar_arrive(&sh.a_empty[r][ra.s]);
          }
          rx.advance(SX);
          ra.advance(SA);
        }
        if (has_tile) mma_commit(&sh.d_full[r]); else mbar_arrive(&sh.d_full[r]);
        dph ^= 1u;
      }
    mma_done:;
    }
  } else {
    // ---- dequantisers, then epilogue: set (g, h) owns row tile g and the K blocks of parity h ----
    const int quad = warp & 3;
    const int L = quad * 32 + lane;
    const int g = ((warp - 4) >> 2) & 1;
    const int h = (warp - 4) >> 3;
    float* stage = epi_base + (size_t)(warp - 4) * (kEpiWarpBytes / 4);
    Ring rw, ra;
    uint32_t dph = 0;
    int count = 0;  // running K block number, as in the producers
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
      int rp, mt, ks, kb0, kb1;
      tile_coords(tile, rp, mt, ks, kb0, kb1);
      const int nt = rp * RT + g;
      const bool has_tile = g < RT && nt < p.n_tiles;
      if (BITS != 16) {
        for (int kb = kb0; kb < kb1; ++kb, ++count) {
          if ((count & 1) != h) {  // the other set's block (ring slots alternate with the parity)
            rw.advance(SW);
            ra.advance(SA);
            continue;
          }
          uint32_t cw[8];
          uint32_t sz = 0;
          // every warp of the set, with or without a tile, takes part in each handshake once
          if (!wait_or_abort(&sh.full_w[rw.s], rw.ph, &sh, p.status)) goto role_done;
          if (has_tile) {
            const unsigned char* st = w_base + (size_t)rw.s * Cfg::kWStageBytes + g * Cfg::kWTileBytes;
            sz = reinterpret_cast<const uint32_t*>(st + Cfg::kWCodeBytes)[L];
            if (BITS == 4) {
              const uint4 w0 = reinterpret_cast<const uint4*>(st)[L];
              const uint4 w1 = reinterpret_cast<const uint4*>(st)[kTileRows + L];
              cw[0] = w0.x; cw[1] = w0.y; cw[2] = w0.z; cw[3] = w0.w;
              cw[4] = w1.x; cw[5] = w1.y; cw[6] = w1.z; cw[7] = w1.w;
            } else {
              // 3-bit: a 2-bit plane and a 1-bit plane; 2-bit: the 2-bit plane alone
              const uint4 a = reinterpret_cast<const uint4*>(st)[L];
              uint2 b = make_uint2(0, 0);
              if (BITS == 3) b = reinterpret_cast<const uint2*>(st + kTileRows * 16)[L];
              cw[0] = a.x; cw[1] = a.y; cw[2] = a.z; cw[3] = a.w;
              cw[4] = b.x; cw[5] = b.y; cw[6] = 0; cw[7] = 0;
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(&sh.empty_w[rw.s]);
          // The first half of the block (32 input features) is dequantised before the wait for
          // the free A slot, the second half while the first half's store is in flight.
          uint32_t r[16];
          float C[5], Sc[5];
          uint32_t z_lo = 0, z_hi = 0, scale2 = 0;
          if (ACT == 1) {
            const uint32_t zero2 = (sz >> 16) * 0x00010001u;          // (zero, zero) as halves
            scale2 = (sz & 0xFFFFu) * 0x00010001u;
            z_lo = h2_sub(zero2, 0xE400E400u);                        // zero - (-1024) = 1024 + zero
            z_hi = h2_sub(0xD400D400u, zero2);                        // -64 - zero
          } else {
            const float scale = __half2float(__ushort_as_half((unsigned short)(sz & 0xFFFFu)));
            const float zero = __half2float(__ushort_as_half((unsigned short)(sz >> 16)));
#pragma unroll
            for (int i = 0; i < 5; ++i) {
              C[i] = 8388608.f + zero * (float)(1 << (4 * i));
              Sc[i] = scale * (1.f / (float)(1 << (4 * i)));
            }
          }
          auto dequant_half = [&](int half) {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              const int u = half * 4 + v;
              uint32_t t;
              if (BITS == 4) {
                t = cw[u];
              } else {
                // 3-bit: low two bits of 16 codes per word (plane A: cw[0..3]), high bit of 32
                // codes per word (plane B: cw[4..5]).  A nibble-style word with the code in
                // the low 3 bits of each 4-bit slot is assembled with one bitwise select.
                const uint32_t a2 = (u & 1) ? (cw[u >> 1] >> 2) : cw[u >> 1];
                const int rr = u & 3;
                const uint32_t bw = cw[4 + (u >> 2)];
                const uint32_t b1 = rr == 0 ? (bw << 2) : rr == 1 ? (bw << 1) : rr == 2 ? bw : (bw >> 1);
                t = (a2 & 0x33333333u) | (b1 & 0xCCCCCCCCu);
              }
              constexpr uint32_t QM = BITS == 4 ? 0xFu : 0x7u;
              if (ACT == 1) dequant8_f16<QM>(t, z_lo, z_hi, scale2, r + 4 * v);
              else dequant8<QM, ACT>(t, C, Sc, r + 4 * v);
            }
          };
          if (has_tile) dequant_half(0);
          if (!wait_or_abort(&sh.a_empty[g][ra.s], ra.ph ^ 1u, &sh, p.status)) goto role_done;
          if (has_tile) {
            tc_fence_after();
            const uint32_t a_taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + Cfg::kAColBase +
                                     (ra.s * RT + g) * kAColsPerSlot;
            tmem_st_x16(a_taddr, r);
            dequant_half(1);  // the store has taken its operands: the registers are free again
            tmem_st_x16(a_taddr + kAColsPerSlot / 2, r);
            tmem_wait_st();
            tc_fence_before();
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(&sh.a_full[g][ra.s]);
          rw.advance(SW);
          ra.advance(SA);
        }
      }
      // ---- epilogue of this tile: sets (g, 0) and (g, 1) drain alternate 16-column chunks of
      // ---- accumulator g, one lane quadrant per warp ----
      if (!wait_or_abort(&sh.d_full[g], dph, &sh, p.status)) goto role_done;
      tc_fence_after();
      if (!SPLIT) {
        if (has_tile) {
          const int m_base = mt * TW;
          const uint32_t d_taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + g * Cfg::kDCols;
          uint32_t r[kEpiCols];
          if (m_base + h * kEpiCols < M) tmem_ld_x16(d_taddr + h * kEpiCols, r);
#pragma unroll 1
          for (int c0 = h * kEpiCols; c0 < TW; c0 += 2 * kEpiCols) {
            const int m0 = m_base + c0;
            if (m0 >= M) break;
            tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < kEpiCols; ++c) stage[c * kEpiRowWords + lane] = __uint_as_float(r[c]);
            __syncwarp();
            // the next chunk's accumulator read overlaps this chunk's global traffic
            if (c0 + 2 * kEpiCols < TW && m0 + 2 * kEpiCols < M) tmem_ld_x16(d_taddr + c0 + 2 * kEpiCols, r);
            EpiOperands eo;
            epilogue_fetch_tok<-1>(p, lane, m0, M, eo);
            epilogue_fetch<-1>(p, lane, nt, quad, m0, M, eo);
            epilogue_chunk<ACT, -1>(p, stage, lane, nt, quad, m0, M, eo);
            __syncwarp();
          }
          tmem_wait_ld();
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.d_empty[g]);
      } else {
        // split K: the raw accumulator goes to this slice's partial tile (row L of row tile g,
        // TN tokens per row), then the accumulator is handed back at once
        const int m_base = mt * TW;
        const int out_tile = mt * n_rp + rp;
        float* part = p.partial + ((size_t)out_tile * S) * (2 * kTileRows * TN) +
                      (size_t)(g * kTileRows + L) * TN;
        if (has_tile) {
          const uint32_t d_taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + g * Cfg::kDCols;
          for (int c0 = h * kEpiCols; c0 < TW; c0 += 2 * kEpiCols) {
            if (m_base + c0 >= M) break;
            uint32_t r[kEpiCols];
            tmem_ld_x16(d_taddr + c0, r);
            tmem_wait_ld();
            float4* dst = reinterpret_cast<float4*>(part + (size_t)ks * (2 * kTileRows * TN) + c0);
#pragma unroll
            for (int q4 = 0; q4 < kEpiCols / 4; ++q4)
              dst[q4] = make_float4(__uint_as_float(r[4 * q4]), __uint_as_float(r[4 * q4 + 1]),
                                    __uint_as_float(r[4 * q4 + 2]), __uint_as_float(r[4 * q4 + 3]));
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.d_empty[g]);
        // this slice is there: one arrival per warp on part_bar, then one thread counts it in
        // global memory (the fences order the partial tile before the count)
        __threadfence();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.part_bar);
        if (warp == 4) {
          if (!wait_or_abort(&sh.part_bar, dph, &sh, p.status)) goto role_done;
          if (lane == 0) {
            __threadfence();
            atomicAdd(p.tickets + out_tile, 1);
          }
        }
      }
      dph ^= 1u;
    }
    if (SPLIT) {
      // ---- split K, second half: every CTA has delivered all its partial tiles; now each sums
      // ---- its share of every output tile it took part in.  An output tile is 32 units of
      // ---- (32 weight rows, 16 tokens); slice ks takes the units ks, ks + S, ...; a unit is one
      // ---- warp's work: the S partials are added in slice order (the result does not depend on
      // ---- timing) and go through the usual epilogue.  Waiting only starts here, after all of
      // ---- this CTA's own partials are out, so CTAs cannot wait for each other in a circle.
      const int wi = warp - 4;
      for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        int rp, mt, ks, kb0, kb1;
        tile_coords(tile, rp, mt, ks, kb0, kb1);
        const int out_tile = mt * n_rp + rp;
        {
          const uint32_t* tk = reinterpret_cast<const uint32_t*>(p.tickets + out_tile);
          uint32_t it = 0, seen = 0;
          while (true) {
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(tk) : "memory");
            if (seen >= (uint32_t)S || sh.abort_flag) break;
            if (++it > (1u << 22)) {
              sh.abort_flag = 1;
              report_device_error(p.status, QTALE_ERR_TIMEOUT);
              break;
            }
            __nanosleep(64);
          }
          if (sh.abort_flag) goto role_done;
        }
        const float* tile_part = p.partial + ((size_t)out_tile * S) * (2 * kTileRows * TN);
        for (int u = ks + S * wi; u < 32; u += S * kDequantWarps) {
          const int qi = u >> 2, c0 = (u & 3) * kEpiCols;
          const int g2 = qi >> 2, quad2 = qi & 3;
          const int nt2 = rp * RT + g2;
          const int m0 = mt * TW + c0;
          if (g2 >= RT || nt2 >= p.n_tiles || m0 >= M) continue;  // uniform over the warp
          EpiOperands eo;
          epilogue_fetch_tok<-1>(p, lane, m0, M, eo);
          epilogue_fetch<-1>(p, lane, nt2, quad2, m0, M, eo);
          splitk_sum_to_stage(tile_part + (size_t)(g2 * kTileRows + quad2 * 32 + lane) * TN + c0, S,
                              (size_t)2 * kTileRows * TN, stage, lane);
          __syncwarp();
          epilogue_chunk<ACT, -1>(p, stage, lane, nt2, quad2, m0, M, eo);
          __syncwarp();
        }
      }
    }
  role_done:;
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
// CTA-pair kernel (prefill shapes): one tile = 256 weight rows x up to 256 tokens,
// computed by two CTAs of a cluster with tcgen05.mma.cta_group::2.
//
// Each CTA dequantises its own 128 weight rows into its own tensor memory (A
// operand, ring of 4 slots of 128 input features) and loads its own half of the
// tile's tokens into its own shared memory (B operand, ring of 4 stages of 32 KB);
// a pipeline step is two 64-wide K blocks, so that the single issuing thread and
// the dequantisers pay their barrier traffic once per eight MMAs;
// the pair leader (cluster rank 0) issues the MMAs for both CTAs.  Against the
// single-CTA kernel this halves the B-operand shared-memory reads and the
// activation bytes loaded per flop, makes every dequantised weight serve 256
// tokens instead of 192, and leaves room for 512 input features of dequantised weights
// in flight instead of 128, so the chain "MMA done -> slot free -> store to tensor
// memory -> MMA" is no longer exposed.
//
// Warp roles per CTA (640 threads): warp 0 activation producer, warp 2 weight
// producer, warp 1 MMA issuer (leader only; in both CTAs it allocates tensor memory),
// warp 3 idle, warps 4-19 dequantisers / epilogue in four sets of four warps: set j
// owns the pipeline steps whose running number is j modulo 4, i.e. ring slot j.
//
// Barriers.  slot_free[s] (both CTAs, multicast commit of the leader): activation stage
// s and A slot s have been consumed.  ready[s] (leader): both CTAs' activation loads of
// stage s have landed and both CTAs have stored A slot s, so the issuer tests one barrier
// per step.  full_w / empty_w (local): packed weights.  d_full (both, multicast commit):
// the accumulator is complete.  d_empty (leader): both CTAs have drained it.
// ------------------------------------------------------------------------------
constexpr int kPairStages = 4;           // activation stages = A slots = weight stages
constexpr int kPairBlocks = 2;           // 64-wide K blocks per pipeline step
constexpr int kPairTokens = 256;         // tokens per pair tile (128 per CTA)
constexpr int kPairDCols = kPairTokens;  // accumulator columns

template <int BITS>
struct PairCfg {
  static constexpr int kXBlockBytes = (kPairTokens / 2) * 128;   // one K block of this CTA's tokens
  static constexpr int kXStageBytes = kPairBlocks * kXBlockBytes;
  static constexpr int kWCodeBytes = kTileRows * kKB * BITS / 8;
  static constexpr int kWTileBytes = kWCodeBytes + kTileRows * 4;  // one row tile, one K block
  static constexpr int kWStageBytes = kPairBlocks * kWTileBytes;
  static constexpr int kAColsPerStage = kPairBlocks * kAColsPerSlot;
  static constexpr size_t kWOffset = (size_t)kPairStages * kXStageBytes;
  static constexpr size_t kEpiOffset = kWOffset + (size_t)kPairStages * kWStageBytes;
  static constexpr size_t kSmemBytes = kEpiOffset + kDequantWarps * kEpiWarpBytes + 1024;
  static_assert(kWTileBytes % 16 == 0, "bulk copies need 16-byte granularity");
  static_assert(kPairDCols + kPairStages * kAColsPerStage <= kTmemCols, "TMEM budget");
  static_assert(kPairStages == 4, "ring slot = low two bits of the step count = dequantiser set");
  static_assert(kXBlockBytes % 1024 == 0, "swizzled blocks must stay 1024-byte aligned");
  static_assert(kSmemBytes <= 232448 - 512, "shared memory budget");
};

// Activation tensor maps for per-CTA token boxes of 16, 32, ..., 128 rows (index rows / 16 - 1).
struct PairTmapSet {
  CUtensorMap m[8];
};

struct __align__(8) PairShared {
  uint64_t ready[kPairStages];
  uint64_t slot_free[kPairStages];
  uint64_t full_w[kPairStages], empty_w[kPairStages];
  uint64_t d_full, d_empty;
  uint32_t tmem_base;
  volatile int abort_flag;
};

__device__ __forceinline__ bool pair_wait(uint64_t* bar, uint32_t parity, PairShared* sh, int* status) {
  if (mbar_try_wait(bar, parity)) return true;
  for (uint32_t it = 0; it < kWaitSlices; ++it) {
    if (mbar_try_wait_suspend(bar, parity, kWaitSliceNs)) return true;
    if (sh->abort_flag) return false;
  }
  sh->abort_flag = 1;
  report_device_error(status, QTALE_ERR_TIMEOUT);
  return false;
}

template <int BITS, int ACT, int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
    wq_gemm_pair_kernel(const __grid_constant__ PairTmapSet tmaps_x, const GemmParams p) {
  using Cfg = PairCfg<BITS>;
  constexpr int S = kPairStages;
  extern __shared__ unsigned char smem_dyn[];
  __shared__ PairShared sh;
  unsigned char* x_base = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
  unsigned char* w_base = x_base + Cfg::kWOffset;
  float* epi_base = reinterpret_cast<float*>(x_base + Cfg::kEpiOffset);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // 0: pair leader
  const bool leader = rank == 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(&sh.ready[s], 9);      // the leader's producer (expecting both halves' bytes) and
                                       // four dequantiser warps of each CTA
      mbar_init(&sh.slot_free[s], 1);  // one multicast commit
      mbar_init(&sh.full_w[s], 1);
      mbar_init(&sh.empty_w[s], 4);    // the four warps of the set that read the stage
    }
    mbar_init(&sh.d_full, 1);
    mbar_init(&sh.d_empty, 2 * kDequantWarps);
    sh.abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc_pair(&sh.tmem_base, kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync();  // both CTAs' barriers exist before anything is signalled across the pair
  tc_fence_after();
  const uint32_t tmem_base = sh.tmem_base;

  int M = p.M_cap;
  if (p.m_dev) M = min(M, *p.m_dev);
  M = max(M, 0);
  const int n_rp = (p.n_tiles + 1) / 2;  // pairs of row tiles: one per tile of the CTA pair
  const int nkb = p.nkb;
  const int n_clusters = gridDim.x >> 1;
  const int cluster_id = blockIdx.x >> 1;
  // Token-tile width: the multiple of 32 (at most 256) that minimises (waves of the persistent
  // grid) x (time of a tile).  Below about 224 tokens a pipeline step is paced by the
  // dequantisers and the issuing thread, not by the MMAs, so narrower tiles are not faster.
  int TW = kPairTokens;
  {
    const int fixed = 1408 / max(nkb, 1);
    long best = -1;
    for (int w = kPairTokens; w >= 32; w -= 32) {
      const long tiles = (long)((M + w - 1) / w) * n_rp;
      const long cost = ((tiles + n_clusters - 1) / n_clusters) * (max(w, 224) + fixed);
      if (best < 0 || cost < best) { best = cost; TW = w; }
    }
  }
  const int HW = TW >> 1;  // tokens of this CTA's half
  const CUtensorMap* tmap_x = &tmaps_x.m[HW / 16 - 1];
  const int n_mt = (M + TW - 1) / TW;
  const int total_tiles = n_mt * n_rp;

  const int n_st = (nkb + kPairBlocks - 1) / kPairBlocks;  // pipeline steps per tile

  if (warp == 0) {
    // ---------------- activation producer: this CTA's half of the tile's tokens ----------------
    if (lane == 0) {
      const uint32_t ready_leader = map_to_cta(smem_u32(&sh.ready[0]), 0);
      uint32_t count = 0;
      for (int tile = cluster_id; tile < total_tiles; tile += n_clusters) {
        const int mt = tile / n_rp;
        for (int st = 0; st < n_st; ++st, ++count) {
          const uint32_t s = count & (S - 1), ph = (count >> 2) & 1u;
          const int nb = min(kPairBlocks, nkb - st * kPairBlocks);
          if (!pair_wait(&sh.slot_free[s], ph ^ 1u, &sh, p.status)) goto x_done;
          if (leader) mbar_arrive_expect_tx(&sh.ready[s], (uint32_t)(TW * 128 * nb));  // both halves
          for (int b = 0; b < nb; ++b)
            tma_load_2d_pair(x_base + (size_t)s * Cfg::kXStageBytes + (size_t)b * Cfg::kXBlockBytes, tmap_x,
                             ready_leader + 8u * s, (st * kPairBlocks + b) * kKB, mt * TW + (int)rank * HW);
        }
      }
    x_done:;
    }
  } else if (warp == 2) {
    // ---------------- weight producer: this CTA's row tile ----------------
    if (lane == 0) {
      uint32_t count = 0;
      for (int tile = cluster_id; tile < total_tiles; tile += n_clusters) {
        const int rp = tile % n_rp;
        for (int st = 0; st < n_st; ++st, ++count) {
          const uint32_t s = count & (S - 1), ph = (count >> 2) & 1u;
          const int nb = min(kPairBlocks, nkb - st * kPairBlocks);
          if (!pair_wait(&sh.empty_w[s], ph ^ 1u, &sh, p.status)) goto w_done;
          mbar_arrive_expect_tx(&sh.full_w[s], (uint32_t)(Cfg::kWTileBytes * nb));
          for (int b = 0; b < nb; ++b)
            bulk_load(w_base + (size_t)s * Cfg::kWStageBytes + (size_t)b * Cfg::kWTileBytes,
                      p.packed + (((size_t)rp * nkb + st * kPairBlocks + b) * 2 + rank) * Cfg::kWTileBytes,
                      Cfg::kWTileBytes, &sh.full_w[s]);
        }
      }
    w_done:;
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (pair leader) ----------------
    // One thread, so every instruction's latency is exposed: the loop tests one barrier per
    // step, and tests the next step's barrier before it issues this step's MMAs so that the
    // answer arrives while they are being issued.
    if (leader && lane == 0) {
      const uint32_t idesc = idesc_16bit_f32(256, TW, ACT == 1);
      const uint64_t b_desc0 = smem_desc_sw128(smem_u32(x_base));
      const uint32_t a_tmem0 = tmem_base + kPairDCols;
      const long total_st = (long)((total_tiles - cluster_id + n_clusters - 1) / n_clusters) * n_st;
      uint32_t count = 0;
      uint32_t dph = 0;
      bool ready_now = false;  // the barrier of step `count` is already known to be complete
      for (int tile = cluster_id; tile < total_tiles; tile += n_clusters) {
        if (!pair_wait(&sh.d_empty, dph ^ 1u, &sh, p.status)) goto mma_done;
        for (int st = 0; st < n_st; ++st, ++count) {
          const uint32_t s = count & (S - 1);
          if (!ready_now && !pair_wait(&sh.ready[s], (count >> 2) & 1u, &sh, p.status)) goto mma_done;
          tc_fence_after();
          const uint32_t nxt = count + 1;
          const bool more = (long)nxt < total_st;
          const bool next_ok = more && mbar_try_wait(&sh.ready[nxt & (S - 1)], (nxt >> 2) & 1u);
          const uint64_t b_desc = b_desc0 + (uint64_t)(s * (Cfg::kXStageBytes >> 4));
          const uint32_t a_tmem = a_tmem0 + s * Cfg::kAColsPerStage;
          const bool two = st * kPairBlocks + 1 < nkb;
#pragma unroll
          for (int j = 0; j < kKB / 16; ++j)
            mma_ts_pair(tmem_base, a_tmem + j * 8, b_desc + 2u * j, idesc, (st | j) != 0 ? 1u : 0u);
          if (two) {
#pragma unroll
            for (int j = 0; j < kKB / 16; ++j)
              mma_ts_pair(tmem_base, a_tmem + kAColsPerSlot + j * 8,
                          b_desc + (uint64_t)(Cfg::kXBlockBytes >> 4) + 2u * j, idesc, 1u);
          }
          mma_commit_pair(&sh.slot_free[s], 3);
          ready_now = next_ok;
        }
        mma_commit_pair(&sh.d_full, 3);
        dph ^= 1u;
      }
    mma_done:;
    }
  } else if (warp >= kPairFirstDq) {
    // ---------------- dequantisers, then epilogue ----------------
    // (a warp reaches the tensor-memory lanes 32 (warp % 4) .. + 31; any four consecutive warps
    // cover the four quadrants)
    const int quad = warp & 3;
    const int L = quad * 32 + lane;
    const int set = (warp - kPairFirstDq) >> 2;
    float* stage = epi_base + (size_t)(warp - kPairFirstDq) * (kEpiWarpBytes / 4);
    const uint32_t ready_leader = map_to_cta(smem_u32(&sh.ready[0]), 0);
    const uint32_t d_empty_leader = map_to_cta(smem_u32(&sh.d_empty), 0);
    const uint32_t a_taddr0 =
        tmem_base + ((uint32_t)(quad * 32) << 16) + kPairDCols + set * Cfg::kAColsPerStage;
    const unsigned char* w_stage = w_base + (size_t)set * Cfg::kWStageBytes;
    uint32_t dph = 0;
    uint32_t count = 0;
    // one pipeline step of this set (step `st` of a tile, running number `cnt`): packed weights of
    // ring slot `set` -> 16-bit values -> tensor memory, then the arrival on the leader's barrier
    auto dequant_step = [&](int st, uint32_t cnt) -> bool {
        const uint32_t ph = (cnt >> 2) & 1u;
        const bool two = st * kPairBlocks + 1 < nkb;
        uint32_t cw[kPairBlocks][8];
        uint32_t sz[kPairBlocks];
        if (!pair_wait(&sh.full_w[set], ph, &sh, p.status)) return false;
#pragma unroll
        for (int b = 0; b < kPairBlocks; ++b) {
          const unsigned char* wt = w_stage + (size_t)b * Cfg::kWTileBytes;
          if (b == 0 || two) {
            sz[b] = reinterpret_cast<const uint32_t*>(wt + Cfg::kWCodeBytes)[L];
            if (BITS == 4) {
              const uint4 w0 = reinterpret_cast<const uint4*>(wt)[L];
              const uint4 w1 = reinterpret_cast<const uint4*>(wt)[kTileRows + L];
              cw[b][0] = w0.x; cw[b][1] = w0.y; cw[b][2] = w0.z; cw[b][3] = w0.w;
              cw[b][4] = w1.x; cw[b][5] = w1.y; cw[b][6] = w1.z; cw[b][7] = w1.w;
            } else {
              const uint4 a = reinterpret_cast<const uint4*>(wt)[L];
              uint2 bb = make_uint2(0, 0);
              if (BITS == 3) bb = reinterpret_cast<const uint2*>(wt + kTileRows * 16)[L];
              cw[b][0] = a.x; cw[b][1] = a.y; cw[b][2] = a.z; cw[b][3] = a.w;
              cw[b][4] = bb.x; cw[b][5] = bb.y; cw[b][6] = 0; cw[b][7] = 0;
            }
          } else {
            sz[b] = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) cw[b][i] = 0;
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.empty_w[set]);
        uint32_t r[16];
        // one K block (64 input features of this thread's weight row) in two halves of 16 registers
        auto dequant_half = [&](const uint32_t (&c8)[8], uint32_t szw, int half) {
          float C[5], Sc[5];
          uint32_t z_lo = 0, z_hi = 0, scale2 = 0;
          if (ACT == 1) {
            const uint32_t zero2 = (szw >> 16) * 0x00010001u;          // (zero, zero) as halves
            scale2 = (szw & 0xFFFFu) * 0x00010001u;
            z_lo = h2_sub(zero2, 0xE400E400u);                         // zero - (-1024) = 1024 + zero
            z_hi = h2_sub(0xD400D400u, zero2);                         // -64 - zero
          } else {
            const float scale = __half2float(__ushort_as_half((unsigned short)(szw & 0xFFFFu)));
            const float zero = __half2float(__ushort_as_half((unsigned short)(szw >> 16)));
#pragma unroll
            for (int i = 0; i < 5; ++i) {
              C[i] = 8388608.f + zero * (float)(1 << (4 * i));
              Sc[i] = scale * (1.f / (float)(1 << (4 * i)));
            }
          }
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            const int u = half * 4 + v;
            uint32_t t;
            if (BITS == 4) {
              t = c8[u];
            } else {
              const uint32_t a2 = (u & 1) ? (c8[u >> 1] >> 2) : c8[u >> 1];
              const int rr = u & 3;
              const uint32_t bw = c8[4 + (u >> 2)];
              const uint32_t b1 = rr == 0 ? (bw << 2) : rr == 1 ? (bw << 1) : rr == 2 ? bw : (bw >> 1);
              t = (a2 & 0x33333333u) | (b1 & 0xCCCCCCCCu);
            }
            constexpr uint32_t QM = BITS == 4 ? 0xFu : 0x7u;
            if (ACT == 1) dequant8_f16<QM>(t, z_lo, z_hi, scale2, r + 4 * v);
            else dequant8<QM, ACT>(t, C, Sc, r + 4 * v);
          }
        };
        // the first quarter is dequantised before the wait for the free A slot; every store has
        // taken its operands when it returns, so the registers are reused at once
        dequant_half(cw[0], sz[0], 0);
        if (!pair_wait(&sh.slot_free[set], ph ^ 1u, &sh, p.status)) return false;
        tc_fence_after();
        tmem_st_x16(a_taddr0, r);
        dequant_half(cw[0], sz[0], 1);
        tmem_st_x16(a_taddr0 + 16, r);
        if (two) {
          dequant_half(cw[1], sz[1], 0);
          tmem_st_x16(a_taddr0 + 32, r);
          dequant_half(cw[1], sz[1], 1);
          tmem_st_x16(a_taddr0 + 48, r);
        }
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(ready_leader + 8u * set);
        return true;
    };
    bool prefilled = false;  // this set's first step of the current tile is in tensor memory already
    for (int tile = cluster_id; tile < total_tiles; tile += n_clusters) {
      const int rp = tile % n_rp, mt = tile / n_rp;
      const int nt = rp * 2 + (int)rank;
      for (int st = 0; st < n_st; ++st, ++count) {
        if ((int)(count & 3u) != set) continue;  // ring slot = set
        if (prefilled) {
          prefilled = false;
          continue;
        }
        if (!dequant_step(st, count)) goto role_done;
      }
      // The set's first step of the NEXT tile is dequantised before this tile's epilogue: its ring
      // slot is free as soon as this tile's last use of it has been multiplied, and the issuer
      // then finds all four slots ready the moment the accumulator is handed back, instead of
      // waiting for the dequantisers to restart after the epilogue.
      if (tile + n_clusters < total_tiles) {
        const int st0 = (int)(((uint32_t)set - count) & 3u);  // count = running number of the next tile's step 0
        if (st0 < n_st) {
          if (!dequant_step(st0, count + (uint32_t)st0)) goto role_done;
          prefilled = true;
        }
      }
      // ---- epilogue: set j drains the 16-column chunks j, j + 4, ... of this CTA's accumulator ----
      if (!pair_wait(&sh.d_full, dph, &sh, p.status)) goto role_done;
      tc_fence_after();
      {
        const int m_base = mt * TW;
        const uint32_t d_taddr = tmem_base + ((uint32_t)(quad * 32) << 16);
        uint32_t r[kEpiCols];
        if (set * kEpiCols < TW && m_base + set * kEpiCols < M) tmem_ld_x16(d_taddr + set * kEpiCols, r);
#pragma unroll 1
        for (int c0 = set * kEpiCols; c0 < TW; c0 += 4 * kEpiCols) {
          const int m0 = m_base + c0;
          if (m0 >= M) break;
          // what the chunk reads from global memory is requested before the wait for its accumulator columns
          EpiOperands eo;
          epilogue_fetch_tok<EPI>(p, lane, m0, M, eo);
          epilogue_fetch<EPI>(p, lane, nt, quad, m0, M, eo);
          tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < kEpiCols; ++c) stage[c * kEpiRowWords + lane] = __uint_as_float(r[c]);
          __syncwarp();
          if (c0 + 4 * kEpiCols < TW && m0 + 4 * kEpiCols < M) tmem_ld_x16(d_taddr + c0 + 4 * kEpiCols, r);
          epilogue_chunk<ACT, EPI>(p, stage, lane, nt, quad, m0, M, eo);
          __syncwarp();
        }
        tmem_wait_ld();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(d_empty_leader);
      dph ^= 1u;
    }
  role_done:;
  }

  // teardown: both CTAs are done with tensor memory and with each other's barriers
  tc_fence_before();
  __syncthreads();
  cluster_sync();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

// ------------------------------------------------------------------------------
// Small-M kernel (up to 64 tokens: the decode step).  Here the product is bound by the
// stream of packed weights, and the tcgen05 kernels above, whose dequantised operand makes a
// round trip through tensor memory and three barriers per K block, cannot pull it fast
// enough: a CTA needs about 0.6 us per 64-wide block whatever the token count.  This kernel
// keeps everything in registers: one CTA owns 64 weight rows (half a blob tile) over the
// whole K, eight warps = four 16-row blocks x two K halves (even / odd K blocks), a ninth
// warp feeds an 8-stage ring with bulk copies of the codes and a tiled load of the
// activations; each warp rebuilds its m16n8k16 A fragments from the packed codes (one shift,
// one logic op, one exact subtract, one multiply per pair of weights) and issues warp MMAs
// against ldmatrix-loaded activation fragments.  With 64 to 344 CTAs per linear and two CTAs
// per SM the weight stream is spread over the whole device.
// ------------------------------------------------------------------------------
constexpr int kSmallStages = 8;
constexpr int kSmallMmaWarps = 8;
constexpr int kSmallThreads = (kSmallMmaWarps + 1) * 32;
constexpr int kSmallTokens = 64;  // token capacity

// ROWS = weight rows per CTA (32, 64 or 128: a quarter, a half or a whole blob tile), chosen on
// the host so that a linear gives between one and two CTAs per SM; the eight MMA warps are
// ROWS / 16 row blocks x 8 / (ROWS / 16) K groups (K block kb belongs to group kb modulo that).
template <int BITS, int ROWS>
struct SmallCfg {
  static constexpr int kRowBlocks = ROWS / 16;
  static constexpr int kGroups = kSmallMmaWarps / kRowBlocks;
  static constexpr int kQuads = ROWS / 32;
  static constexpr int kXBytes = kSmallTokens * 128;                   // 64 tokens x 64 k
  static constexpr int kCodeA = ROWS * 16;                             // 16 bytes per row
  static constexpr int kCodeB = BITS == 4 ? ROWS * 16 : (BITS == 3 ? ROWS * 8 : 0);  // second code piece
  static constexpr int kSzBytes = ROWS * 4;
  static constexpr int kWBytes = kCodeA + kCodeB + kSzBytes;
  static constexpr int kTileCodeBytes = kTileRows * kKB * BITS / 8;    // code bytes of a full tile block
  static constexpr int kTileBytes = kTileCodeBytes + kTileRows * 4;
  static constexpr size_t kWOffset = (size_t)kSmallStages * kXBytes;
  static constexpr size_t kSmemBytes = kWOffset + (size_t)kSmallStages * kWBytes + 1024;
  // after the K loop the activation ring is reused: partial sums of the K groups but the first,
  // then the output tile for the epilogue
  static constexpr int kRedBytes = (kGroups - 1) * kRowBlocks * 32 * 32 * 4;
  static constexpr int kOutBytes = kQuads * kSmallTokens * kEpiRowWords * 4;
  static_assert(ROWS == 32 || ROWS == 64 || ROWS == 128, "rows per CTA");
  static_assert(kSmallStages % kGroups == 0, "a ring stage always meets the same K group");
  static_assert(kRedBytes + kOutBytes <= kSmallStages * kXBytes, "epilogue buffers fit the ring");
};

struct __align__(8) SmallShared {
  uint64_t full[kSmallStages], empty[kSmallStages];
  volatile int abort_flag;
};

__device__ __forceinline__ bool small_wait(uint64_t* bar, uint32_t parity, SmallShared* sh, int* status) {
  if (mbar_try_wait(bar, parity)) return true;
  for (uint32_t it = 0; it < kWaitSlices; ++it) {
    if (mbar_try_wait_suspend(bar, parity, kWaitSliceNs)) return true;
    if (sh->abort_flag) return false;
  }
  sh->abort_flag = 1;
  report_device_error(status, QTALE_ERR_TIMEOUT);
  return false;
}

// two weights of one row (the codes in bits 4 t .. 4 t + 3 of both halves of `word`) as a pair of
// 16-bit values: (code - zero) * scale, exact difference, one rounding
template <int BITS, int ACT>
__device__ __forceinline__ uint32_t small_dequant_pair(uint32_t word, int shift, uint32_t z_lo,
                                                       uint32_t scale2, float zero, float scale) {
  constexpr uint32_t QM = BITS == 4 ? 0x000F000Fu : 0x00070007u;
  const uint32_t q = (word >> shift) & QM;
  if (ACT == 1) return h2_mul(h2_sub(q | 0x64006400u, z_lo), scale2);
  return pack_bf16x2(((float)(q & 0xFFFFu) - zero) * scale, ((float)(q >> 16) - zero) * scale);
}

template <int BITS, int ACT, int ROWS>
__global__ void __launch_bounds__(kSmallThreads, 2)
    wq_gemm_small_kernel(const __grid_constant__ CUtensorMap tmap_x, const GemmParams p) {
  using Cfg = SmallCfg<BITS, ROWS>;
  constexpr int S = kSmallStages;
  constexpr int RB = Cfg::kRowBlocks, KG = Cfg::kGroups;
  constexpr int SLICES = kTileRows / ROWS;  // CTAs per blob tile
  extern __shared__ unsigned char smem_dyn[];
  __shared__ SmallShared sh;
  unsigned char* x_base = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
  unsigned char* w_base = x_base + Cfg::kWOffset;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  int M = p.M_cap;
  if (p.m_dev) M = min(M, *p.m_dev);
  if (M <= 0) return;  // every thread: nothing to do
  M = min(M, kSmallTokens);
  const int nt = blockIdx.x / SLICES;     // blob tile
  const int slice = blockIdx.x % SLICES;  // rows ROWS * slice .. of the tile
  const int nkb = p.nkb;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(&sh.full[s], 1);
      mbar_init(&sh.empty[s], RB);  // the warps of the K group that reads the stage
    }
    sh.abort_flag = 0;
    fence_barrier_init();
  }
  __syncthreads();

  if (warp == kSmallMmaWarps) {
    // ---------------- producer ----------------
    if (lane == 0) {
      const uint8_t* tile0 = p.packed + (((size_t)(nt >> 1) * nkb) * 2 + (nt & 1)) * Cfg::kTileBytes;
      for (int kb = 0; kb < nkb; ++kb) {
        const int s = kb & (S - 1);
        const uint32_t ph = (uint32_t)(kb >> 3) & 1u;
        if (!small_wait(&sh.empty[s], ph ^ 1u, &sh, p.status)) break;
        mbar_arrive_expect_tx(&sh.full[s], Cfg::kXBytes + Cfg::kWBytes);
        tma_load_2d(x_base + (size_t)s * Cfg::kXBytes, &tmap_x, &sh.full[s], kb * kKB, 0);
        const uint8_t* blk = tile0 + (size_t)kb * 2 * Cfg::kTileBytes;  // (pair, kb) chunks are two tiles apart
        unsigned char* w = w_base + (size_t)s * Cfg::kWBytes;
        // int4: two 32-feature parts of 16 bytes per row; int3: a 2-bit plane of 16 and a 1-bit
        // plane of 8 bytes per row; either way the second piece starts 2 KB into the block
        bulk_load(w, blk + slice * Cfg::kCodeA, Cfg::kCodeA, &sh.full[s]);
        if (Cfg::kCodeB > 0)
          bulk_load(w + Cfg::kCodeA, blk + kTileRows * 16 + slice * Cfg::kCodeB, Cfg::kCodeB, &sh.full[s]);
        bulk_load(w + Cfg::kCodeA + Cfg::kCodeB, blk + Cfg::kTileCodeBytes + slice * Cfg::kSzBytes,
                  Cfg::kSzBytes, &sh.full[s]);
      }
    }
    return;  // the producer takes no part in the epilogue barriers
  }

  // ---------------- MMA warps ----------------
  const int kgroup = warp / RB;  // K blocks kb with kb % KG == kgroup
  const int rb = warp % RB;      // 16-row block of the CTA's rows
  const int g = lane >> 2, t = lane & 3;
  const int r0 = rb * 16 + g, r1 = r0 + 8;
  float acc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[i][e] = 0.f;
  for (int kb = kgroup; kb < nkb; kb += KG) {
    const int s = kb & (S - 1);
    const uint32_t ph = (uint32_t)(kb >> 3) & 1u;
    if (!small_wait(&sh.full[s], ph, &sh, p.status)) break;
    const unsigned char* w = w_base + (size_t)s * Cfg::kWBytes;
    uint32_t c[2][8];  // eight nibble-style words (8 codes each) of rows r0 and r1
    uint32_t szw[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int r = h ? r1 : r0;
      szw[h] = reinterpret_cast<const uint32_t*>(w + Cfg::kCodeA + Cfg::kCodeB)[r];
      if (BITS == 4) {
        const uint4 a = reinterpret_cast<const uint4*>(w)[r];
        const uint4 b = reinterpret_cast<const uint4*>(w + Cfg::kCodeA)[r];
        c[h][0] = a.x; c[h][1] = a.y; c[h][2] = a.z; c[h][3] = a.w;
        c[h][4] = b.x; c[h][5] = b.y; c[h][6] = b.z; c[h][7] = b.w;
      } else {
        const uint4 a = reinterpret_cast<const uint4*>(w)[r];
        uint2 b = make_uint2(0, 0);
        if (BITS == 3) b = reinterpret_cast<const uint2*>(w + Cfg::kCodeA)[r];
        const uint32_t pa[4] = {a.x, a.y, a.z, a.w};
        const uint32_t pb[2] = {b.x, b.y};
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const uint32_t a2 = (u & 1) ? (pa[u >> 1] >> 2) : pa[u >> 1];
          const int rr = u & 3;
          const uint32_t bw = pb[u >> 2];
          const uint32_t b1 = rr == 0 ? (bw << 2) : rr == 1 ? (bw << 1) : rr == 2 ? bw : (bw >> 1);
          c[h][u] = (a2 & 0x33333333u) | (b1 & 0xCCCCCCCCu);
        }
      }
    }
    uint32_t z_lo[2], scale2[2];
    float zf[2], sf[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const uint32_t zero2 = (szw[h] >> 16) * 0x00010001u;
      scale2[h] = (szw[h] & 0xFFFFu) * 0x00010001u;
      z_lo[h] = h2_sub(zero2, 0xE400E400u);  // 1024 + zero
      zf[h] = __half2float(__ushort_as_half((unsigned short)(szw[h] >> 16)));
      sf[h] = __half2float(__ushort_as_half((unsigned short)(szw[h] & 0xFFFFu)));
    }
    const uint32_t x_stage = smem_u32(x_base + (size_t)s * Cfg::kXBytes);
#pragma unroll
    for (int s16 = 0; s16 < 4; ++s16) {
      // word 2 s16 holds k = 16 s16 .. + 7, word 2 s16 + 1 the next eight; in a word, bits 4 t of
      // the low half are feature 2 t and of the high half feature 2 t + 1
      uint32_t a[4];
      a[0] = small_dequant_pair<BITS, ACT>(c[0][2 * s16], 4 * t, z_lo[0], scale2[0], zf[0], sf[0]);
      a[1] = small_dequant_pair<BITS, ACT>(c[1][2 * s16], 4 * t, z_lo[1], scale2[1], zf[1], sf[1]);
      a[2] = small_dequant_pair<BITS, ACT>(c[0][2 * s16 + 1], 4 * t, z_lo[0], scale2[0], zf[0], sf[0]);
      a[3] = small_dequant_pair<BITS, ACT>(c[1][2 * s16 + 1], 4 * t, z_lo[1], scale2[1], zf[1], sf[1]);
#pragma unroll
      for (int tg2 = 0; tg2 < 4; ++tg2) {
        // matrices: (tokens 16 tg2 .. + 7, k chunk 2 s16), (same tokens, chunk 2 s16 + 1),
        //           (tokens 16 tg2 + 8 .., chunk 2 s16), (.., chunk 2 s16 + 1); 128-byte swizzle
        if (tg2 * 16 >= M) break;  // no executed token in these sixteen (same for the whole CTA)
        const int mi = lane >> 3;
        const int token = tg2 * 16 + (mi >> 1) * 8 + (lane & 7);
        const int chunk = 2 * s16 + (mi & 1);
        uint32_t b[4];
        ldmatrix_x4(x_stage + token * 128 + ((chunk ^ (token & 7)) << 4), b);
        mma_m16n8k16<ACT == 1>(acc[2 * tg2], a, b[0], b[1]);
        mma_m16n8k16<ACT == 1>(acc[2 * tg2 + 1], a, b[2], b[3]);
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sh.empty[s]);
  }
  // ---- the other K groups hand their sums to the first; then the tile goes through the common epilogue ----
  named_barrier(1, kSmallMmaWarps * 32);  // every stage has been read: the ring is free
  float* red = reinterpret_cast<float*>(x_base);
  float* out = reinterpret_cast<float*>(x_base + Cfg::kRedBytes);
  if (kgroup > 0) {
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int e = 0; e < 4; ++e)
        red[((((kgroup - 1) * RB + rb) * 32) + i * 4 + e) * 32 + lane] = acc[i][e];
  }
  named_barrier(1, kSmallMmaWarps * 32);
  if (kgroup == 0) {
    const int ql = rb >> 1;              // quadrant (32 rows) of the CTA's rows
    const int nl = (rb & 1) * 16 + g;    // row inside the quadrant
#pragma unroll
    for (int i = 0; i < 8; ++i) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float v = acc[i][e];
#pragma unroll
        for (int kg = 1; kg < KG; ++kg) v += red[((((kg - 1) * RB + rb) * 32) + i * 4 + e) * 32 + lane];
        const int token = i * 8 + 2 * t + (e & 1);
        out[(ql * kSmallTokens + token) * kEpiRowWords + nl + (e >> 1) * 8] = v;
      }
    }
  }
  named_barrier(1, kSmallMmaWarps * 32);
  // units of (quadrant, 16-token chunk) over the eight warps
  for (int unit = warp; unit < Cfg::kQuads * (kSmallTokens / kEpiCols); unit += kSmallMmaWarps) {
    const int ql = unit % Cfg::kQuads, chunk = unit / Cfg::kQuads;
    const int m0 = chunk * kEpiCols;
    if (m0 < M) {
      EpiOperands eo;
      epilogue_fetch_tok<-1>(p, lane, m0, M, eo);
      epilogue_fetch<-1>(p, lane, nt, slice * Cfg::kQuads + ql, m0, M, eo);
      epilogue_chunk<ACT, -1>(p, out + (ql * kSmallTokens + m0) * kEpiRowWords, lane, nt,
                          slice * Cfg::kQuads + ql, m0, M, eo);
    }
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

// tensor maps for every token-tile width (multiples of 32) up to tn
static int make_tmap_set(TmapSet* set, const void* base, int rows, int cols, int ld, int tn,
                         int act) {
  for (int w = 32; w <= tn; w += 32) {
    const int rc = make_tmap_16(&set->m[w / 32 - 1], base, rows, cols, ld, w, act);
    if (rc != QTALE_OK) return rc;
  }
  return QTALE_OK;
}

template <int TN, int BITS, int ACT, bool SPLIT = false>
static int launch_gemm(const TmapSet& tx, const CUtensorMap& tw, const GemmParams& p,
                       cudaStream_t s) {
  using Cfg = GemmCfg<TN, BITS>;
  static bool configured[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    if (cudaFuncSetAttribute(wq_gemm_kernel<TN, BITS, ACT, SPLIT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)Cfg::kSmemBytes) != cudaSuccess)
      return QTALE_ERR_CUDA;
    configured[dev] = true;
  }
  const int max_tiles = ((p.M_cap + 31) / 32) * ((p.n_tiles + Cfg::kRowTiles - 1) / Cfg::kRowTiles) *
                        (p.split_k > 1 ? p.split_k : 1);
  int grid = sm_count();
  if (grid > max_tiles) grid = max_tiles;
  if (grid < 1) grid = 1;
  wq_gemm_kernel<TN, BITS, ACT, SPLIT><<<grid, kGemmThreads, Cfg::kSmemBytes, s>>>(tx, tw, p);
  return launch_status(cudaGetLastError());
}

template <int BITS, int ACT>
static int dispatch_tn(const TmapSet& tx, const CUtensorMap& tw, const GemmParams& p, int tn,
                       cudaStream_t s) {
  if (tn == 64) return launch_gemm<64, BITS, ACT>(tx, tw, p, s);
  if (tn == 128) return launch_gemm<128, BITS, ACT>(tx, tw, p, s);
  return launch_gemm<192, BITS, ACT>(tx, tw, p, s);
}

// ---- CTA-pair kernel ----
template <int BITS, int ACT, int EPI>
static int launch_pair_epi(const PairTmapSet& tx, const GemmParams& p, cudaStream_t s) {
  using Cfg = PairCfg<BITS>;
  static int clusters_of_device[64] = {0};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) return QTALE_ERR_CUDA;
  if (clusters_of_device[dev] == 0) {
    if (cudaFuncSetAttribute(wq_gemm_pair_kernel<BITS, ACT, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)Cfg::kSmemBytes) != cudaSuccess)
      return QTALE_ERR_CUDA;
    // how many CTA pairs the device can hold at once: the persistent grid is sized to it
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)sm_count() & ~1u);
    cfg.blockDim = dim3(kPairThreads);
    cfg.dynamicSmemBytes = Cfg::kSmemBytes;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, wq_gemm_pair_kernel<BITS, ACT, EPI>, &cfg) != cudaSuccess || n < 1) {
      cudaGetLastError();
      n = sm_count() / 2;
    }
    clusters_of_device[dev] = n;
  }
  const int max_tiles = ((p.M_cap + 31) / 32) * ((p.n_tiles + 1) / 2);
  int clusters = clusters_of_device[dev];
  if (clusters > max_tiles) clusters = max_tiles;
  if (clusters < 1) clusters = 1;
  wq_gemm_pair_kernel<BITS, ACT, EPI><<<2 * clusters, kPairThreads, Cfg::kSmemBytes, s>>>(tx, p);
  return launch_status(cudaGetLastError());
}

// one instantiation per epilogue: each carries only its own epilogue code and registers
template <int BITS, int ACT>
static int launch_pair(const PairTmapSet& tx, const GemmParams& p, cudaStream_t s) {
  switch (p.epilogue) {
    case QTALE_EPI_STORE_16: return launch_pair_epi<BITS, ACT, QTALE_EPI_STORE_16>(tx, p, s);
    case QTALE_EPI_STORE_F32: return launch_pair_epi<BITS, ACT, QTALE_EPI_STORE_F32>(tx, p, s);
    case QTALE_EPI_RESID_F32: return launch_pair_epi<BITS, ACT, QTALE_EPI_RESID_F32>(tx, p, s);
    case QTALE_EPI_RESID_SCATTER: return launch_pair_epi<BITS, ACT, QTALE_EPI_RESID_SCATTER>(tx, p, s);
    case QTALE_EPI_SWIGLU: return launch_pair_epi<BITS, ACT, QTALE_EPI_SWIGLU>(tx, p, s);
    case QTALE_EPI_ROPE: return launch_pair_epi<BITS, ACT, QTALE_EPI_ROPE>(tx, p, s);
  }
  return QTALE_ERR_MODE;
}

static int make_pair_tmaps(PairTmapSet* set, const void* base, int rows, int cols, int ld, int act) {
  for (int h = 16; h <= kPairTokens / 2; h += 16) {
    const int rc = make_tmap_16(&set->m[h / 16 - 1], base, rows, cols, ld, h, act);
    if (rc != QTALE_OK) return rc;
  }
  return QTALE_OK;
}

// ---- small-M kernel ----
template <int BITS, int ACT, int ROWS>
static int launch_small_rows(const CUtensorMap& tx, const GemmParams& p, cudaStream_t s) {
  using Cfg = SmallCfg<BITS, ROWS>;
  static bool configured[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) return QTALE_ERR_CUDA;
  if (!configured[dev]) {
    if (cudaFuncSetAttribute(wq_gemm_small_kernel<BITS, ACT, ROWS>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)Cfg::kSmemBytes) != cudaSuccess)
      return QTALE_ERR_CUDA;
    configured[dev] = true;
  }
  wq_gemm_small_kernel<BITS, ACT, ROWS>
      <<<p.n_tiles * (kTileRows / ROWS), kSmallThreads, Cfg::kSmemBytes, s>>>(tx, p);
  return launch_status(cudaGetLastError());
}

// Rows per CTA: the most that still fills the device (each CTA streams all the activations, so
// fewer, taller CTAs read less); a quarter tile at the least.
template <int BITS, int ACT>
static int launch_small(const CUtensorMap& tx, const GemmParams& p, cudaStream_t s) {
  const int sms = sm_count();  // two CTAs fit an SM
  if (p.n_tiles >= 2 * sms) return launch_small_rows<BITS, ACT, 128>(tx, p, s);
  if (2 * p.n_tiles >= sms) return launch_small_rows<BITS, ACT, 64>(tx, p, s);
  return launch_small_rows<BITS, ACT, 32>(tx, p, s);
}

template <int BITS, int ACT>
static int launch_gemm64(const TmapSet& tx, const CUtensorMap& tw, const GemmParams& p, cudaStream_t s) {
  return launch_gemm<64, BITS, ACT, false>(tx, tw, p, s);
}
template <int BITS, int ACT>
static int launch_gemm64_split(const TmapSet& tx, const CUtensorMap& tw, const GemmParams& p, cudaStream_t s) {
  return launch_gemm<64, BITS, ACT, true>(tx, tw, p, s);
}

// FN<bits, act> ARGS for the weight's bit-width (2, 3, 4) and the activation format
#define QTALE_BY_BITS_ACT(FN, ARGS)                                              \
  do {                                                                           \
    if (act == QTALE_ACT_F16) {                                                  \
      if (w->bits == 4) return FN<4, 1> ARGS;                                    \
      if (w->bits == 3) return FN<3, 1> ARGS;                                    \
      return FN<2, 1> ARGS;                                                      \
    }                                                                            \
    if (w->bits == 4) return FN<4, 0> ARGS;                                      \
    if (w->bits == 3) return FN<3, 0> ARGS;                                      \
    return FN<2, 0> ARGS;                                                        \
  } while (0)

// Token counts from which the CTA-pair kernel is used (below, a tile of 256 tokens is mostly padding).
constexpr int kPairMinTokens = 129;

static int pick_tn(int M_cap) { return M_cap <= 64 ? 64 : (M_cap <= 128 ? 128 : 192); }

size_t wq_blob_bytes(int N, int K, int bits, int group, int row_mode, WqGeometry* g) {
  WqGeometry q;
  q.K_pad = (K + group - 1) / group * group;
  q.nkb = q.K_pad / kKB;
  q.ng = q.K_pad / group;
  q.n_tiles = row_mode == QTALE_WQ_ROWS_SWIGLU ? ((N / 2) + 63) / 64 : (N + kTileRows - 1) / kTileRows;
  q.block_bytes = kTileRows * kKB * bits / 8;
  q.tile_bytes = q.block_bytes + kTileRows * 4;  // codes + (scale, zero) words of one row tile, one K block
  q.n_rp = (q.n_tiles + 1) / 2;                  // row tiles are stored in pairs
  q.sz_offset = 0;
  q.total = (size_t)q.n_rp * q.nkb * 2 * q.tile_bytes;
  if (g) *g = q;
  return q.total;
}

// Split K for token counts of a decode step (single-CTA tcgen05 kernel, 256 weight rows per
// tile): the number of K slices that minimises (waves of the grid) x (K blocks per slice + the
// cost of writing and re-reading a partial tile, about four K blocks).
static int pick_split_k(int n_rp, int nkb, int sms, size_t ws_bytes) {
  long best = -1;
  int best_s = 1;
  for (int sp = 1; sp <= 8 && sp * 2 <= nkb; ++sp) {
    if (wq_splitk_ticket_bytes() + (size_t)n_rp * sp * kSplitTileBytes > ws_bytes) break;
    const long waves = ((long)n_rp * sp + sms - 1) / sms;
    // in K blocks (about half a microsecond each): per tile of the slowest CTA its K blocks plus
    // the pipeline refill and the epilogue (4) or the partial tile's write and fence (8); split
    // only: the second half of the kernel (waiting for the other slices, summing, epilogue: 14)
    const long cost = waves * ((nkb + sp - 1) / sp + (sp > 1 ? 8 : 4)) + (sp > 1 ? 14 : 0);
    if (best < 0 || cost < best) { best = cost; best_s = sp; }
  }
  return best_s;
}

size_t wq_splitk_ticket_bytes() { return 4 * 4096; }  // one 4 KB region of counters per linear of a layer

size_t wq_splitk_workspace_bytes() {
  // tickets + partial tiles for up to sixteen slices of 148 tile groups is more than any layer
  // needs; 48 MB covers (groups x slices) <= 768
  return wq_splitk_ticket_bytes() + (size_t)768 * kSplitTileBytes;
}

int wq_gemm_launch(const void* a, int lda, const int32_t* m_dev, int M_cap,
                   const qtale_wq_weight* w, int act, int epilogue, const qtale_epilogue_args* epi,
                   void* y, int ldy, cudaStream_t s, void* splitk_ws, size_t splitk_bytes,
                   int splitk_slot) {
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
  p.rope_hd = w->row_mode == QTALE_WQ_ROWS_ROPE64 ? 64 : (w->row_mode == QTALE_WQ_ROWS_ROPE128 ? 128 : 0);
  if (epilogue == QTALE_EPI_ROPE) {
    p.rope_cs = static_cast<const float2*>(epi->rope_cs);
    p.rope_limit = epi->rope_features;
  }
  p.status = device_status_ptr();
  if (M_cap >= kPairMinTokens) {
    PairTmapSet px;
    memset(&px, 0, sizeof(px));
    const int rc = make_pair_tmaps(&px, a, M_cap, w->K, lda, act);
    if (rc != QTALE_OK) return rc;
    QTALE_BY_BITS_ACT(launch_pair, (px, p, s));
  }
  if (M_cap <= kSmallTokens && splitk_ws && g.n_rp <= 1024 && w->bits != 16) {
    // decode step inside a layer: the tcgen05 kernel with the K dimension split over the SMs
    TmapSet tx;
    CUtensorMap tw;
    memset(&tx, 0, sizeof(tx));
    memset(&tw, 0, sizeof(tw));
    const int rc = make_tmap_set(&tx, a, M_cap, w->K, lda, 64, act);
    if (rc != QTALE_OK) return rc;
    p.split_k = pick_split_k(g.n_rp, g.nkb, sm_count(), splitk_bytes);
    p.tickets = static_cast<int*>(splitk_ws) + (splitk_slot & 3) * 1024;
    p.partial = reinterpret_cast<float*>(static_cast<unsigned char*>(splitk_ws) + wq_splitk_ticket_bytes());
    if (p.split_k <= 1) {  // enough row tiles for the device: the plain kernel, no partial tiles
      p.split_k = 1;
      QTALE_BY_BITS_ACT(launch_gemm64, (tx, tw, p, s));
    }
    QTALE_BY_BITS_ACT(launch_gemm64_split, (tx, tw, p, s));
  }
  if (M_cap <= kSmallTokens) {
    CUtensorMap tx1;
    memset(&tx1, 0, sizeof(tx1));
    const int rc = make_tmap_16(&tx1, a, M_cap, w->K, lda, kSmallTokens, act);
    if (rc != QTALE_OK) return rc;
    QTALE_BY_BITS_ACT(launch_small, (tx1, p, s));
  }
  const int tn = pick_tn(M_cap);
  TmapSet tx;
  CUtensorMap tw;
  memset(&tx, 0, sizeof(tx));
  memset(&tw, 0, sizeof(tw));
  int rc = make_tmap_set(&tx, a, M_cap, w->K, lda, tn, act);
  if (rc != QTALE_OK) return rc;
  QTALE_BY_BITS_ACT(dispatch_tn, (tx, tw, p, tn, s));
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
  TmapSet tx;
  CUtensorMap tw;
  memset(&tx, 0, sizeof(tx));
  int rc = make_tmap_set(&tx, a, M_cap, K, lda, tn, QTALE_ACT_BF16);
  if (rc != QTALE_OK) return rc;
  rc = make_tmap_16(&tw, w_bf16, N, K, ldw, kTileRows, QTALE_ACT_BF16);
  if (rc != QTALE_OK) return rc;
  return dispatch_tn<16, 0>(tx, tw, p, tn, s);
}

// ---- offline repack (host) -------------------------------------------------------

static inline unsigned canon_code(const uint8_t* row, int k, int bits) {
  if (bits == 4) return (k & 1) ? (row[k >> 1] >> 4) : (row[k >> 1] & 0xF);
  if (bits == 2) return (row[k >> 2] >> (2 * (k & 3))) & 3u;
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
  if (bits < 2 || bits > 4) return QTALE_ERR_BITS;
  if (group != 64 && group != 128) return QTALE_ERR_GROUP;
  if (N < 1 || K < 1) return QTALE_ERR_SHAPE;
  if (row_mode < QTALE_WQ_ROWS_PLAIN || row_mode > QTALE_WQ_ROWS_ROPE128) return QTALE_ERR_MODE;
  if (row_mode == QTALE_WQ_ROWS_SWIGLU && (N % 2) != 0) return QTALE_ERR_SHAPE;
  if (row_mode == QTALE_WQ_ROWS_ROPE64 && (N % 64) != 0) return QTALE_ERR_SHAPE;
  if (row_mode == QTALE_WQ_ROWS_ROPE128 && (N % 128) != 0) return QTALE_ERR_SHAPE;
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
  const int row_bytes = bits == 4 ? (K + 1) / 2 : (bits == 3 ? (3 * K + 7) / 8 : (K + 3) / 4);
  const int ng_in = (K + group - 1) / group;
  const int F = N / 2;
  for (int nt = 0; nt < g.n_tiles; ++nt) {
    for (int L = 0; L < kTileRows; ++L) {
      int n;
      if (row_mode == QTALE_WQ_ROWS_SWIGLU) {
        const int q = L >> 5, r = L & 31;
        const int j = nt * 64 + q * 16 + (r & 15);
        n = (j < F) ? ((r < 16) ? j : F + j) : -1;
      } else if (row_mode == QTALE_WQ_ROWS_ROPE64 || row_mode == QTALE_WQ_ROWS_ROPE128) {
        const int hd = row_mode == QTALE_WQ_ROWS_ROPE64 ? 64 : 128, half = hd / 2;
        const int q = L >> 5, r = L & 31;
        const int e = q * 16 + (r & 15);
        n = nt * kTileRows + (e / half) * hd + (e % half) + (r < 16 ? 0 : half);
        if (n >= N) n = -1;
      } else {
        n = nt * kTileRows + L;
        if (n >= N) n = -1;
      }
      // chunk of (pair nt/2, K block kb): [tile nt%2]{codes, 128 (scale | zero << 16) words}
      auto chunk = [&](int kb) {
        return out + (((size_t)(nt >> 1) * g.nkb + kb) * 2 + (nt & 1)) * g.tile_bytes;
      };
      if (n < 0) continue;  // padding rows keep scale 0, zero 0, codes 0
      for (int kb = 0; kb < g.nkb; ++kb) {
        const int gi = kb * kKB / group;
        uint32_t v = 0;
        if (gi < ng_in)
          v = (uint32_t)scales[(size_t)n * ng_in + gi] | ((uint32_t)zeros[(size_t)n * ng_in + gi] << 16);
        reinterpret_cast<uint32_t*>(chunk(kb) + g.block_bytes)[L] = v;
      }
      const uint8_t* row = codes + (size_t)n * row_bytes;
      for (int kb = 0; kb < g.nkb; ++kb) {
        uint8_t* blk = chunk(kb);
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
        // slot i of an 8-code word holds feature 2i (i < 4) or 2(i-4)+1 (i >= 4) of the word
        auto slot_k = [](int i) { return i < 4 ? 2 * i : 2 * (i - 4) + 1; };
        if (bits == 4) {
          // [part][lane][4 words]; word j of part p covers k = 32p + 8j .. +7, slot i in nibble i
          for (int part = 0; part < 2; ++part) {
            uint32_t* wdst = reinterpret_cast<uint32_t*>(blk) + ((size_t)part * kTileRows + L) * 4;
            for (int j = 0; j < 4; ++j) {
              uint32_t wv = 0;
              for (int i = 0; i < 8; ++i) wv |= (q[32 * part + 8 * j + slot_k(i)] & 0xFu) << (4 * i);
              wdst[j] = wv;
            }
          }
        } else {
          // plane A: [lane][4 words], 2-bit field f of word w2 <- low bits of slot f/2 of word
          //          u = 2 w2 + f%2;  plane B: [lane][2 words], bit 4i + u%4 of word u/4 <- high
          //          bit of slot i of word u
          uint32_t* a = reinterpret_cast<uint32_t*>(blk) + (size_t)L * 4;
          uint32_t* b = reinterpret_cast<uint32_t*>(blk + kTileRows * 16) + (size_t)L * 2;
          for (int w2 = 0; w2 < 4; ++w2) {
            uint32_t wv = 0;
            for (int f = 0; f < 16; ++f)
              wv |= (q[8 * (2 * w2 + (f & 1)) + slot_k(f >> 1)] & 3u) << (2 * f);
            a[w2] = wv;
          }
          if (bits == 3) {
            uint32_t b0 = 0, b1 = 0;
            for (int u = 0; u < 8; ++u)
              for (int i = 0; i < 8; ++i) {
                const uint32_t hb = (q[8 * u + slot_k(i)] >> 2) & 1u;
                if (u < 4) b0 |= hb << (4 * i + (u & 3)); else b1 |= hb << (4 * i + (u & 3));
              }
            b[0] = b0;
            b[1] = b1;
          }
        }
      }
    }
  }
  return QTALE_OK;
}

size_t qtale_wq_gemm_workspace_bytes(void) { return wq_splitk_workspace_bytes(); }

int qtale_wq_gemm(const void* a, int lda, const int32_t* m_dev, int M_cap, const qtale_wq_weight* w,
                  int act_dtype, int epilogue, const qtale_epilogue_args* epi, void* y, int ldy,
                  void* ws, size_t ws_bytes, void* stream) {
  if (!a || !w || !w->packed) return QTALE_ERR_NULL;
  if (act_dtype != QTALE_ACT_BF16 && act_dtype != QTALE_ACT_F16) return QTALE_ERR_MODE;
  if (w->bits < 2 || w->bits > 4) return QTALE_ERR_BITS;
  if (w->group != 64 && w->group != 128) return QTALE_ERR_GROUP;
  if (M_cap < 1 || w->N < 1 || w->K < 1 || lda < w->K) return QTALE_ERR_SHAPE;
  if (epilogue < QTALE_EPI_STORE_16 || epilogue > QTALE_EPI_ROPE) return QTALE_ERR_MODE;
  if (epilogue == QTALE_EPI_SWIGLU && w->row_mode != QTALE_WQ_ROWS_SWIGLU) return QTALE_ERR_MODE;
  if (epilogue == QTALE_EPI_ROPE) {
    if (w->row_mode != QTALE_WQ_ROWS_ROPE64 && w->row_mode != QTALE_WQ_ROWS_ROPE128) return QTALE_ERR_MODE;
    if (!epi || !epi->rope_cs) return QTALE_ERR_NULL;
    const int hd = w->row_mode == QTALE_WQ_ROWS_ROPE64 ? 64 : 128;
    if (epi->rope_features < 0 || epi->rope_features > w->N || epi->rope_features % hd != 0)
      return QTALE_ERR_SHAPE;
    if (!aligned16(epi->rope_cs)) return QTALE_ERR_ALIGN;
  }
  if (epilogue == QTALE_EPI_RESID_F32 || epilogue == QTALE_EPI_RESID_SCATTER) {
    if (!epi || !epi->idx || !epi->resid) return QTALE_ERR_NULL;
    if (epilogue == QTALE_EPI_RESID_SCATTER && !epi->dst) return QTALE_ERR_NULL;
  }
  if (epilogue != QTALE_EPI_RESID_SCATTER && !y) return QTALE_ERR_NULL;
  if (!aligned16(a) || !aligned16(w->packed) || (lda * 2) % 16 != 0) return QTALE_ERR_ALIGN;
  // the epilogue moves 8 consecutive output features (16 bytes of 16-bit data) per lane
  if (w->N % 8 != 0 || (w->row_mode == QTALE_WQ_ROWS_SWIGLU && (w->N / 2) % 8 != 0))
    return QTALE_ERR_SHAPE;
  if (y && (!aligned16(y) || ldy % 8 != 0)) return QTALE_ERR_ALIGN;
  if (epi && epi->resid && (!aligned16(epi->resid) || epi->ld_resid % 8 != 0)) return QTALE_ERR_ALIGN;
  if (epi && epi->dst && (!aligned16(epi->dst) || epi->ld_dst % 8 != 0)) return QTALE_ERR_ALIGN;
  if (ws) {
    if (!aligned16(ws)) return QTALE_ERR_ALIGN;
    if (ws_bytes < wq_splitk_workspace_bytes()) return QTALE_ERR_WORKSPACE;
    if (M_cap <= kSmallTokens &&  // the counters of the split-K path start at zero
        cudaMemsetAsync(ws, 0, 4096, static_cast<cudaStream_t>(stream)) != cudaSuccess)
      return QTALE_ERR_CUDA;
  }
  return wq_gemm_launch(a, lda, m_dev, M_cap, w, act_dtype, epilogue, epi, y, ldy,
                        static_cast<cudaStream_t>(stream), ws, ws_bytes, 0);
}

}  // extern "C"
