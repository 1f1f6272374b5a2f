// Causal attention among the executed tokens of each sequence (prefill) on the
// tcgen05 tensor cores (Eq. 3: bypassed tokens have no query, key or value here).
//
// A work item is 128 consecutive executed tokens (query rows) of one sequence and one
// head; the grid is persistent (one CTA per SM walks the items sequence by sequence) and an item
// streams that sequence's executed keys / values in tiles of 128:
//   S = Q K^T     SS MMA, Q and K tiles from 128-byte-swizzled shared memory (TMA),
//                 fp32 scores in tensor memory, double buffered;
//   softmax       eight warps, two threads per query row (64 keys each; the half-row maxima
//                 meet through shared memory): running max / sum in the log2 domain (one fma
//                 and one ex2.approx per score), probabilities written back to tensor memory
//                 in the 16-bit activation format (the A operand of the next MMA);
//   O += P V      TS MMA with V read straight from its row-major tile (MN-major B
//                 operand), fp32 output accumulator in tensor memory, rescaled by the
//                 softmax warps only when a row's maximum has outgrown the reference by 2^8.
// Keys and values have rings of their own (three and two tiles) and a producer thread each:
// a key tile is free as soon as its scores exist, so its successor is loaded three tiles
// ahead; with one two-stage ring released after P V the load latency (about 1800 cycles) sat
// in the loop of every tile.  Barrier phases run on across items (tiles are counted per
// CTA), so the loads and the first Q K^T of the next item overlap the output stage of the
// current one.
// Warp roles (352 threads): warp 0 Q / K producer, warp 1 MMA issuer and TMEM allocator,
// warps 2-9 softmax / correction / output, warp 10 V producer.  Every wait is bounded.
#include <cuda.h>

#include <string.h>

#include "attention.cuh"
#include "ptx.cuh"

namespace qtale {

using namespace ptx;

constexpr int kTcThreads = 352;  // K producer, issuer, eight softmax warps, V producer
constexpr int kTcKStages = 3;    // key tiles in flight (the first thing a tile needs)
constexpr int kTcVStages = 2;    // value tiles in flight
constexpr int kTcTile = 128;  // query rows per CTA and keys per tile
constexpr uint32_t kTcSlices = 1u << 16;  // suspended barrier tests before a wait gives up
constexpr float kTcMaxSlack = 8.f;        // log2 growth of a row maximum that moves the softmax reference

struct TcShared {
  uint64_t q_full, q_empty, o_empty;
  uint64_t k_full[kTcKStages], k_empty[kTcKStages];
  uint64_t v_full[kTcVStages], v_empty[kTcVStages];
  uint64_t max_bar, sum_bar;  // the two threads of a query row exchange their half-row maximum / sum
  float row_max[2][2][kTcTile];  // [tile parity][half][row]
  float row_sum[2][kTcTile];     // [half][row]
  uint64_t s_full[2], p_full[2];
  uint64_t pv_done;
  uint32_t tmem_base;
  volatile int abort_flag;
};

struct TcParams {
  const int32_t* cu_exec;
  int B, rep, H;
  int k_off, v_off;      // column offsets of the K and V heads inside a qkv row
  void* out;
  int ldo;
  float scale_log2;
  int* status;
};

// 2^x by the special-function unit alone (about 2 ulp; -inf gives 0): the softmax is bound by
// this unit, so nothing is spent on the range fix-ups of exp2f
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ bool tc_wait(uint64_t* bar, uint32_t parity, TcShared* sh, int* status) {
  // the first test is plain; after that the thread lets the hardware suspend it (up to 20 us a
  // test), so waiting roles leave the issue slots to the softmax warps
  if (mbar_try_wait(bar, parity)) return true;
  for (uint32_t it = 0; it < kTcSlices; ++it) {
    if (mbar_try_wait_suspend(bar, parity, 20000u)) return true;
    if (sh->abort_flag) return false;
  }
  sh->abort_flag = 1;
  report_device_error(status, QTALE_ERR_TIMEOUT);
  return false;
}

// K-major tile of 128 rows x 64 elements per 16 KB chunk (128-byte swizzle): descriptor
// of the 16-element K step `kk` (chunks follow each other every 16 KB)
__device__ __forceinline__ uint64_t kmajor_desc(uint32_t smem_addr, int kk) {
  return smem_desc_sw128(smem_addr + (kk >> 2) * 16384) + 2u * (kk & 3);
}
// V tile used as the MN-major B operand: rows are keys (the MMA's K), a row holds 64
// head-dim elements per chunk.  Eight key rows form one 1024-byte group (stride offset),
// the next 64 head-dim elements are 16 KB further (leading offset).
__device__ __forceinline__ uint64_t v_desc(uint32_t smem_addr, int key16) {
  uint64_t d = 0;
  d |= (uint64_t)(((smem_addr + key16 * 2048) & 0x3FFFFu) >> 4);
  d |= (uint64_t)(16384 >> 4) << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// Work items of the persistent grid, sequence by sequence; within a sequence by query tile
// (longest first in even sequences, shortest first in odd ones), each tile for every head.  CTA
// c takes items c, c + grid, ...  The CTAs running at one time then work on one or two
// sequences, whose keys and values stay in L2 (with the tiles of all sequences sorted into one
// list, every sequence's keys were live at once and were re-read from DRAM 3.6 times), and
// the alternating direction evens out the CTAs' total tile counts.  The cursor only moves forward.
struct ItemCursor {
  int seq;    // sequence being enumerated
  int base;   // index of its first item
  int nt;     // its query tiles (-1: not counted yet)
};

__device__ __forceinline__ int seq_tiles(const TcParams& p, int s) {
  return (p.cu_exec[s + 1] - p.cu_exec[s] + kTcTile - 1) / kTcTile;
}

// item i (i must not decrease between calls) -> sequence, head, query tile; false past the end
__device__ __forceinline__ bool item_at(const TcParams& p, ItemCursor& c, int i, int& b, int& h, int& qt) {
  while (c.seq < p.B) {
    if (c.nt < 0) c.nt = seq_tiles(p, c.seq);
    const int n = c.nt * p.H;
    if (i < c.base + n) {
      const int r = i - c.base;
      b = c.seq;
      h = r % p.H;
      qt = (c.seq & 1) ? r / p.H : c.nt - 1 - r / p.H;
      return true;
    }
    c.base += n;
    c.nt = -1;
    ++c.seq;
  }
  return false;
}

template <int HD, int ACT>
__global__ void __launch_bounds__(kTcThreads, 1)
    attn_prefill_tc_kernel(const __grid_constant__ CUtensorMap tmap, const TcParams p) {
  constexpr int CH = HD / 64;                       // 16 KB chunks per tile
  constexpr int TILE_BYTES = kTcTile * HD * 2;
  constexpr int S_COL = 0;                          // two score buffers of 128 columns
  constexpr int P_COL = 256;                        // two probability buffers of 64 columns
  constexpr int O_COL = 384;                        // output accumulator, HD columns
  extern __shared__ unsigned char smem_dyn[];
  __shared__ TcShared sh;
  unsigned char* base = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
  unsigned char* sQ = base;
  unsigned char* sK = base + TILE_BYTES;                     // kTcKStages stages
  unsigned char* sV = base + (1 + kTcKStages) * TILE_BYTES;  // kTcVStages stages

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  int n_pairs = 0;
  for (int s = 0; s < p.B; ++s) n_pairs += seq_tiles(p, s);
  const int n_items = n_pairs * p.H;
  if ((int)blockIdx.x >= n_items) return;  // uniform for the CTA: nothing allocated yet

  if (threadIdx.x == 0) {
    mbar_init(&sh.q_full, 1);
    mbar_init(&sh.q_empty, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sh.s_full[s], 1);
      mbar_init(&sh.p_full[s], 8);
    }
    for (int s = 0; s < kTcKStages; ++s) {
      mbar_init(&sh.k_full[s], 1);
      mbar_init(&sh.k_empty[s], 1);
    }
    for (int s = 0; s < kTcVStages; ++s) {
      mbar_init(&sh.v_full[s], 1);
      mbar_init(&sh.v_empty[s], 1);
    }
    mbar_init(&sh.max_bar, 8);
    mbar_init(&sh.sum_bar, 8);
    mbar_init(&sh.pv_done, 1);
    mbar_init(&sh.o_empty, 8);
    sh.abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(&sh.tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh.tmem_base;

  // every role walks the same item sequence with its own cursor and its own running counters:
  // t = key tiles so far (ring stage t & 1, phase (t >> 1) & 1), it = items so far
  ItemCursor cur;
  cur.seq = 0;
  cur.base = 0;
  cur.nt = -1;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      uint32_t t = 0, it = 0;
      for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++it) {
        int b, h, qt;
        if (!item_at(p, cur, item, b, h, qt)) break;
        const int hk = h / p.rep;
        const int seq0 = p.cu_exec[b];
        if (!tc_wait(&sh.q_empty, (it & 1u) ^ 1u, &sh, p.status)) break;
        mbar_arrive_expect_tx(&sh.q_full, TILE_BYTES);
        for (int c = 0; c < CH; ++c)
          tma_load_2d(sQ + c * 16384, &tmap, &sh.q_full, h * HD + c * 64, seq0 + qt * kTcTile);
        bool ok = true;
        for (int j = 0; j <= qt; ++j, ++t) {
          const int s = t % kTcKStages;
          const uint32_t ph = (t / kTcKStages) & 1u;
          if (!tc_wait(&sh.k_empty[s], ph ^ 1u, &sh, p.status)) { ok = false; break; }
          mbar_arrive_expect_tx(&sh.k_full[s], TILE_BYTES);
          for (int c = 0; c < CH; ++c)
            tma_load_2d(sK + s * TILE_BYTES + c * 16384, &tmap, &sh.k_full[s],
                        p.k_off + hk * HD + c * 64, seq0 + j * kTcTile);
        }
        if (!ok) break;
      }
    }
  } else if (warp == 10) {
    // ------------------------------ TMA producer of the value tiles ------------------------------
    // (a thread of its own: a full value ring must not hold back the key loads)
    if (lane == 0) {
      uint32_t t = 0;
      bool ok = true;
      for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
        int b, h, qt;
        if (!item_at(p, cur, item, b, h, qt)) break;
        const int hk = h / p.rep;
        const int seq0 = p.cu_exec[b];
        for (int j = 0; j <= qt; ++j, ++t) {
          const int s = t % kTcVStages;
          const uint32_t ph = (t / kTcVStages) & 1u;
          if (!tc_wait(&sh.v_empty[s], ph ^ 1u, &sh, p.status)) { ok = false; break; }
          mbar_arrive_expect_tx(&sh.v_full[s], TILE_BYTES);
          for (int c = 0; c < CH; ++c)
            tma_load_2d(sV + s * TILE_BYTES + c * 16384, &tmap, &sh.v_full[s],
                        p.v_off + hk * HD + c * 64, seq0 + j * kTcTile);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer -------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc_qk = idesc_16bit_f32(128, kTcTile, ACT == 1);
      constexpr uint32_t idesc_pv = idesc_16bit_f32(128, HD, ACT == 1) | (1u << 16);  // B is MN-major
      const uint32_t qa = smem_u32(sQ);
      auto issue_qk = [&](uint32_t tt) {
        const int s = tt & 1;
        const int ks = tt % kTcKStages;
        if (!tc_wait(&sh.k_full[ks], (tt / kTcKStages) & 1u, &sh, p.status)) return false;
        tc_fence_after();
        const uint32_t ka = smem_u32(sK + ks * TILE_BYTES);
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk)
          mma_ss(tmem + S_COL + s * 128, kmajor_desc(qa, kk), kmajor_desc(ka, kk), idesc_qk,
                 kk != 0 ? 1u : 0u);
        mma_commit(&sh.s_full[s]);
        mma_commit(&sh.k_empty[ks]);  // the key tile is free as soon as its scores exist
        return true;
      };
      uint32_t t = 0, it = 0;
      bool ok = true;
      for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x, ++it) {
        int b, h, qt;
        if (!item_at(p, cur, item, b, h, qt)) break;
        const int n_kt = qt + 1;
        if (!tc_wait(&sh.q_full, it & 1u, &sh, p.status)) break;
        ok = issue_qk(t);
        if (ok && n_kt == 1) mma_commit(&sh.q_empty);  // the query tile has been read for the last time
        for (int j = 0; ok && j < n_kt; ++j) {
          const uint32_t tt = t + j;
          const int s = tt & 1;
          const uint32_t ph = (tt >> 1) & 1u;
          // scores of the next tile are computed while the softmax of this one runs
          if (j + 1 < n_kt) {
            ok = issue_qk(tt + 1);
            if (ok && j + 2 == n_kt) mma_commit(&sh.q_empty);
          }
          if (!ok) break;
          if (!tc_wait(&sh.p_full[s], ph, &sh, p.status)) { ok = false; break; }
          const int vs = tt % kTcVStages;
          if (!tc_wait(&sh.v_full[vs], (tt / kTcVStages) & 1u, &sh, p.status)) { ok = false; break; }
          // the first P V of an item overwrites the accumulator: the previous item's output
          // must have been read
          if (j == 0 && !tc_wait(&sh.o_empty, (it & 1u) ^ 1u, &sh, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t va = smem_u32(sV + vs * TILE_BYTES);
#pragma unroll
          for (int kk = 0; kk < kTcTile / 16; ++kk)
            mma_ts(tmem + O_COL, tmem + P_COL + s * 64 + kk * 8, v_desc(va, kk), idesc_pv,
                   (j | kk) != 0 ? 1u : 0u);
          mma_commit(&sh.v_empty[vs]);
          mma_commit(&sh.pv_done);
        }
        t += n_kt;
      }
    }
  } else {
    // ---------- softmax, correction and output: two threads per query row ----------
    // Warps 2-5 take keys 0..63 of a tile, warps 6-9 keys 64..127 (the same split of the output
    // columns at the end); a warp reaches the TMEM lanes 32 (warp % 4) .. + 31.  The two threads
    // of a row exchange their half-row maximum through shared memory and an mbarrier (bounded
    // wait, like every other wait here), and their partial sums once per item.
    const int quad = warp & 3;
    const int half = (warp - 2) >> 2;
    const int row = quad * 32 + lane;          // TMEM lane = query row of the tile
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    constexpr int OC = HD / 2;                 // output columns of this thread
    uint32_t t = 0, it = 0;
    bool alive = true;
    for (int item = blockIdx.x; alive && item < n_items; item += gridDim.x, ++it) {
      int b, h, qt;
      if (!item_at(p, cur, item, b, h, qt)) break;
      const int seq0 = p.cu_exec[b];
      const int len = p.cu_exec[b + 1] - seq0;
      const int q0 = qt * kTcTile;
      const int n_kt = qt + 1;
      const int q_row = q0 + row;
      float m_run = -INFINITY, l_run = 0.f;  // l_run: this thread's half of the row sum
      for (int j = 0; j < n_kt && alive; ++j) {
        const uint32_t tt = t + j;
        const int s = tt & 1;
        const uint32_t ph = (tt >> 1) & 1u;
        if (!tc_wait(&sh.s_full[s], ph, &sh, p.status)) { alive = false; break; }
        tc_fence_after();
        const uint32_t s_addr = tmem + lane_addr + S_COL + s * 128 + half * 64;
        const int k0 = j * kTcTile + half * 64;
        const bool masked = (j == qt) || (j * kTcTile + kTcTile > len);
        // half a score row (64 keys) in registers, unscaled; the scale (positive) is folded into
        // the exponent's multiply-add, so an element costs one max, one fma, one ex2, one add
        float sc[64];
        {
          uint32_t r0[32], r1[32];
          tmem_ld_x32(s_addr, r0);
          tmem_ld_x32(s_addr + 32, r1);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            sc[i] = __uint_as_float(r0[i]);
            sc[32 + i] = __uint_as_float(r1[i]);
          }
        }
        if (masked) {
#pragma unroll
          for (int i = 0; i < 64; ++i) {
            const int key = k0 + i;
            if (key > q_row || key >= len) sc[i] = -INFINITY;
          }
        }
        float mq[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int i = 0; i < 64; i += 4) {
          mq[0] = fmaxf(mq[0], sc[i]);
          mq[1] = fmaxf(mq[1], sc[i + 1]);
          mq[2] = fmaxf(mq[2], sc[i + 2]);
          mq[3] = fmaxf(mq[3], sc[i + 3]);
        }
        const float my_max = fmaxf(fmaxf(mq[0], mq[1]), fmaxf(mq[2], mq[3]));
        sh.row_max[tt & 1][half][row] = my_max;
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.max_bar);
        if (!tc_wait(&sh.max_bar, tt & 1u, &sh, p.status)) { alive = false; break; }
        const float row_raw = fmaxf(my_max, sh.row_max[tt & 1][half ^ 1][row]);
        // The reference maximum only moves when the row's maximum has grown by more than 2^8
        // (always on the first tile): until then the probabilities are at most 256, which both
        // 16-bit formats and the fp32 sums hold, and the output accumulator needs no rescaling.
        const float cand = row_raw * p.scale_log2;
        const bool moved = cand > m_run + kTcMaxSlack;
        float corr = 1.f;
        if (moved) {
          corr = ex2_approx(m_run - cand);  // 0 on the first tile (m_run = -inf)
          m_run = cand;
          l_run *= corr;
        }
        // probabilities in the 16-bit format, two keys per 32-bit column
        const float neg_m = (m_run == -INFINITY) ? 0.f : -m_run;
        float sq[4] = {0.f, 0.f, 0.f, 0.f};
        uint32_t pr[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float p0 = ex2_approx(fmaf(sc[2 * i], p.scale_log2, neg_m));
          const float p1 = ex2_approx(fmaf(sc[2 * i + 1], p.scale_log2, neg_m));
          sq[i & 3] += p0 + p1;
          pr[i] = Act16<ACT>::pack(p0, p1);
        }
        l_run += (sq[0] + sq[1]) + (sq[2] + sq[3]);
        // The previous P V must be complete before O is rescaled.  Every tile waits for it, moved
        // or not, so that the barrier is never more than one phase ahead of a parity test (by now
        // that P V, issued a whole softmax earlier, has long finished).
        if (j > 0) {
          if (!tc_wait(&sh.pv_done, (tt - 1) & 1u, &sh, p.status)) { alive = false; break; }
          tc_fence_after();
        }
        if (j > 0 && __any_sync(0xffffffffu, moved)) {
#pragma unroll 1
          for (int c = 0; c < OC / 32; ++c) {
            uint32_t r[32];
            tmem_ld_x32(tmem + lane_addr + O_COL + half * OC + c * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * corr);
            tmem_st_x32(tmem + lane_addr + O_COL + half * OC + c * 32, r);
          }
        }
        tmem_st_x32(tmem + lane_addr + P_COL + s * 64 + half * 32, pr);
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.p_full[s]);
      }
      if (!alive) break;
      // output: O / l for the rows that exist; then the accumulator is handed back
      sh.row_sum[half][row] = l_run;
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.sum_bar);
      if (!tc_wait(&sh.sum_bar, it & 1u, &sh, p.status)) { alive = false; break; }
      const float l_tot = l_run + sh.row_sum[half ^ 1][row];
      if (!tc_wait(&sh.pv_done, (t + n_kt - 1) & 1u, &sh, p.status)) { alive = false; break; }
      tc_fence_after();
      const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;
      unsigned short* out = static_cast<unsigned short*>(p.out) + (size_t)(seq0 + q_row) * p.ldo +
                            (size_t)h * HD + half * OC;
#pragma unroll 1
      for (int c = 0; c < OC / 32; ++c) {
        uint32_t r[32];
        tmem_ld_x32(tmem + lane_addr + O_COL + half * OC + c * 32, r);
        tmem_wait_ld();
        if (c == OC / 32 - 1) {  // every column of this warp's part is in registers
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sh.o_empty);
        }
        if (q_row < len) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint4 o;
            o.x = Act16<ACT>::pack(__uint_as_float(r[8 * i + 0]) * inv, __uint_as_float(r[8 * i + 1]) * inv);
            o.y = Act16<ACT>::pack(__uint_as_float(r[8 * i + 2]) * inv, __uint_as_float(r[8 * i + 3]) * inv);
            o.z = Act16<ACT>::pack(__uint_as_float(r[8 * i + 4]) * inv, __uint_as_float(r[8 * i + 5]) * inv);
            o.w = Act16<ACT>::pack(__uint_as_float(r[8 * i + 6]) * inv, __uint_as_float(r[8 * i + 7]) * inv);
            st_16(out + c * 32 + i * 8, o);
          }
        }
      }
      t += n_kt;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// ---------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFnA)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                   const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                   const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFnA encode_fn_a() {
  static EncodeTiledFnA fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) ==
            cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFnA>(p);
  }
  return fn;
}

template <int HD, int ACT>
static int launch_tc(const CUtensorMap& tm, const TcParams& p, int max_tiles, int H, cudaStream_t s) {
  const size_t smem = (size_t)(1 + kTcKStages + kTcVStages) * kTcTile * HD * 2 + 1024;
  static bool configured[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    if (cudaFuncSetAttribute(attn_prefill_tc_kernel<HD, ACT>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return QTALE_ERR_CUDA;
    configured[dev] = true;
  }
  // persistent grid: one CTA per SM walks the (sequence, query tile, head) items
  (void)max_tiles;
  (void)H;
  attn_prefill_tc_kernel<HD, ACT><<<sm_count(), kTcThreads, smem, s>>>(tm, p);
  return launch_status(cudaGetLastError());
}

int launch_attn_prefill(const void* qkv, int ld, int H, int Hkv, int hd, int act,
                        const int32_t* cu_exec, int B, int T_cap, void* out, int ldo,
                        cudaStream_t s) {
  EncodeTiledFnA fn = encode_fn_a();
  if (!fn) return QTALE_ERR_CUDA;
  CUtensorMap tm;
  cuuint64_t gdim[2] = {(cuuint64_t)ld, (cuuint64_t)T_cap};
  cuuint64_t gstr[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {64, (cuuint32_t)kTcTile};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(&tm, act == QTALE_ACT_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                  2, const_cast<void*>(qkv), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return QTALE_ERR_CUDA;
  TcParams p;
  p.cu_exec = cu_exec;
  p.B = B;
  p.rep = H / Hkv;
  p.H = H;
  p.k_off = H * hd;
  p.v_off = (H + Hkv) * hd;
  p.out = out;
  p.ldo = ldo;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)hd);
  p.status = device_status_ptr();
  const int max_tiles = (T_cap + kTcTile - 1) / kTcTile + B;
  if (hd == 128)
    return act == QTALE_ACT_F16 ? launch_tc<128, 1>(tm, p, max_tiles, H, s) : launch_tc<128, 0>(tm, p, max_tiles, H, s);
  if (hd == 64)
    return act == QTALE_ACT_F16 ? launch_tc<64, 1>(tm, p, max_tiles, H, s) : launch_tc<64, 0>(tm, p, max_tiles, H, s);
  return QTALE_ERR_SHAPE;
}

}  // namespace qtale

extern "C" int qtale_attention_prefill(const void* qkv, int ld, int n_heads, int n_kv_heads, int head_dim,
                                       int act_dtype, const int32_t* cu_exec, int B, int T_cap, void* out,
                                       int ldo, void* stream) {
  using namespace qtale;
  if (act_dtype != QTALE_ACT_BF16 && act_dtype != QTALE_ACT_F16) return QTALE_ERR_MODE;
  if (!qkv || !cu_exec || !out) return QTALE_ERR_NULL;
  if (B < 1 || T_cap < 1 || n_heads < 1 || n_kv_heads < 1 || n_heads % n_kv_heads != 0 ||
      (head_dim != 64 && head_dim != 128))
    return QTALE_ERR_SHAPE;
  if (ld < (n_heads + 2 * n_kv_heads) * head_dim || ldo < n_heads * head_dim || ld % 8 != 0 || ldo % 8 != 0)
    return QTALE_ERR_SHAPE;
  if (!aligned16(qkv) || !aligned16(out)) return QTALE_ERR_ALIGN;
  return launch_attn_prefill(qkv, ld, n_heads, n_kv_heads, head_dim, act_dtype, cu_exec, B, T_cap, out, ldo,
                             static_cast<cudaStream_t>(stream));
}
