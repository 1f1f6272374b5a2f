// Causal attention among the executed tokens of each sequence (prefill) on the
// tcgen05 tensor cores (Eq. 3: bypassed tokens have no query, key or value here).
//
// A work item is 256 consecutive executed tokens of one sequence and one head, handled as two
// query tiles A and B of 128 rows that share one stream of key / value tiles (128 keys each).
// The grid is persistent (one CTA per SM walks the items sequence by sequence).  Per query
// tile X and key tile j:
//   S_X = Q_X K^T   SS MMA, Q and K tiles from 128-byte-swizzled shared memory (TMA), fp32
//                   scores in tensor memory (128 columns per query tile);
//   softmax         four warps per query tile, one thread per query row: the 128 scores of the
//                   row in registers, running max / sum in the log2 domain (one fma and one
//                   ex2.approx per score), probabilities written over the scores' own columns in
//                   the 16-bit activation format (the A operand of the next MMA);
//   O_X += P_X V    TS MMA with V read straight from its row-major tile (MN-major B operand),
//                   fp32 output accumulator in tensor memory, rescaled by the softmax warps only
//                   when a row's maximum has outgrown the softmax reference by 2^8.
// Scores, probabilities and outputs of both tiles fill the 512 tensor-memory columns, so a
// tile's next scores can only be computed once its probabilities have been consumed; the two
// tiles alternate instead: while the warps of one tile are in their softmax (bound by the
// special-function unit) the tensor pipe works on P V and Q K^T of the other.  The single
// issuing thread orders the work A, B, A, B, ...: P_X V (j), then Q_X K^T (j + 1).
// Tile B of the last item of a sequence may lie wholly behind the sequence: it is skipped.
// Warp roles (384 threads): warp 0 Q / K producer, warp 1 MMA issuer and TMEM allocator,
// warp 2 V producer, warps 4-7 softmax of tile A, warps 8-11 of tile B.  Every wait is bounded.
#include <cuda.h>

#include <string.h>

#include "attention.cuh"
#include "ptx.cuh"

namespace qtale {

using namespace ptx;

constexpr int kTcThreads = 384;
constexpr int kTcKStages = 2;    // key tiles in flight
constexpr int kTcVStages = 2;    // value tiles in flight
constexpr int kTcTile = 128;     // query rows per tile and keys per tile
constexpr int kTcItemRows = 2 * kTcTile;
constexpr uint32_t kTcSlices = 1u << 16;  // suspended barrier tests before a wait gives up
constexpr float kTcMaxSlack = 8.f;        // log2 growth of a row maximum that moves the softmax reference

struct TcShared {
  uint64_t q_full, q_empty;
  uint64_t k_full[kTcKStages], k_empty[kTcKStages];
  uint64_t v_full[kTcVStages], v_empty[kTcVStages];
  uint64_t s_full[2], p_full[2], pv_done[2], o_empty[2];  // per query tile
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

// Work items of the persistent grid: (sequence, block of 256 query rows, head), a block for every
// head.  An item's cost grows with its block index (causal attention), and each CTA takes its
// items in a fixed pattern, so the order of the list decides the balance.  Two orders:
//  * level order, when the keys and values of the whole call fit the L2 cache: the last blocks of
//    all sequences first, then the blocks before them, ... (cost descending), dealt to the CTAs
//    forwards and backwards in alternate rounds, so a CTA that drew the dearest item of one round
//    draws the cheapest of the next;
//  * sequence order otherwise: sequence by sequence (longest block first in even sequences,
//    shortest first in odd ones), dealt round-robin.  The CTAs running at one time then work on
//    one or two sequences, whose keys and values stay in L2 (with all sequences live at once they
//    were re-read from DRAM several times).
// A cursor only moves forward: the k-th item of a CTA has a larger index than its (k-1)-th.
constexpr long long kTcLevelOrderBytes = 72ll << 20;

struct ItemCursor {
  int seq;    // sequence (sequence order) or level (level order) being enumerated
  int base;   // index of its first item
  int nt;     // its blocks (sequence order) or sequences (level order); -1: not counted yet
};

struct ItemOrder {
  bool level;      // level order
  int max_blocks;  // blocks of the longest sequence
  int n_items;
};

__device__ __forceinline__ int seq_blocks(const TcParams& p, int s) {
  return (p.cu_exec[s + 1] - p.cu_exec[s] + kTcItemRows - 1) / kTcItemRows;
}

__device__ __forceinline__ ItemOrder item_order(const TcParams& p, int hd) {
  ItemOrder o;
  int n_blocks = 0;
  o.max_blocks = 0;
  for (int s = 0; s < p.B; ++s) {
    const int nb = seq_blocks(p, s);
    n_blocks += nb;
    o.max_blocks = max(o.max_blocks, nb);
  }
  o.n_items = n_blocks * p.H;
  const long long kv_bytes = (long long)(p.cu_exec[p.B] - p.cu_exec[0]) * (p.H / p.rep) * hd * 4;
  o.level = kv_bytes <= kTcLevelOrderBytes;
  return o;
}

// index of the r-th item of CTA c (grid g)
__device__ __forceinline__ int item_index(const ItemOrder& o, int r, int c, int g) {
  return r * g + ((o.level && (r & 1)) ? g - 1 - c : c);
}

// item i (i must not decrease between calls) -> sequence, head, query block; false past the end
__device__ __forceinline__ bool item_at(const TcParams& p, const ItemOrder& o, ItemCursor& c, int i, int& b,
                                        int& h, int& qb) {
  if (o.level) {
    while (c.seq < o.max_blocks) {
      qb = o.max_blocks - 1 - c.seq;
      if (c.nt < 0) {
        c.nt = 0;
        for (int s = 0; s < p.B; ++s) c.nt += seq_blocks(p, s) > qb ? 1 : 0;
      }
      const int n = c.nt * p.H;
      if (i < c.base + n) {
        const int r = i - c.base;
        h = r % p.H;
        int k = r / p.H;  // the k-th sequence that has this block
        b = 0;
        for (int s = 0; s < p.B; ++s)
          if (seq_blocks(p, s) > qb) {
            if (k == 0) { b = s; break; }
            --k;
          }
        return true;
      }
      c.base += n;
      c.nt = -1;
      ++c.seq;
    }
    return false;
  }
  while (c.seq < p.B) {
    if (c.nt < 0) c.nt = seq_blocks(p, c.seq);
    const int n = c.nt * p.H;
    if (i < c.base + n) {
      const int r = i - c.base;
      b = c.seq;
      h = r % p.H;
      qb = (c.seq & 1) ? r / p.H : c.nt - 1 - r / p.H;
      return true;
    }
    c.base += n;
    c.nt = -1;
    ++c.seq;
  }
  return false;
}

// What an item asks of the two query tiles
struct ItemShape {
  int seq0, len;
  int jA, jB;   // last key tile of query tile A / B (B = -1 when its rows lie behind the sequence)
  int nj;       // key tiles the item streams
};

__device__ __forceinline__ ItemShape item_shape(const TcParams& p, int b, int qb) {
  ItemShape s;
  s.seq0 = p.cu_exec[b];
  s.len = p.cu_exec[b + 1] - s.seq0;
  s.jA = 2 * qb;
  s.jB = (qb * kTcItemRows + kTcTile < s.len) ? 2 * qb + 1 : -1;
  s.nj = (s.jB >= 0 ? s.jB : s.jA) + 1;
  return s;
}

template <int HD, int ACT>
__global__ void __launch_bounds__(kTcThreads, 1)
    attn_prefill_tc_kernel(const __grid_constant__ CUtensorMap tmap, const TcParams p) {
  constexpr int CH = HD / 64;                       // 16 KB chunks per tile
  constexpr int TILE_BYTES = kTcTile * HD * 2;
  constexpr int S_COL = 0;                          // scores of tile X: 128 columns at 128 X; its
                                                    // probabilities reuse the first 64 of them
  constexpr int O_COL = 256;                        // output accumulator of tile X: HD columns at 256 + 128 X
  extern __shared__ unsigned char smem_dyn[];
  __shared__ TcShared sh;
  unsigned char* base = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
  unsigned char* sQ = base;                                  // tiles A and B
  unsigned char* sK = base + 2 * TILE_BYTES;                 // kTcKStages stages
  unsigned char* sV = base + (2 + kTcKStages) * TILE_BYTES;  // kTcVStages stages

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const ItemOrder order = item_order(p, HD);
  const int n_items = order.n_items;
  if ((int)blockIdx.x >= n_items) return;  // uniform for the CTA: nothing allocated yet

  if (threadIdx.x == 0) {
    mbar_init(&sh.q_full, 1);
    mbar_init(&sh.q_empty, 1);
    for (int s = 0; s < kTcKStages; ++s) {
      mbar_init(&sh.k_full[s], 1);
      mbar_init(&sh.k_empty[s], 1);
    }
    for (int s = 0; s < kTcVStages; ++s) {
      mbar_init(&sh.v_full[s], 1);
      mbar_init(&sh.v_empty[s], 1);
    }
    for (int x = 0; x < 2; ++x) {
      mbar_init(&sh.s_full[x], 1);
      mbar_init(&sh.p_full[x], 4);   // the four softmax warps of the tile
      mbar_init(&sh.pv_done[x], 1);
      mbar_init(&sh.o_empty[x], 4);
    }
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

  // every role walks the same item sequence with its own cursor and its own running counters
  // (key / value tiles so far pick the ring stage and phase; tiles so far of query tile X the
  // phase of X's barriers)
  ItemCursor cur;
  cur.seq = 0;
  cur.base = 0;
  cur.nt = -1;

  if (warp == 0) {
    // ------------------------------ TMA producer: queries and keys ------------------------------
    if (lane == 0) {
      uint32_t t = 0, it = 0;
      for (int rd = 0;; ++rd, ++it) {
        const int item = item_index(order, rd, blockIdx.x, gridDim.x);
        int b, h, qb;
        if (item >= n_items || !item_at(p, order, cur, item, b, h, qb)) break;
        const ItemShape is = item_shape(p, b, qb);
        const int hk = h / p.rep;
        const int n_q = is.jB >= 0 ? 2 : 1;
        if (!tc_wait(&sh.q_empty, (it & 1u) ^ 1u, &sh, p.status)) break;
        mbar_arrive_expect_tx(&sh.q_full, (uint32_t)(n_q * TILE_BYTES));
        for (int x = 0; x < n_q; ++x)
          for (int c = 0; c < CH; ++c)
            tma_load_2d(sQ + x * TILE_BYTES + c * 16384, &tmap, &sh.q_full, h * HD + c * 64,
                        is.seq0 + qb * kTcItemRows + x * kTcTile);
        bool ok = true;
        for (int j = 0; j < is.nj; ++j, ++t) {
          const int s = t % kTcKStages;
          const uint32_t ph = (t / kTcKStages) & 1u;
          if (!tc_wait(&sh.k_empty[s], ph ^ 1u, &sh, p.status)) { ok = false; break; }
          mbar_arrive_expect_tx(&sh.k_full[s], TILE_BYTES);
          for (int c = 0; c < CH; ++c)
            tma_load_2d(sK + s * TILE_BYTES + c * 16384, &tmap, &sh.k_full[s],
                        p.k_off + hk * HD + c * 64, is.seq0 + j * kTcTile);
        }
        if (!ok) break;
      }
    }
  } else if (warp == 2) {
    // ------------------------------ TMA producer of the value tiles ------------------------------
    // (a thread of its own: a full value ring must not hold back the key loads)
    if (lane == 0) {
      uint32_t t = 0;
      bool ok = true;
      for (int rd = 0; ok; ++rd) {
        const int item = item_index(order, rd, blockIdx.x, gridDim.x);
        int b, h, qb;
        if (item >= n_items || !item_at(p, order, cur, item, b, h, qb)) break;
        const ItemShape is = item_shape(p, b, qb);
        const int hk = h / p.rep;
        for (int j = 0; j < is.nj; ++j, ++t) {
          const int s = t % kTcVStages;
          const uint32_t ph = (t / kTcVStages) & 1u;
          if (!tc_wait(&sh.v_empty[s], ph ^ 1u, &sh, p.status)) { ok = false; break; }
          mbar_arrive_expect_tx(&sh.v_full[s], TILE_BYTES);
          for (int c = 0; c < CH; ++c)
            tma_load_2d(sV + s * TILE_BYTES + c * 16384, &tmap, &sh.v_full[s],
                        p.v_off + hk * HD + c * 64, is.seq0 + j * kTcTile);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer -------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc_qk = idesc_16bit_f32(128, kTcTile, ACT == 1);
      constexpr uint32_t idesc_pv = idesc_16bit_f32(128, HD, ACT == 1) | (1u << 16);  // B is MN-major
      const uint32_t qa = smem_u32(sQ);
      // scores of query tile x against the key tile in ring stage ks
      auto issue_qk = [&](int x, int ks) {
        const uint32_t ka = smem_u32(sK + ks * TILE_BYTES);
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk)
          mma_ss(tmem + S_COL + x * 128, kmajor_desc(qa + x * TILE_BYTES, kk), kmajor_desc(ka, kk), idesc_qk,
                 kk != 0 ? 1u : 0u);
        mma_commit(&sh.s_full[x]);
      };
      auto issue_pv = [&](int x, int vs, bool first) {
        const uint32_t va = smem_u32(sV + vs * TILE_BYTES);
#pragma unroll
        for (int kk = 0; kk < kTcTile / 16; ++kk)
          mma_ts(tmem + O_COL + x * 128, tmem + S_COL + x * 128 + kk * 8, v_desc(va, kk), idesc_pv,
                 (first && kk == 0) ? 0u : 1u);
        mma_commit(&sh.pv_done[x]);
      };
      uint32_t tk = 0, tv = 0, it = 0;
      uint32_t cx[2] = {0, 0};    // tiles so far of query tile x
      uint32_t itx[2] = {0, 0};   // items so far in which query tile x took part
      bool ok = true;
      for (int rd = 0; ok; ++rd, ++it) {
        const int item = item_index(order, rd, blockIdx.x, gridDim.x);
        int b, h, qb;
        if (item >= n_items || !item_at(p, order, cur, item, b, h, qb)) break;
        const ItemShape is = item_shape(p, b, qb);
        const bool has_b = is.jB >= 0;
        if (!tc_wait(&sh.q_full, it & 1u, &sh, p.status)) break;
        {
          const int ks = tk % kTcKStages;
          if (!tc_wait(&sh.k_full[ks], (tk / kTcKStages) & 1u, &sh, p.status)) break;
          tc_fence_after();
          issue_qk(0, ks);
          if (has_b) issue_qk(1, ks);
          mma_commit(&sh.k_empty[ks]);
          if (is.nj == 1) mma_commit(&sh.q_empty);  // the query tiles have been read for the last time
        }
        for (int j = 0; ok && j < is.nj; ++j) {
          const int vs = (tv + j) % kTcVStages;
          const uint32_t vph = ((tv + j) / kTcVStages) & 1u;
          const int ks1 = (tk + j + 1) % kTcKStages;
          const uint32_t kph1 = ((tk + j + 1) / kTcKStages) & 1u;
          // Every barrier this key tile (at most 32 MMAs) will need is tested once up front, without
          // blocking: in the steady state all of them are complete, and the MMAs then follow one
          // another without a barrier's round trip between the groups, during which the tensor
          // pipe would drain.  What is not complete yet is waited for where it is needed.
          bool p_ok[2];
          p_ok[0] = j <= is.jA && mbar_try_wait(&sh.p_full[0], cx[0] & 1u);
          p_ok[1] = j <= is.jB && mbar_try_wait(&sh.p_full[1], cx[1] & 1u);
          bool v_ok = mbar_try_wait(&sh.v_full[vs], vph);
          bool k_ok = j + 1 < is.nj && mbar_try_wait(&sh.k_full[ks1], kph1);
#pragma unroll
          for (int x = 0; x < 2; ++x) {
            const int jx = x == 0 ? is.jA : is.jB;
            if (j > jx) continue;
            // P_x V of this key tile, then the scores of the next one (they overwrite P_x: the
            // tensor pipe runs the two in issue order)
            if (!p_ok[x] && !tc_wait(&sh.p_full[x], cx[x] & 1u, &sh, p.status)) { ok = false; break; }
            // the first P V of an item overwrites the accumulator: the previous item's output
            // must have been read
            if (j == 0 && !tc_wait(&sh.o_empty[x], (itx[x] & 1u) ^ 1u, &sh, p.status)) { ok = false; break; }
            if (!v_ok && !tc_wait(&sh.v_full[vs], vph, &sh, p.status)) { ok = false; break; }
            v_ok = true;
            tc_fence_after();
            issue_pv(x, vs, j == 0);
            ++cx[x];
            const bool last_v_user = x == 1 || !(has_b && j <= is.jB);
            if (last_v_user) mma_commit(&sh.v_empty[vs]);
            if (j + 1 <= jx) {
              if (!k_ok && !tc_wait(&sh.k_full[ks1], kph1, &sh, p.status)) { ok = false; break; }
              k_ok = true;
              tc_fence_after();
              issue_qk(x, ks1);
              const bool last_k_user = x == 1 || !has_b;
              if (last_k_user) {
                mma_commit(&sh.k_empty[ks1]);
                if (j + 2 == is.nj) mma_commit(&sh.q_empty);
              }
            }
          }
        }
        tk += is.nj;
        tv += is.nj;
        ++itx[0];
        if (has_b) ++itx[1];
      }
    }
  } else if (warp >= 4) {
    // ---------- softmax, correction and output of one query tile: one thread per query row ----------
    // Warps 4-7 serve tile A, warps 8-11 tile B; a warp reaches the TMEM lanes 32 (warp % 4) .. + 31.
    const int x = (warp - 4) >> 2;
    const int quad = warp & 3;
    const int row = quad * 32 + lane;          // TMEM lane = query row of the tile
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const uint32_t s_addr = tmem + lane_addr + S_COL + x * 128;
    const uint32_t o_addr = tmem + lane_addr + O_COL + x * 128;
    uint32_t c = 0, itx = 0;   // tiles / items so far of this query tile
    bool alive = true;
    for (int rd = 0; alive; ++rd) {
      const int item = item_index(order, rd, blockIdx.x, gridDim.x);
      int b, h, qb;
      if (item >= n_items || !item_at(p, order, cur, item, b, h, qb)) break;
      const ItemShape is = item_shape(p, b, qb);
      const int jx = x == 0 ? is.jA : is.jB;
      if (jx < 0) continue;  // tile B lies behind the sequence
      const int len = is.len;
      const int q_row = qb * kTcItemRows + x * kTcTile + row;
      float m_run = -INFINITY, l_run = 0.f;
      for (int j = 0; j <= jx && alive; ++j) {
        if (!tc_wait(&sh.s_full[x], c & 1u, &sh, p.status)) { alive = false; break; }
        tc_fence_after();
        // the row's 128 scores in registers, unscaled; the scale (positive) is folded into the
        // exponent's multiply-add, so an element costs one max, one fma, one ex2, one add
        uint32_t sc[4][32];
        tmem_ld_x32(s_addr, sc[0]);
        tmem_ld_x32(s_addr + 32, sc[1]);
        tmem_ld_x32(s_addr + 64, sc[2]);
        tmem_ld_x32(s_addr + 96, sc[3]);
        tmem_wait_ld();
        if (j == jx || j * kTcTile + kTcTile > len) {
#pragma unroll
          for (int cc = 0; cc < 4; ++cc)
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const int key = j * kTcTile + cc * 32 + i;
              if (key > q_row || key >= len) sc[cc][i] = 0xFF800000u;  // -inf
            }
        }
        float mq[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int cc = 0; cc < 4; ++cc)
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            mq[0] = fmaxf(mq[0], __uint_as_float(sc[cc][i]));
            mq[1] = fmaxf(mq[1], __uint_as_float(sc[cc][i + 1]));
            mq[2] = fmaxf(mq[2], __uint_as_float(sc[cc][i + 2]));
            mq[3] = fmaxf(mq[3], __uint_as_float(sc[cc][i + 3]));
          }
        const float row_raw = fmaxf(fmaxf(mq[0], mq[1]), fmaxf(mq[2], mq[3]));
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
        const float neg_m = (m_run == -INFINITY) ? 0.f : -m_run;
        // probabilities in the 16-bit format, two keys per 32-bit column, written over the first
        // 64 score columns (every score is in registers by now)
        float sq[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
          uint32_t pr[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float p0 = ex2_approx(fmaf(__uint_as_float(sc[cc][2 * i]), p.scale_log2, neg_m));
            const float p1 = ex2_approx(fmaf(__uint_as_float(sc[cc][2 * i + 1]), p.scale_log2, neg_m));
            sq[i & 3] += p0 + p1;
            pr[i] = Act16<ACT>::pack(p0, p1);
          }
          tmem_st_x16(s_addr + cc * 16, pr);
        }
        l_run += (sq[0] + sq[1]) + (sq[2] + sq[3]);
        // The previous P V of this tile was issued before these scores and is complete; the wait
        // keeps the barrier's phase in step, and the fence orders the rescaling after it.
        if (j > 0) {
          if (!tc_wait(&sh.pv_done[x], (c - 1) & 1u, &sh, p.status)) { alive = false; break; }
          tc_fence_after();
          if (__any_sync(0xffffffffu, moved)) {
#pragma unroll 1
            for (int cc = 0; cc < HD / 32; ++cc) {
              uint32_t r[32];
              tmem_ld_x32(o_addr + cc * 32, r);
              tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * corr);
              tmem_st_x32(o_addr + cc * 32, r);
            }
          }
        }
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.p_full[x]);
        ++c;
      }
      if (!alive) break;
      // output: O / l for the rows that exist; then the accumulator is handed back
      if (!tc_wait(&sh.pv_done[x], (c - 1) & 1u, &sh, p.status)) { alive = false; break; }
      tc_fence_after();
      const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
      unsigned short* out = static_cast<unsigned short*>(p.out) + (size_t)(is.seq0 + q_row) * p.ldo +
                            (size_t)h * HD;
#pragma unroll 1
      for (int cc = 0; cc < HD / 32; ++cc) {
        uint32_t r[32];
        tmem_ld_x32(o_addr + cc * 32, r);
        tmem_wait_ld();
        if (cc == HD / 32 - 1) {  // every column of this warp's rows is in registers
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sh.o_empty[x]);
        }
        if (q_row < len) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint4 o;
            o.x = Act16<ACT>::pack(__uint_as_float(r[8 * i + 0]) * inv, __uint_as_float(r[8 * i + 1]) * inv);
            o.y = Act16<ACT>::pack(__uint_as_float(r[8 * i + 2]) * inv, __uint_as_float(r[8 * i + 3]) * inv);
            o.z = Act16<ACT>::pack(__uint_as_float(r[8 * i + 4]) * inv, __uint_as_float(r[8 * i + 5]) * inv);
            o.w = Act16<ACT>::pack(__uint_as_float(r[8 * i + 6]) * inv, __uint_as_float(r[8 * i + 7]) * inv);
            st_16(out + cc * 32 + i * 8, o);
          }
        }
      }
      ++itx;
    }
    (void)itx;
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
  const size_t smem = (size_t)(2 + kTcKStages + kTcVStages) * kTcTile * HD * 2 + 1024;
  static bool configured[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    if (cudaFuncSetAttribute(attn_prefill_tc_kernel<HD, ACT>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return QTALE_ERR_CUDA;
    configured[dev] = true;
  }
  // persistent grid: one CTA per SM walks the (sequence, block of 256 query rows, head) items
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
