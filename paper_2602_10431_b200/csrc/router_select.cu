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
constexpr int kBins = 2048;          // first-level histogram of the top-k selection
constexpr int kScoreSmem = 4096;     // a CTA keeps its tokens' scores in shared memory up to this many
constexpr int kCandSmem = 1024;      // candidates ranked in shared memory (more: radix select by one CTA)
constexpr int kMaxGrid = 1024;
constexpr int kLocalHistTokens = 16384;  // up to here every CTA builds the score histogram itself
constexpr uint32_t kSpinLimit = 1u << 20;  // polls of a global word before a wait gives up

// Scratch in the caller's workspace (32-bit words).  The first kZeroWords(grid) words are
// cleared on the stream before every launch; the candidate list needs no clearing.
constexpr int kWsBarrier = 0;      // grid barrier arrivals
constexpr int kWsValid = 1;        // valid tokens of the call
constexpr int kWsCand = 2;         // candidates appended so far
constexpr int kWsCutKey = 3;       // cut-off of the top-k selection (published by CTA 0 when the
constexpr int kWsCutTok = 4;       //   candidates do not fit shared memory)
constexpr int kWsHist = 16;        // kBins counters
constexpr int kWsCount = kWsHist + kBins;  // one word per CTA: executed tokens of its chunk | 2^31
constexpr size_t kWsHeaderBytes = 16384;   // candidates (key, ~token) follow
static_assert((kWsCount + kMaxGrid) * 4 <= (int)kWsHeaderBytes, "scratch header");

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
  int32_t* n_exec_copy;  // optional second destination of the count
  int32_t* cu_exec;
  int32_t* pos;
  uint32_t* ws;
  int* status;
  int T, d, B, mode, k;  // k < 0 (top-k): k = floor(ratio * valid tokens + 0.5), counted here
  int chunk;             // consecutive tokens per CTA
  double ratio;
  float bias, theta;
};

__device__ __forceinline__ uint32_t score_key(float s) {
  uint32_t b = __float_as_uint(s);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
// first-level bin of a score: uniform over [0, 1) (scores are probabilities), monotone for any input
__device__ __forceinline__ int score_bin(float s) {
  return s <= 0.f ? 0 : (s >= 1.f ? kBins - 1 : min(kBins - 1, (int)(s * (float)kBins)));
}
__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(uint32_t* p, uint32_t v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Barrier over the whole (co-resident) grid: arrival number `target` completes it.  Bounded.
__device__ bool grid_barrier(const RouterParams& p, uint32_t target, int* s_abort) {
  __syncthreads();
  if (gridDim.x == 1) return true;  // a single CTA: nothing to wait for, no counter touched
  if (threadIdx.x == 0) {
    __threadfence();
    atomicAdd(p.ws + kWsBarrier, 1u);
    uint32_t it = 0;
    while (ld_acquire(p.ws + kWsBarrier) < target) {
      if (++it > kSpinLimit) {
        *s_abort = 1;
        report_device_error(p.status, QTALE_ERR_TIMEOUT);
        break;
      }
    }
  }
  __syncthreads();
  return *s_abort == 0;
}

// inclusive prefix sum over the CTA's threads in thread order (s_w: one word per warp)
__device__ __forceinline__ int block_inclusive_scan(int v, int* s_w, int& total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  __syncthreads();  // s_w may still be read from the previous use
  if (lane == 31) s_w[wid] = inc;
  __syncthreads();
  int before = 0, tot = 0;
  for (int w = 0; w < nw; ++w) {
    const int c = s_w[w];
    if (w < wid) before += c;
    tot += c;
  }
  total = tot;
  return inc + before;
}

// ---- the fused kernel -------------------------------------------------------
// CTA c owns the consecutive tokens [c * chunk, (c + 1) * chunk).
//   1. scores of its tokens (bandwidth-bound sweep of their rows of x, fp64 accumulation);
//   2. top-k only: after a grid barrier every CTA knows the histogram of all scores over kBins
//      uniform bins (small calls: built by each CTA from the scores of all; large calls:
//      accumulated in global memory during the sweep), finds the bin holding the k-th largest
//      score, collects the (few) tokens of that bin as candidates (small calls: from its own
//      registers; large: a shared list and a second barrier) and ranks them by (score descending,
//      token ascending) to get the cut-off;
//   3. each CTA counts its executed tokens, publishes the count, adds up the counts of the CTAs
//      before it (they publish as soon as they know theirs) and writes its part of the ascending
//      index list, the positions and the per-sequence offsets.
// Launched cooperatively, so all CTAs are resident while they wait for each other.
__global__ void __launch_bounds__(kRouterThreads, 2) router_select_kernel(const RouterParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ float s_sc[kScoreSmem];
  __shared__ uint2 s_cand[kCandSmem];
  __shared__ int s_w[32];
  __shared__ uint32_t s_hist[256];
  __shared__ uint32_t s_h[kBins];
  __shared__ int s_abort, s_bstar, s_rank, s_nvalid, s_ncand, s_fill;
  __shared__ uint32_t s_cut_key, s_cut_tok, s_prefix_hi, s_prefix_lo;

  const int tid = threadIdx.x, nthr = blockDim.x;
  const int lane = tid & 31, wid = tid >> 5, nwarps = nthr >> 5;
  const int T = p.T, G = gridDim.x, cta = blockIdx.x;
  const int c0 = min(T, cta * p.chunk), c1 = min(T, c0 + p.chunk);
  const int n_own = c1 - c0;
  const bool in_smem = p.chunk <= kScoreSmem;
  if (tid == 0) s_abort = 0;

  // cu_seqlens must be 0 = cu[0] <= cu[1] <= ... <= cu[B] = T.  Anything else is reported in the
  // status word; tokens outside [cu[0], cu[B]) then never execute and every walk below stays
  // inside the B + 1 entries.
  const int t_begin = min(max(__ldg(p.cu_seqlens), 0), T);
  const int t_end = min(max(__ldg(p.cu_seqlens + p.B), t_begin), T);
  if (cta == 0) {
    bool bad = tid == 0 && (__ldg(p.cu_seqlens) != 0 || __ldg(p.cu_seqlens + p.B) != T);
    for (int q = tid; q < p.B; q += nthr) bad |= __ldg(p.cu_seqlens + q) > __ldg(p.cu_seqlens + q + 1);
    if (bad) report_device_error(p.status, QTALE_ERR_SHAPE);
  }

  // ---- 1. scores ----
  if (p.scores_override == nullptr) {
    // Router weights staged in shared memory as fp32, laid out [iteration][lane][8] so a lane's
    // eight weights are two 16-byte loads.  Each 16-byte load of x (8 bf16) is reduced with fp32
    // FMAs into a block sum, and the block sums are accumulated in fp64: conversions and fp64
    // adds are one per 8 elements, which keeps the sweep bandwidth bound, and the result stays
    // within about 1e-8 of the all-fp64 dot product.
    float* w_s = reinterpret_cast<float*>(smem_raw);
    const int d = p.d;
    const int n_it = (d + 255) / 256;
    constexpr int kUnroll = 4;  // 16-byte loads in flight per lane: kUnroll x rows per warp
    auto load_block = [&](int r0, int it0, uint4 (&v)[kUnroll][kRowsPerWarp]) {
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int col = (it0 + u) * 256 + lane * 8;
#pragma unroll
        for (int r = 0; r < kRowsPerWarp; ++r) {
          const int row = min(r0 + r, c1 - 1);
          v[u][r] = (it0 + u < n_it && col < d) ? ld_nc_16(p.x + (size_t)row * d + col)
                                                : make_uint4(0, 0, 0, 0);
        }
      }
    };
    const int n_groups = (n_own + kRowsPerWarp - 1) / kRowsPerWarp;
    // the first loads of x are in flight while the router weights are staged
    uint4 v0[kUnroll][kRowsPerWarp];
    if (wid < n_groups) load_block(c0 + wid * kRowsPerWarp, 0, v0);
    for (int i = tid; i < n_it * 256; i += nthr) w_s[i] = (i < d) ? p.w[i] : 0.f;
    __syncthreads();
    for (int g = wid; g < n_groups; g += nwarps) {
      const int r0 = c0 + g * kRowsPerWarp;
      double acc[kRowsPerWarp];
#pragma unroll
      for (int r = 0; r < kRowsPerWarp; ++r) acc[r] = 0.0;
      for (int it0 = 0; it0 < n_it; it0 += kUnroll) {
        uint4 (&v)[kUnroll][kRowsPerWarp] = v0;
        if (it0 != 0 || g != wid) load_block(r0, it0, v);  // the very first block is already there
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
        if (lane == 0 && r0 + r < c1) {
          const float sc = (float)(1.0 / (1.0 + exp(-z)));
          p.scores[r0 + r] = sc;
          if (in_smem) s_sc[r0 + r - c0] = sc;
        }
      }
    }
  } else {
    for (int i = tid; i < n_own; i += nthr) {
      const float sc = p.scores_override[c0 + i];
      p.scores[c0 + i] = sc;
      if (in_smem) s_sc[i] = sc;
    }
  }
  __syncthreads();  // the CTA's scores are in shared memory (or, for huge chunks, in p.scores)

  auto score_at = [&](int i) { return in_smem ? s_sc[i] : p.scores[c0 + i]; };
  auto ok_at = [&](int i) {
    const int t = c0 + i;
    return i < n_own && t >= t_begin && t < t_end && (p.valid == nullptr || p.valid[t] != 0);
  };
  const int n_slab = (n_own + nthr - 1) / nthr;

  // ---- 2. top-k: cut-off = k-th largest (score, lower token first) among the valid tokens ----
  const bool topk = p.mode == QTALE_SELECT_TOPK;
  bool none = false;                        // top-k with k = 0 (or no valid token)
  int bstar = 0;                            // bin of the k-th score
  uint64_t cut = 0;                         // (key << 32 | ~token) of the k-th token
  if (topk) {
    uint32_t step = 0;  // grid barriers passed
    // Calls of up to kLocalHistTokens tokens: after the barrier every CTA reads ALL scores
    // (a few 16-byte loads per thread, issued together), builds the histogram in its own shared
    // memory and keeps the scores in registers for the candidate pass: one barrier, no global
    // atomics.  Larger calls accumulate the histogram in global memory during the sweep.
    const bool local = T <= kLocalHistTokens;
    constexpr int kLocalVec = kLocalHistTokens / (kRouterThreads * 4);  // float4 loads per thread
    float lsc[kLocalVec * 4];
    uint32_t lok = 0;  // bit j: score j of this thread belongs to a valid token
    int n_valid = 0;
    if (local) {
      for (int i = tid; i < kBins; i += nthr) s_h[i] = 0;
      if (tid == 0) s_nvalid = 0;
      if (!grid_barrier(p, ++step * G, &s_abort)) return;
#pragma unroll
      for (int j = 0; j < kLocalVec; ++j) {
        const int t0 = (j * nthr + tid) * 4;
        float4 q = make_float4(0.f, 0.f, 0.f, 0.f);
        if (t0 + 3 < T) {
          q = __ldcg(reinterpret_cast<const float4*>(p.scores + t0));
        } else if (t0 < T) {
          q.x = __ldcg(p.scores + t0);
          if (t0 + 1 < T) q.y = __ldcg(p.scores + t0 + 1);
          if (t0 + 2 < T) q.z = __ldcg(p.scores + t0 + 2);
        }
        lsc[4 * j] = q.x; lsc[4 * j + 1] = q.y; lsc[4 * j + 2] = q.z; lsc[4 * j + 3] = q.w;
      }
      int nv = 0;
#pragma unroll
      for (int j = 0; j < kLocalVec; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int t = (j * nthr + tid) * 4 + e;
          if (t < T && t >= t_begin && t < t_end && (p.valid == nullptr || p.valid[t] != 0)) {
            lok |= 1u << (4 * j + e);
            ++nv;
            atomicAdd(&s_h[score_bin(lsc[4 * j + e])], 1u);
          }
        }
      }
      nv = __reduce_add_sync(0xffffffffu, nv);
      if (lane == 0 && nv) atomicAdd(&s_nvalid, nv);
      __syncthreads();
      n_valid = s_nvalid;
    } else {
      int nv = 0;
      for (int sl = 0; sl < n_slab; ++sl) {
        const int i = sl * nthr + tid;
        if (ok_at(i)) {
          ++nv;
          atomicAdd(p.ws + kWsHist + score_bin(score_at(i)), 1u);
        }
      }
      nv = __reduce_add_sync(0xffffffffu, nv);
      if (lane == 0 && nv) atomicAdd(p.ws + kWsValid, (uint32_t)nv);
      if (!grid_barrier(p, ++step * G, &s_abort)) return;
    }
    // thread j reads bins from the top: tid 0 owns the four highest
    constexpr int PER = kBins / kRouterThreads;
    const int hi_bin = kBins - 1 - tid * PER;
    uint32_t h[PER];
#pragma unroll
    for (int e = 0; e < PER; ++e)
      h[e] = local ? s_h[hi_bin - e] : __ldcg(p.ws + kWsHist + hi_bin - e);
    if (!local) n_valid = (int)__ldcg(p.ws + kWsValid);
    int k = p.k;
    if (k < 0) {  // k for a requested ratio of the valid tokens (padding does not count)
      double kd = floor(p.ratio * (double)n_valid + 0.5);
      k = kd < 0.0 ? 0 : (kd > (double)n_valid ? n_valid : (int)kd);
    }
    k = min(k, n_valid);
    none = k <= 0;
    if (!none) {
      // with `above` = valid tokens in higher bins, the k-th sits in the bin where
      // above < k <= above + count
      int v = 0;
#pragma unroll
      for (int e = 0; e < PER; ++e) v += (int)h[e];
      int total;
      int above = block_inclusive_scan(v, s_w, total) - v;
#pragma unroll
      for (int e = 0; e < PER; ++e) {
        if (above < k && k <= above + (int)h[e]) {
          s_bstar = hi_bin - e;
          s_rank = k - above;       // 1-based rank of the k-th inside its bin
          s_ncand = (int)h[e];      // tokens in that bin
        }
        above += (int)h[e];
      }
      __syncthreads();
      bstar = s_bstar;
      const int r = s_rank, c = s_ncand;
      uint2* cand = reinterpret_cast<uint2*>(reinterpret_cast<unsigned char*>(p.ws) + kWsHeaderBytes);
      // candidates = the valid tokens of bin bstar
      if (local && c <= kCandSmem) {
        if (tid == 0) s_fill = 0;
        __syncthreads();
#pragma unroll
        for (int j = 0; j < kLocalVec * 4; ++j) {
          if (((lok >> j) & 1u) && score_bin(lsc[j]) == bstar) {
            const int slot = atomicAdd(&s_fill, 1);
            if (slot < kCandSmem)
              s_cand[slot] = make_uint2(score_key(lsc[j]), ~(uint32_t)(((j >> 2) * nthr + tid) * 4 + (j & 3)));
          }
        }
        __syncthreads();
      } else {
        for (int sl = 0; sl < n_slab; ++sl) {
          const int i = sl * nthr + tid;
          if (ok_at(i)) {
            const float sc = score_at(i);
            if (score_bin(sc) == bstar) {
              const uint32_t slot = atomicAdd(p.ws + kWsCand, 1u);
              if (slot < (uint32_t)T) cand[slot] = make_uint2(score_key(sc), ~(uint32_t)(c0 + i));
            }
          }
        }
        if (!grid_barrier(p, ++step * G, &s_abort)) return;
        if (c <= kCandSmem) {
          for (int i = tid; i < c; i += nthr) s_cand[i] = __ldcg(cand + i);
          __syncthreads();
        }
      }
      if (c <= kCandSmem) {
        // every CTA ranks the candidates itself: the r-th in the order is the cut-off
        for (int i = tid; i < c; i += nthr) {
          const uint64_t me = ((uint64_t)s_cand[i].x << 32) | s_cand[i].y;
          int before = 0;
          for (int j = 0; j < c; ++j)
            before += ((((uint64_t)s_cand[j].x << 32) | s_cand[j].y) > me) ? 1 : 0;
          if (before == r - 1) {
            s_cut_key = s_cand[i].x;
            s_cut_tok = s_cand[i].y;
          }
        }
        __syncthreads();
      } else {
        // many equal or close scores: CTA 0 finds the r-th largest 64-bit (key, ~token) by an
        // MSB-first radix select over the list in global memory and publishes it
        if (cta == 0) {
          if (tid == 0) {
            s_prefix_hi = 0;
            s_prefix_lo = 0;
            s_rank = r;
          }
          for (int pass = 0; pass < 8; ++pass) {
            const int shift = 56 - 8 * pass;
            for (int i = tid; i < 256; i += nthr) s_hist[i] = 0;
            __syncthreads();
            const uint64_t prefix = ((uint64_t)s_prefix_hi << 32) | s_prefix_lo;
            const uint64_t mask = pass == 0 ? 0ull : ~0ull << (shift + 8);
            for (int i = tid; i < c; i += nthr) {
              const uint2 e = __ldcg(cand + i);
              const uint64_t v64 = ((uint64_t)e.x << 32) | e.y;
              if ((v64 & mask) == prefix) atomicAdd(&s_hist[(uint32_t)(v64 >> shift) & 0xFFu], 1u);
            }
            __syncthreads();
            if (tid == 0) {
              int rem = s_rank, digit = 0;
              for (int b = 255; b >= 0; --b) {
                const int cnt = (int)s_hist[b];
                if (rem <= cnt) { digit = b; break; }
                rem -= cnt;
              }
              const uint64_t np = prefix | ((uint64_t)digit << shift);
              s_prefix_hi = (uint32_t)(np >> 32);
              s_prefix_lo = (uint32_t)np;
              s_rank = rem;
            }
            __syncthreads();
          }
          if (tid == 0) {
            p.ws[kWsCutKey] = s_prefix_hi;
            p.ws[kWsCutTok] = s_prefix_lo;
          }
        }
        if (!grid_barrier(p, ++step * G, &s_abort)) return;
        if (tid == 0) {
          s_cut_key = __ldcg(p.ws + kWsCutKey);
          s_cut_tok = __ldcg(p.ws + kWsCutTok);
        }
        __syncthreads();
      }
      cut = ((uint64_t)s_cut_key << 32) | s_cut_tok;
    }
  }

  // execute / bypass decision of the CTA's token i
  auto decide = [&](int i) {
    if (!ok_at(i)) return false;
    const float sc = score_at(i);
    if (!topk) return sc >= p.theta;
    if (none) return false;
    const int b = score_bin(sc);
    if (b != bstar) return b > bstar;
    return (((uint64_t)score_key(sc) << 32) | ~(uint32_t)(c0 + i)) >= cut;
  };

  // ---- 3. ordered compaction ----
  int own = 0;
  for (int sl = 0; sl < n_slab; ++sl) own += __syncthreads_count(decide(sl * nthr + tid) ? 1 : 0);
  if (tid == 0) st_release(p.ws + kWsCount + cta, (uint32_t)own | 0x80000000u);
  // executed tokens of the CTAs before this one
  int before = 0;
  for (int j = tid; j < cta; j += nthr) {
    uint32_t v, it = 0;
    while (((v = ld_acquire(p.ws + kWsCount + j)) & 0x80000000u) == 0) {
      if (++it > kSpinLimit) {
        s_abort = 1;
        report_device_error(p.status, QTALE_ERR_TIMEOUT);
        break;
      }
    }
    before += (int)(v & 0x7FFFFFFFu);
  }
  {
    int total;
    block_inclusive_scan(before, s_w, total);
    before = total;
  }
  __syncthreads();
  if (s_abort) return;

  const uint32_t lt = (1u << lane) - 1u;
  int run = before;  // executed tokens before the current slab
  for (int sl = 0; sl < n_slab; ++sl) {
    const int i = sl * nthr + tid;
    const int t = c0 + i;
    const bool take = decide(i);
    const uint32_t m_take = __ballot_sync(0xffffffffu, take);
    __syncthreads();
    if (lane == 0) s_w[wid] = __popc(m_take);
    __syncthreads();
    int wbase = 0, slab_total = 0;
    for (int w = 0; w < nwarps; ++w) {
      const int c = s_w[w];
      if (w < wid) wbase += c;
      slab_total += c;
    }
    const int my_out = run + wbase + __popc(m_take & lt);  // executed tokens before token t
    if (i < n_own) {
      // b = sequence holding t (largest b with cu_seqlens[b] <= t)
      int lo = 0, hi = p.B;
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(p.cu_seqlens + mid) <= t) lo = mid; else hi = mid;
      }
      const int seq_start = __ldg(p.cu_seqlens + lo);
      if (t == seq_start) {  // first token of sequence lo and of the empty sequences before it
        for (int q = lo; q >= 0 && __ldg(p.cu_seqlens + q) == t; --q) p.cu_exec[q] = my_out;
      }
      if (take) {
        p.idx[my_out] = t;
        p.pos[my_out] = t - seq_start + (p.pos0 ? __ldg(p.pos0 + lo) : 0);
      }
    }
    run += slab_total;
  }
  if (cta == G - 1) {
    if (tid == 0) {
      *p.n_exec = run;
      if (p.n_exec_copy) *p.n_exec_copy = run;
    }
    for (int q = tid; q <= p.B; q += nthr)
      if (__ldg(p.cu_seqlens + q) >= T) p.cu_exec[q] = run;
  }
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
  // counters, histogram and per-CTA counts, then one (key, token) pair per token for the
  // candidates of the top-k selection (all of them when every score is the same)
  return kWsHeaderBytes + (size_t)(T > 0 ? T : 0) * 8;
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
                         size_t ws_bytes, cudaStream_t s, int32_t* n_exec_copy) {
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
  p.n_exec_copy = n_exec_copy;
  p.cu_exec = cu_exec_out;
  p.pos = pos_out;
  p.ws = static_cast<uint32_t*>(ws);
  p.status = device_status_ptr();
  p.T = T; p.d = d; p.B = B; p.mode = mode;
  p.k = (mode == QTALE_SELECT_TOPK && ratio >= 0.0) ? -1 : k;
  p.ratio = ratio;
  p.bias = bias; p.theta = theta;

  const size_t smem = scores_override ? 0 : (size_t)((d + 255) / 256) * 256 * sizeof(float);
  // The CTAs wait for each other, so the grid must fit the device at once: at most what the
  // occupancy calculator allows, at least 32 tokens per CTA (two per warp), an even chunk.
  static int cached_dev = -1, cached_per_sm = 0;
  static size_t cached_smem = 0;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return QTALE_ERR_CUDA;
  if (dev != cached_dev || smem != cached_smem) {
    if (smem > 0 &&  // static + dynamic shared memory may exceed the default 48 KB
        cudaFuncSetAttribute(router_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)smem) != cudaSuccess)
      return QTALE_ERR_CUDA;
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, router_select_kernel, kRouterThreads,
                                                      smem) != cudaSuccess || per_sm < 1)
      return QTALE_ERR_CUDA;
    cached_per_sm = per_sm > 2 ? 2 : per_sm;
    cached_dev = dev;
    cached_smem = smem;
  }
  int grid = sm_count() * cached_per_sm;
  if (grid > kMaxGrid) grid = kMaxGrid;
  // with the scores supplied there is no sweep of x to spread: one CTA per 1024 tokens
  const int want = scores_override ? (T + 1023) / 1024 : (T + 31) / 32;
  if (grid > want) grid = want;
  int chunk = (T + grid - 1) / grid;
  chunk = (chunk + 1) & ~1;
  grid = (T + chunk - 1) / chunk;
  p.chunk = chunk;

  // a single CTA (decode steps, small calls) neither waits nor counts: nothing to clear
  if (grid > 1 &&
      cudaMemsetAsync(ws, 0, (size_t)(kWsCount + grid) * sizeof(uint32_t), s) != cudaSuccess)
    return QTALE_ERR_CUDA;
  void* args[] = {&p};
  return launch_status(cudaLaunchCooperativeKernel(router_select_kernel, dim3(grid),
                                                   dim3(kRouterThreads), args, smem, s));
}

}  // namespace qtale

extern "C" {

// ---- variant for callers that cannot allocate device memory -------------------
// The kernel's scratch (counters, histogram, per-CTA counts and the candidate list of the
// top-k selection) lives in a static device array, sized for QTALE_ROUTER_STATIC_MAX_TOKENS
// tokens, that every GPU loading the library carries until exit.
#define QTALE_ROUTER_STATIC_SCRATCH_BYTES (16384 + 8 * QTALE_ROUTER_STATIC_MAX_TOKENS)
static_assert(QTALE_ROUTER_STATIC_SCRATCH_BYTES >= kWsHeaderBytes + 8 * (size_t)QTALE_ROUTER_STATIC_MAX_TOKENS,
              "static scratch must cover the workspace of the largest accepted call");
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
  // The shared entry point clears the counters (cudaMemsetAsync on the stream) before
  // the launch, so whatever the previous call left behind does not matter.
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
