// Internal interface of the tensor-core GEMMs (quantised weights and bf16 weights).
#pragma once
#include "common.cuh"

namespace qtale {

struct WqGeometry {
  int K_pad;          // K rounded up to a multiple of the group
  int nkb;            // 64-wide K blocks
  int ng;             // groups per row
  int n_tiles;        // 128-row tiles
  int block_bytes;    // code bytes of one (tile, K block)
  int tile_bytes;     // codes + scale / zero words of one (tile, K block)
  int n_rp;           // pairs of row tiles
  size_t sz_offset;   // unused (scale / zero words travel with the codes)
  size_t total;       // blob size in bytes
};

size_t wq_blob_bytes(int N, int K, int bits, int group, int row_mode, WqGeometry* g);

// y = epilogue(a W^T); arguments as qtale_wq_gemm (already validated).
// splitk_ws (optional): scratch of wq_splitk_workspace_bytes() whose first wq_splitk_ticket_bytes()
// hold four regions of counters; region `splitk_slot` must be zero at launch and is left
// non-zero (a layer clears all four once and gives each of its linears its own).  With it,
// products of up to 64 tokens run on the tcgen05 kernel with the K dimension split over the SMs
// (partial tiles through this scratch) instead of the warp-MMA kernel.
size_t wq_splitk_ticket_bytes();
size_t wq_splitk_workspace_bytes();
int wq_gemm_launch(const void* a, int lda, const int32_t* m_dev, int M_cap,
                   const qtale_wq_weight* w, int act, int epilogue, const qtale_epilogue_args* epi,
                   void* y, int ldy, cudaStream_t s, void* splitk_ws = nullptr,
                   size_t splitk_bytes = 0, int splitk_slot = 0);

// y[m, n] = sum_k a[m, k] * w[n, k] with bf16 weights W[N, K] (pitch ldw), fp32 output.
int bf16_gemm_launch(const void* a, int lda, const int32_t* m_dev, int M_cap, const void* w_bf16,
                     int N, int K, int ldw, float* y, int ldy, cudaStream_t s);

}  // namespace qtale
