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
int wq_gemm_launch(const void* a, int lda, const int32_t* m_dev, int M_cap,
                   const qtale_wq_weight* w, int act, int epilogue, const qtale_epilogue_args* epi,
                   void* y, int ldy, cudaStream_t s);

// y[m, n] = sum_k a[m, k] * w[n, k] with bf16 weights W[N, K] (pitch ldw), fp32 output.
int bf16_gemm_launch(const void* a, int lda, const int32_t* m_dev, int M_cap, const void* w_bf16,
                     int N, int K, int ldw, float* y, int ldy, cudaStream_t s);

}  // namespace qtale
