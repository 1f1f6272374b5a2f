// Launchers of the bandwidth-bound row kernels (internal to libqtale).
#pragma once
#include "common.cuh"

namespace qtale {

// Work the gather kernel can do on the side for the layer (all optional, see compact_kernel).
struct GatherExtras {
  const int32_t* pos;  // [cap] positions of the executed tokens
  float2* cs;          // rotary table out: [cap, half] (cos, sin); NULL: none
  int half;            // head_dim / 2 (at most 128)
  float rope_base;
  uint4* tail;         // 16-bit [cap, tail_ld] tensor whose rows after the count are cleared; NULL: none
  int tail_ld, tail_col0, tail_cols, tail_rows;  // elements (multiples of 8), rows
};

int launch_compact(const void* x, const int32_t* idx, const int32_t* n_exec, int cap, int d,
                   const float* gamma, float eps, int act, void* xc, void* hn, cudaStream_t s,
                   const GatherExtras* extras = nullptr);
int launch_scatter_add(void* x, const void* xc, const float* f, const int32_t* idx,
                       const int32_t* n_exec, int cap, int d, cudaStream_t s);
// RMSNorm of fp32 rows into bf16; n_rows may be NULL (all `cap` rows).
int launch_rmsnorm_f32(const float* u, const int32_t* n_rows, int cap, int d, const float* gamma,
                       float eps, int act, void* out, cudaStream_t s);
int launch_rope(void* qkv, const int32_t* n_exec, int cap, int ld, int n_rot, int hd,
                const float* cs, int act, cudaStream_t s);
int launch_swiglu(const void* gu, const int32_t* n_exec, int cap, int F, void* act, int act_dtype,
                  cudaStream_t s);
int launch_kv_append(const void* qkv, const int32_t* n_exec, int cap_rows, int ld, int q_dim,
                     int kv_dim, int hd, const int32_t* cu_exec, int B, void* cache_k, void* cache_v,
                     int32_t* kv_len, int cap, cudaStream_t s);
int launch_iota(int32_t* cu, int n, cudaStream_t s);
int launch_advance_pos(int32_t* pos, const uint8_t* valid, int B, cudaStream_t s);
int launch_argmax_rows(const float* logits, int rows, int V, int32_t* out, cudaStream_t s);
int launch_embed(const void* embed, const int32_t* ids, int T, int d, int vocab, void* out,
                 cudaStream_t s);

}  // namespace qtale
