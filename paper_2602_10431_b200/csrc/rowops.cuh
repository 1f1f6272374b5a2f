// Launchers of the bandwidth-bound row kernels (internal to libqtale).
#pragma once
#include "common.cuh"

namespace qtale {

int launch_compact(const void* x, const int32_t* idx, const int32_t* n_exec, int cap, int d,
                   const float* gamma, float eps, int act, void* xc, void* hn, cudaStream_t s);
int launch_scatter_add(void* x, const void* xc, const float* f, const int32_t* idx,
                       const int32_t* n_exec, int cap, int d, cudaStream_t s);
// RMSNorm of fp32 rows into bf16; n_rows may be NULL (all `cap` rows).
int launch_rmsnorm_f32(const float* u, const int32_t* n_rows, int cap, int d, const float* gamma,
                       float eps, int act, void* out, cudaStream_t s);
// cs: float2 [cap, hd/2] = (cos, sin) of pos[i] * base^(-2j/hd)
int launch_rope_table(const int32_t* pos, const int32_t* n_exec, int cap, int hd, float base,
                      float* cs, cudaStream_t s);
int launch_rope(void* qkv, const int32_t* n_exec, int cap, int ld, int n_rot, int hd,
                const float* cs, int act, cudaStream_t s);
int launch_swiglu(const void* gu, const int32_t* n_exec, int cap, int F, void* act, int act_dtype,
                  cudaStream_t s);
int launch_kv_append(const void* qkv, const int32_t* n_exec, int cap_rows, int ld, int q_dim,
                     int kv_dim, const int32_t* cu_exec, int B, void* cache_k, void* cache_v,
                     int32_t* kv_len, int cap, cudaStream_t s);
// zeroes rows [*n_exec, *n_exec + tile) (below cap) of a 16-bit [cap, ld] tensor
int launch_zero_tail_rows(void* buf, const int32_t* n_exec, int cap, int ld, int tile,
                          cudaStream_t s);
int launch_embed(const void* embed, const int32_t* ids, int T, int d, int vocab, void* out,
                 cudaStream_t s);

}  // namespace qtale
