// Launcher of the fused router / selection / compaction kernel (internal to libqtale).
#pragma once
#include "common.cuh"

namespace qtale {

// Arguments as qtale_router_select.  In top-k mode with ratio >= 0 the count is taken on the
// device as floor(ratio * valid tokens + 0.5) (k is ignored): padding does not count towards
// the execution ratio.
int router_select_launch(const void* x, int T, int d, const float* w_router, float bias,
                         const float* scores_override, const uint8_t* valid,
                         const int32_t* cu_seqlens, int B, const int32_t* pos0, int mode,
                         float theta, int k, double ratio, float* scores_out, int32_t* idx_out,
                         int32_t* n_exec_out, int32_t* cu_exec_out, int32_t* pos_out, void* ws,
                         size_t ws_bytes, cudaStream_t s, int32_t* n_exec_copy = nullptr);

// MLP router scores (arguments as qtale_router_mlp_scores, already validated)
int router_mlp_launch(const void* x, int T, int d, const void* w1, const float* b1, const float* w2,
                      int h, float b2_execute, float b2_bypass, float* scores, cudaStream_t s);

}  // namespace qtale
