// Launchers of the attention kernels (internal to libqtale).
#pragma once
#include "common.cuh"

namespace qtale {

// Causal attention among the executed tokens of each sequence.
// qkv: 16-bit (act) [T_e, ld] = [q heads | k heads | v heads] (q, k already rotated);
// cu_exec: int32 [B+1] device; out: same format [T_e, ldo].
int launch_attn_prefill(const void* qkv, int ld, int H, int Hkv, int hd, int act,
                        const int32_t* cu_exec, int B, int T_cap, void* out, int ldo,
                        cudaStream_t s);

// One query per executed sequence i < *n_exec (sequence idx[i]) against the
// first kv_len[idx[i]] cache entries of that sequence (the new token included).
int launch_attn_decode(const void* qkv, int ld, int H, int Hkv, int hd, int act, const int32_t* idx,
                       const int32_t* n_exec, int B_cap, const void* cache_k, const void* cache_v,
                       const int32_t* kv_len, int cap, void* out, int ldo, cudaStream_t s);

}  // namespace qtale
