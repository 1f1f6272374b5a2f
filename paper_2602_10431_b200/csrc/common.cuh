// Shared device / host helpers of libqtale (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "qtale.h"

#define QTALE_SM_COUNT_FALLBACK 148

namespace qtale {

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int sm_count();                    // SMs of the current device (cached per device)
int launch_status(cudaError_t e);  // maps a CUDA error to QTALE_ERR_CUDA

// Device address of the current device's status word (first device-side error
// since the last qtale_device_status call).  Kernels receive it as an argument.
int* device_status_ptr();

// ---------------------------------------------------------------------------
// device side
// ---------------------------------------------------------------------------

__device__ __forceinline__ void report_device_error(int* status, int code) {
  if (status) atomicCAS(status, 0, code);
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t b16) {
  return __uint_as_float(b16 << 16);
}
__device__ __forceinline__ float bf16_lo(uint32_t packed) { return __uint_as_float(packed << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t packed) {
  return __uint_as_float(packed & 0xFFFF0000u);
}
// two floats -> packed bf16x2 (lo in bits 0..15), round to nearest even
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// 16-bit activation formats of the tensors the layer keeps between its kernels.
// ACT = QTALE_ACT_BF16 (0) or QTALE_ACT_F16 (1).  Both are read as two values per
// 32-bit word (element 0 in the low half) and written with one rounding.
template <int ACT>
struct Act16;
template <>
struct Act16<0> {
  static __device__ __forceinline__ float lo(uint32_t p) { return bf16_lo(p); }
  static __device__ __forceinline__ float hi(uint32_t p) { return bf16_hi(p); }
  static __device__ __forceinline__ uint32_t pack(float l, float h) { return pack_bf16x2(l, h); }
  static __device__ __forceinline__ unsigned short one(float v) {
    return __bfloat16_as_ushort(__float2bfloat16_rn(v));
  }
};
template <>
struct Act16<1> {
  static __device__ __forceinline__ float lo(uint32_t p) {
    return __half2float(__ushort_as_half((unsigned short)(p & 0xFFFFu)));
  }
  static __device__ __forceinline__ float hi(uint32_t p) {
    return __half2float(__ushort_as_half((unsigned short)(p >> 16)));
  }
  static __device__ __forceinline__ uint32_t pack(float l, float h) {
    uint32_t r;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(h), "f"(l));
    return r;
  }
  static __device__ __forceinline__ unsigned short one(float v) {
    return __half_as_ushort(__float2half_rn(v));
  }
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// barrier among `threads` threads (a multiple of 32) of the CTA; id 1..15 (0 is __syncthreads)
__device__ __forceinline__ void named_barrier(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// 16-byte global accesses
__device__ __forceinline__ uint4 ld_nc_16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
__device__ __forceinline__ void st_16(void* p, uint4 v) {
  asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
               "r"(v.w)
               : "memory");
}

}  // namespace qtale
