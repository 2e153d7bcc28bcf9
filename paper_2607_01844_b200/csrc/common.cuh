// Shared device helpers for the routed-expert kernels (sm_100a only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace mop {

typedef __nv_bfloat16 bf16;

// Codes written to the context's device status word by bounded waits.
enum : int { STATUS_OK = 0, STATUS_WAIT_FULL = 1, STATUS_WAIT_EMPTY = 2, STATUS_WAIT_TMEM_FULL = 3,
             STATUS_WAIT_TMEM_EMPTY = 4, STATUS_BAD_TILE = 5 };

__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

// two fp32 -> packed bf16x2 (round to nearest even), lo in the low half
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&p);
}

__device__ __forceinline__ float round_bf16(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }

__device__ __forceinline__ float sigmoidf_acc(float v) { return 1.0f / (1.0f + expf(-v)); }

static inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

}  // namespace mop
