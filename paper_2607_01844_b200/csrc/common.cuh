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
// Sigmoid of the SwiGLU epilogues: fast exponential and division (about 2 ulp), far inside the bf16
// rounding of every value it feeds; all GEMM schedules share it, so they stay bit-identical.  (The
// router's gates keep the accurate form above.)
__device__ __forceinline__ float sigmoidf_fast(float v) { return __fdividef(1.0f, 1.0f + __expf(-v)); }

static inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Optional per-kernel timing: a pool of CUDA event pairs recorded around every launch on the
// launching stream, aggregated by kernel name when read.  Off by default (no events, no cost).
struct Profiler {
    static constexpr int MAX_REC = 8192;
    bool on = false;
    cudaEvent_t* ev = nullptr;          // 2 * MAX_REC events once enabled
    const char* names[MAX_REC];
    int n = 0;
    void begin(const char* name, cudaStream_t st) {
        if (on && n < MAX_REC) { names[n] = name; cudaEventRecord(ev[2 * n], st); }
    }
    void end(cudaStream_t st) {
        if (on && n < MAX_REC) { cudaEventRecord(ev[2 * n + 1], st); ++n; }
    }
};

}  // namespace mop
