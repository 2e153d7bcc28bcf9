// Router kernels: exact fp32 scoring and warp-per-token top-k with gate renormalisation.
// Section 2.1 of the paper ("a lightweight router that sends each token to its top-k experts").
#pragma once
#include "common.cuh"

namespace mop {

// ---------------------------------------------------------------------------------------------
// Scoring.  z[t,e] = sum_i x[t,i] * W_r[i,e] as ONE chain of fused multiply-adds per (t,e), i
// ascending, each step rounded once to fp32.  The chain order is part of the routing contract
// (it makes top-k indices reproducible bit for bit), so there is no split over i and no tensor
// core here; parallelism comes from the T*E independent chains.  Tile: 64 tokens x 64 experts
// per 256-thread block, 4x4 chains per thread, operands staged through shared memory in slabs
// of 32 along i.
// ---------------------------------------------------------------------------------------------
constexpr int SC_TT = 64, SC_TE = 64, SC_TK = 32;

__global__ void __launch_bounds__(256) route_score_kernel(const bf16* __restrict__ x, const float* __restrict__ W_r,
                                                          float* __restrict__ z, int T, int d, int E) {
    __shared__ __align__(16) float xs[SC_TK][SC_TT + 4];
    __shared__ __align__(16) float ws[SC_TK][SC_TE + 4];
    const int t0 = blockIdx.x * SC_TT, e0 = blockIdx.y * SC_TE;
    const int tid = threadIdx.x;
    const int tt = (tid / 16) * 4, te = (tid % 16) * 4;
    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.0f;

    for (int i0 = 0; i0 < d; i0 += SC_TK) {
        // x slab: 64 tokens x 32 i  (each thread 8 elements: one token, 8 consecutive i)
        {
            const int tok = tid / 4, ii = (tid % 4) * 8;
            const int t = t0 + tok;
            float v[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) v[q] = 0.0f;
            if (t < T) {
                if (i0 + ii + 8 <= d) {
                    const uint4 raw = *reinterpret_cast<const uint4*>(x + (size_t)t * d + i0 + ii);
                    v[0] = bf16_lo(raw.x); v[1] = bf16_hi(raw.x); v[2] = bf16_lo(raw.y); v[3] = bf16_hi(raw.y);
                    v[4] = bf16_lo(raw.z); v[5] = bf16_hi(raw.z); v[6] = bf16_lo(raw.w); v[7] = bf16_hi(raw.w);
                } else {
                    for (int q = 0; q < 8; ++q)
                        if (i0 + ii + q < d) v[q] = __bfloat162float(x[(size_t)t * d + i0 + ii + q]);
                }
            }
#pragma unroll
            for (int q = 0; q < 8; ++q) xs[ii + q][tok] = v[q];
        }
        // W_r slab: 32 i x 64 experts
#pragma unroll
        for (int r = 0; r < (SC_TK * SC_TE) / 256; ++r) {
            const int lin = r * 256 + tid;
            const int ii = lin / SC_TE, ee = lin % SC_TE;
            float w = 0.0f;
            if (i0 + ii < d && e0 + ee < E) w = W_r[(size_t)(i0 + ii) * E + e0 + ee];
            ws[ii][ee] = w;
        }
        __syncthreads();
        // Past-the-end i (d not a multiple of 32) contributes fma(0, 0, acc) = acc: exact.
#pragma unroll 8
        for (int kk = 0; kk < SC_TK; ++kk) {
            const float4 xv = *reinterpret_cast<const float4*>(&xs[kk][tt]);
            const float4 wv = *reinterpret_cast<const float4*>(&ws[kk][te]);
            const float xa[4] = {xv.x, xv.y, xv.z, xv.w};
            const float wa[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) acc[a][b] = __fmaf_rn(xa[a], wa[b], acc[a][b]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int t = t0 + tt + a;
        if (t >= T) continue;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int e = e0 + te + b;
            if (e < E) z[(size_t)t * E + e] = acc[a][b];
        }
    }
}

// Sigmoid of the routing contract: a fixed sequence of fp32 operations, each rounded once
// (explicit-rounding intrinsics so that no contraction or fast path can change a step).
__device__ __forceinline__ float sigmoid_contract(float zv) {
    float u = -zv;
    u = fminf(fmaxf(u, -80.0f), 80.0f);
    const float n = rintf(__fmul_rn(u, 1.44269504088896341f));
    float r = __fmaf_rn(n, -0.693145751953125f, u);
    r = __fmaf_rn(n, -1.42860682030941723e-6f, r);
    float p = __fdiv_rn(1.0f, 720.0f);
    p = __fmaf_rn(p, r, __fdiv_rn(1.0f, 120.0f));
    p = __fmaf_rn(p, r, __fdiv_rn(1.0f, 24.0f));
    p = __fmaf_rn(p, r, __fdiv_rn(1.0f, 6.0f));
    p = __fmaf_rn(p, r, 0.5f);
    p = __fmaf_rn(p, r, 1.0f);
    p = __fmaf_rn(p, r, 1.0f);
    const float scale = __int_as_float(((int)n + 127) << 23);
    const float e = __fmul_rn(p, scale);
    return __fdiv_rn(1.0f, __fadd_rn(1.0f, e));
}

// ---------------------------------------------------------------------------------------------
// Selection: one warp per token.  Keys live in shared memory (E floats per warp); each lane owns
// the experts e = lane, lane+32, ... and a bitmask of those already taken.  k rounds of
// (lane-local best) -> (warp argmax by shuffle), comparison "key greater, or equal and id lower".
// ---------------------------------------------------------------------------------------------
constexpr int SEL_WARPS = 4;
constexpr int SEL_MAX_E = 1024;  // 32 lanes x 32 mask bits

__global__ void __launch_bounds__(SEL_WARPS * 32) route_select_kernel(const float* __restrict__ z,
                                                                      const float* __restrict__ bias,
                                                                      int32_t* __restrict__ idx,
                                                                      float* __restrict__ gate, int T, int E, int k,
                                                                      int score_fn, int bias_mode) {
    extern __shared__ float sel_smem[];
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    float* key = sel_smem + (size_t)warp * 2 * E;  // keys
    float* zg = key + E;                            // logit that the gate is computed from
    const int t = blockIdx.x * SEL_WARPS + warp;
    if (t >= T) return;
    for (int e = lane; e < E; e += 32) {
        float zz = z[(size_t)t * E + e];
        if (bias_mode == 2) zz = __fadd_rn(zz, bias[e]);
        float kk = zz;
        if (score_fn == 1 && bias_mode == 1) kk = __fadd_rn(sigmoid_contract(zz), bias[e]);
        key[e] = kk;
        zg[e] = zz;
    }
    __syncwarp();
    uint32_t taken = 0;
    float my_z = 0.0f;     // lane j keeps the gate logit of the j-th pick (k <= 32) ...
    int my_e = 0;
    for (int j = 0; j < k; ++j) {
        int best = -1;
        float bk = 0.0f;
        for (int q = 0, e = lane; e < E; ++q, e += 32) {
            if ((taken >> q) & 1u) continue;
            const float v = key[e];
            if (best < 0 || v > bk) { best = e; bk = v; }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float ok = __shfl_xor_sync(0xffffffffu, bk, off);
            const int oe = __shfl_xor_sync(0xffffffffu, best, off);
            const bool take = (oe >= 0) && (best < 0 || ok > bk || (ok == bk && oe < best));
            if (take) { bk = ok; best = oe; }
        }
        // every lane now holds the same winner (the comparison is a total order on (key, id))
        if ((best & 31) == lane) taken |= 1u << (best >> 5);
        if ((j & 31) == lane) {
            // picks beyond 32 are handled in a second pass below (k <= 32 in every workload)
            my_e = best;
            my_z = zg[best];
        }
        if (k > 32 && lane == 0) idx[(size_t)t * k + j] = best;
    }
    if (k <= 32) {
        const bool act = lane < k;
        float s;
        if (score_fn == 0) {
            float m = act ? my_z : -INFINITY;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
            s = act ? expf(my_z - m) : 0.0f;
        } else {
            s = act ? sigmoidf_acc(my_z) : 0.0f;
        }
        float sum = s;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
        if (act) {
            idx[(size_t)t * k + lane] = my_e;
            gate[(size_t)t * k + lane] = s / sum;
        }
    } else {
        // generic tail (k > 32): lane 0 recomputes the gates from the stored indices
        __syncwarp();
        if (lane == 0) {
            float m = -INFINITY, sum = 0.0f;
            for (int j = 0; j < k; ++j) m = fmaxf(m, zg[idx[(size_t)t * k + j]]);
            for (int j = 0; j < k; ++j) {
                const float zz = zg[idx[(size_t)t * k + j]];
                sum += (score_fn == 0) ? expf(zz - m) : sigmoidf_acc(zz);
            }
            for (int j = 0; j < k; ++j) {
                const float zz = zg[idx[(size_t)t * k + j]];
                gate[(size_t)t * k + j] = ((score_fn == 0) ? expf(zz - m) : sigmoidf_acc(zz)) / sum;
            }
        }
    }
}

}  // namespace mop
