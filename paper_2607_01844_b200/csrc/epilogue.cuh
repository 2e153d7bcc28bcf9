// Epilogues of the grouped expert GEMMs.  Each function receives the fp32 accumulators of C
// consecutive columns of ONE output row and finishes the layer's elementwise math there, so no
// fp32 intermediate ever reaches HBM:
//   SWIGLU     H = silu(G) * U from the two accumulators (+ bf16 stash of G and U)
//   GATE       Yp = gate(row) * acc
//   DH         SwiGLU backward from dHu = dY W_down^T: dG, dU, gate*H and the partial <dHu, H>
//   BF16/F32   plain stores (dXp; weight gradients)
#pragma once
#include "common.cuh"

namespace mop {

enum : int { EPI_SWIGLU = 0, EPI_GATE = 1, EPI_DH = 2, EPI_BF16 = 3, EPI_F32 = 4 };

struct EpiArgs {
    bf16* out0;            // SWIGLU: H      GATE: Yp     DH: dG      BF16: out
    bf16* out1;            // SWIGLU: G_save (or null)    DH: dU
    bf16* out2;            // SWIGLU: U_save (or null)    DH: gate*H
    const bf16* in0;       // DH: G_save
    const bf16* in1;       // DH: U_save
    const bf16* in2;       // DH: H
    const float* gate;     // [T*k] indexed by assignment
    const int32_t* row_src;
    float* part;           // DH: partial dot products [n_tiles][M_total]
    float* outf;           // F32: output base (per expert: + e * Mfix * N)
    int ldo;               // row pitch (elements) of the bf16 / fp32 outputs and of in0..in2
    int M_total;
    int accumulate;        // F32: add into the output
};

template <int C>
__device__ __forceinline__ void store_bf16_run(bf16* dst, const float (&v)[C]) {
    static_assert(C % 4 == 0, "runs are multiples of 4 columns");
    if constexpr (C % 8 == 0) {
#pragma unroll
        for (int c = 0; c < C; c += 8) {
            uint4 o;
            o.x = pack_bf16x2(v[c], v[c + 1]);
            o.y = pack_bf16x2(v[c + 2], v[c + 3]);
            o.z = pack_bf16x2(v[c + 4], v[c + 5]);
            o.w = pack_bf16x2(v[c + 6], v[c + 7]);
            *reinterpret_cast<uint4*>(dst + c) = o;
        }
    } else {
#pragma unroll
        for (int c = 0; c < C; c += 4) {
            uint2 o;
            o.x = pack_bf16x2(v[c], v[c + 1]);
            o.y = pack_bf16x2(v[c + 2], v[c + 3]);
            *reinterpret_cast<uint2*>(dst + c) = o;
        }
    }
}

template <int C>
__device__ __forceinline__ void load_bf16_run(const bf16* src, float (&v)[C]) {
    if constexpr (C % 8 == 0) {
#pragma unroll
        for (int c = 0; c < C; c += 8) {
            const uint4 r = *reinterpret_cast<const uint4*>(src + c);
            v[c] = bf16_lo(r.x); v[c + 1] = bf16_hi(r.x); v[c + 2] = bf16_lo(r.y); v[c + 3] = bf16_hi(r.y);
            v[c + 4] = bf16_lo(r.z); v[c + 5] = bf16_hi(r.z); v[c + 6] = bf16_lo(r.w); v[c + 7] = bf16_hi(r.w);
        }
    } else {
#pragma unroll
        for (int c = 0; c < C; c += 4) {
            const uint2 r = *reinterpret_cast<const uint2*>(src + c);
            v[c] = bf16_lo(r.x); v[c + 1] = bf16_hi(r.x); v[c + 2] = bf16_lo(r.y); v[c + 3] = bf16_hi(r.y);
        }
    }
}

// SwiGLU forward on one run.  g, u: fp32 accumulators.
template <int C>
__device__ __forceinline__ void epi_swiglu(const EpiArgs& ep, int row, int col, const float (&g)[C],
                                           const float (&u)[C]) {
    float h[C];
#pragma unroll
    for (int c = 0; c < C; ++c) h[c] = g[c] * sigmoidf_fast(g[c]) * u[c];
    const size_t o = (size_t)row * ep.ldo + col;
    store_bf16_run<C>(ep.out0 + o, h);
    if (ep.out1) {
        store_bf16_run<C>(ep.out1 + o, g);
        store_bf16_run<C>(ep.out2 + o, u);
    }
}

template <int C>
__device__ __forceinline__ void epi_gate(const EpiArgs& ep, int row, int col, float gate, const float (&acc)[C]) {
    float y[C];
#pragma unroll
    for (int c = 0; c < C; ++c) y[c] = gate * acc[c];
    store_bf16_run<C>(ep.out0 + (size_t)row * ep.ldo + col, y);
}

// SwiGLU backward on one run; returns this run's share of <dHu, H>.
template <int C>
__device__ __forceinline__ float epi_dh(const EpiArgs& ep, int row, int col, float gate, const float (&dhu)[C]) {
    const size_t o = (size_t)row * ep.ldo + col;
    float G[C], U[C], H[C], dG[C], dU[C], gH[C];
    load_bf16_run<C>(ep.in0 + o, G);
    load_bf16_run<C>(ep.in1 + o, U);
    load_bf16_run<C>(ep.in2 + o, H);
    float dot = 0.0f;
#pragma unroll
    for (int c = 0; c < C; ++c) {
        dot = fmaf(dhu[c], H[c], dot);
        const float dh = gate * dhu[c];
        const float s = sigmoidf_fast(G[c]);
        dG[c] = dh * U[c] * s * (1.0f + G[c] * (1.0f - s));
        dU[c] = dh * (G[c] * s);
        gH[c] = gate * H[c];
    }
    store_bf16_run<C>(ep.out0 + o, dG);
    store_bf16_run<C>(ep.out1 + o, dU);
    store_bf16_run<C>(ep.out2 + o, gH);
    return dot;
}

template <int C>
__device__ __forceinline__ void epi_f32(float* dst, const float (&acc)[C], int accumulate) {
#pragma unroll
    for (int c = 0; c < C; c += 4) {
        float4 v = make_float4(acc[c], acc[c + 1], acc[c + 2], acc[c + 3]);
        if (accumulate) {
            const float4 old = *reinterpret_cast<const float4*>(dst + c);
            v.x += old.x; v.y += old.y; v.z += old.z; v.w += old.w;
        }
        *reinterpret_cast<float4*>(dst + c) = v;
    }
}

}  // namespace mop
