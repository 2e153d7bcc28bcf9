// Scalar (CUDA-core) grouped GEMM: the generic path for shapes the tensor-core kernels do not
// take (d or f not a multiple of 64) and the on-device cross-check used while bringing those
// kernels up.  bf16 operands, fp32 accumulation, any operand strides, ragged M (rows of an
// expert) or ragged K (weight gradients), same epilogues as the tensor-core path.
#pragma once
#include "epilogue.cuh"

namespace mop {

struct ScalarGemmArgs {
    const bf16* A[2];
    const bf16* B[2];
    long sAm, sAk;        // A(m,k) element strides
    long sBk, sBn, sBe;   // B(k,n) element strides and per-expert stride
    const int32_t* offsets;
    int ragged_k;         // 0: rows m are the expert's rows; 1: k runs over the expert's rows
    int Mfix, N, Kfix;
    int npairs;           // 1 or 2 operand pairs
    int dual_acc;         // pair 1 feeds a second accumulator (SwiGLU) instead of the first
    int epi;
    EpiArgs ep;
};

constexpr int SG_BM = 64, SG_BN = 64, SG_BK = 16;

__global__ void __launch_bounds__(256) scalar_grouped_gemm_kernel(const ScalarGemmArgs g) {
    __shared__ float As[SG_BK][SG_BM + 4];
    __shared__ float Bs[SG_BK][SG_BN + 4];
    const int e = blockIdx.y;
    const int n0 = blockIdx.x * SG_BN;
    const int off = g.offsets[e], rows = g.offsets[e + 1] - off;
    const int M = g.ragged_k ? g.Mfix : rows;
    const int K = g.ragged_k ? rows : g.Kfix;
    const int tid = threadIdx.x, ty = tid / 16, tx = tid % 16;

    for (int m0 = 0; m0 < M; m0 += SG_BM) {
        float acc[4][4], acc2[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = acc2[i][j] = 0.0f;
        for (int pair = 0; pair < g.npairs; ++pair) {
            const bf16* A = g.A[pair];
            const bf16* B = g.B[pair];
            for (int k0 = 0; k0 < K; k0 += SG_BK) {
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const int lin = r * 256 + tid;
                    int m, k;
                    if (g.sAk == 1) { k = lin % SG_BK; m = lin / SG_BK; } else { m = lin % SG_BM; k = lin / SG_BM; }
                    float v = 0.0f;
                    if (m0 + m < M && k0 + k < K) {
                        const size_t idx = g.ragged_k ? (size_t)(off + k0 + k) * g.sAk + (size_t)(m0 + m) * g.sAm
                                                      : (size_t)(off + m0 + m) * g.sAm + (size_t)(k0 + k) * g.sAk;
                        v = __bfloat162float(A[idx]);
                    }
                    As[k][m] = v;
                }
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const int lin = r * 256 + tid;
                    int n, k;
                    if (g.sBk == 1) { k = lin % SG_BK; n = lin / SG_BK; } else { n = lin % SG_BN; k = lin / SG_BN; }
                    float v = 0.0f;
                    if (n0 + n < g.N && k0 + k < K) {
                        const size_t idx = g.ragged_k ? (size_t)(off + k0 + k) * g.sBk + (size_t)(n0 + n) * g.sBn
                                                      : (size_t)e * g.sBe + (size_t)(k0 + k) * g.sBk +
                                                            (size_t)(n0 + n) * g.sBn;
                        v = __bfloat162float(B[idx]);
                    }
                    Bs[k][n] = v;
                }
                __syncthreads();
                const bool second = g.dual_acc && pair == 1;
#pragma unroll
                for (int kk = 0; kk < SG_BK; ++kk) {
                    const float4 av = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
                    const float4 bv = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
                    const float a[4] = {av.x, av.y, av.z, av.w};
                    const float b[4] = {bv.x, bv.y, bv.z, bv.w};
                    if (second) {
#pragma unroll
                        for (int i = 0; i < 4; ++i)
#pragma unroll
                            for (int j = 0; j < 4; ++j) acc2[i][j] = fmaf(a[i], b[j], acc2[i][j]);
                    } else {
#pragma unroll
                        for (int i = 0; i < 4; ++i)
#pragma unroll
                            for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
                    }
                }
                __syncthreads();
            }
        }
        // epilogue: thread owns rows m0+ty*4+i, columns n0+tx*4 .. +3 (N is a multiple of 8)
        const int col = n0 + tx * 4;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int m = m0 + ty * 4 + i;
            const bool ok = (m < M) && (col < g.N);
            float dot = 0.0f;
            if (ok) {
                if (g.epi == EPI_F32) {
                    epi_f32<4>(g.ep.outf + (size_t)e * g.Mfix * g.N + (size_t)m * g.N + col, acc[i], g.ep.accumulate);
                } else {
                    const int row = off + m;
                    if (g.epi == EPI_SWIGLU) epi_swiglu<4>(g.ep, row, col, acc[i], acc2[i]);
                    else if (g.epi == EPI_BF16) store_bf16_run<4>(g.ep.out0 + (size_t)row * g.ep.ldo + col, acc[i]);
                    else {
                        const float gate = g.ep.gate[g.ep.row_src[row]];
                        if (g.epi == EPI_GATE) epi_gate<4>(g.ep, row, col, gate, acc[i]);
                        else dot = epi_dh<4>(g.ep, row, col, gate, acc[i]);
                    }
                }
            }
            if (g.epi == EPI_DH) {
                // the 16 threads tx = 0..15 of one row are 16 consecutive lanes
                dot += __shfl_xor_sync(0xffffffffu, dot, 8);
                dot += __shfl_xor_sync(0xffffffffu, dot, 4);
                dot += __shfl_xor_sync(0xffffffffu, dot, 2);
                dot += __shfl_xor_sync(0xffffffffu, dot, 1);
                if (tx == 0 && m < M) g.ep.part[(size_t)blockIdx.x * g.ep.M_total + off + m] = dot;
            }
        }
    }
    // weight gradients of an expert without rows: the loop above ran with K = 0 and stored zeros
}

}  // namespace mop
