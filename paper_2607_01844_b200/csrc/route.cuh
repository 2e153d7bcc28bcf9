// Router kernels: exact fp32 scoring and warp-per-token top-k with gate renormalisation
// (the router of the MoE block, Section 2.1 of the paper).
#pragma once
#include "common.cuh"

namespace mop {

// ---------------------------------------------------------------------------------------------
// Scoring.  z[t,e] = sum_i x[t,i] * W_r[i,e] as ONE chain of fused multiply-adds per (t,e), i
// ascending, each step rounded once to fp32.  The chain order is part of the routing contract
// (it makes top-k indices reproducible bit for bit), so there is no split over i and no tensor
// core here; parallelism comes from the T*E independent chains and the kernel is bound by the
// fp32 pipes.  Each thread owns RT tokens x RE experts (RT*RE chains) and advances two chains
// per instruction with the packed fma.rn.f32x2 of sm_100 (two independent IEEE fused
// multiply-adds: the rounding of each chain is unchanged).  A 128-thread CTA covers
// (16 RT) tokens x (8 RE) experts; operands are staged through shared memory in slabs of 16 or 32
// along i, double-buffered, the next slab prefetched into registers while the current one is
// multiplied.  <8,8> needs 4 shared loads per 64 FMAs; smaller tiles trade that for more CTAs
// when T*E is small.  Both slabs are laid out so that every shared access of a warp is free of
// bank conflicts (interleaved expert columns, XOR-swizzled token columns).
// ---------------------------------------------------------------------------------------------
constexpr int SC_THREADS = 128;

__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ void fma_f32x2(unsigned long long& acc, unsigned long long a, unsigned long long b) {
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(a), "l"(b));
}

template <int RT, int RE, int SC_TK>
__global__ void __launch_bounds__(SC_THREADS, 4) route_score_kernel(const bf16* __restrict__ x,
                                                                 const float* __restrict__ W_r,
                                                                 float* __restrict__ z, int T, int d, int E) {
    constexpr int TT = 16 * RT, TE = 8 * RE;          // CTA tile
    constexpr int LDX = TT + 4, LDW = TE + 4;
    constexpr int XV = TT * SC_TK / 8 / SC_THREADS;   // 16-byte x vectors fetched per thread per slab
    constexpr int WV = TE * SC_TK / 4 / SC_THREADS;   // float4 W vectors per thread per slab
    static_assert(RT % 2 == 0 && RE % 4 == 0 && XV >= 1 && WV >= 1, "tile shape");
    __shared__ __align__(16) float xs[2][SC_TK][LDX];
    __shared__ __align__(16) float ws[2][SC_TK][LDW];
    const int t0 = blockIdx.x * TT, e0 = blockIdx.y * TE;
    const int tid = threadIdx.x;
    // Expert columns of a thread: groups of 4 at te + 32 b, so that the 8 threads that differ in
    // tid % 8 read 32 consecutive floats (one conflict-free wavefront) per group.
    const int tt = (tid / 8) * RT, te = (tid % 8) * 4;
    constexpr int EG = (RE > 4) ? 32 : 4;             // column pitch between a thread's groups of 4
    // Token columns of the x slab are XOR-swizzled by the 8-row chunk of i they belong to: the
    // threads of a warp that stash different chunks of the same tokens then hit different banks.
    constexpr int CH = SC_TK / 8, SWZ = 32 / CH;
    static_assert(TT >= 32 && (SWZ % 4) == 0, "swizzle keeps float4 groups intact and stays inside the tile");
    const bool w_vec = (E % 4 == 0);

    unsigned long long acc[RT / 2][RE];   // acc[a][b] = chains of tokens (2a, 2a+1) for expert b
#pragma unroll
    for (int a = 0; a < RT / 2; ++a)
#pragma unroll
        for (int b = 0; b < RE; ++b) acc[a][b] = 0ull;

    uint4 xr[XV];
    float4 wr[WV];
    // x slab: TT tokens x SC_TK i, vector v of a thread = token lin / (SC_TK/8), i offset (lin % (SC_TK/8)) * 8
    auto fetch = [&](int i0) {
#pragma unroll
        for (int v = 0; v < XV; ++v) {
            const int lin = v * SC_THREADS + tid;
            const int t = t0 + lin / (SC_TK / 8), i = i0 + (lin % (SC_TK / 8)) * 8;
            xr[v] = (t < T && i < d) ? *reinterpret_cast<const uint4*>(x + (size_t)t * d + i) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int v = 0; v < WV; ++v) {
            const int lin = v * SC_THREADS + tid;
            const int i = i0 + lin / (TE / 4), e = e0 + (lin % (TE / 4)) * 4;
            float4 q = make_float4(0.f, 0.f, 0.f, 0.f);
            if (i < d) {
                const float* src = W_r + (size_t)i * E + e;
                if (w_vec && e + 3 < E) q = *reinterpret_cast<const float4*>(src);
                else {
                    if (e < E) q.x = src[0];
                    if (e + 1 < E) q.y = src[1];
                    if (e + 2 < E) q.z = src[2];
                    if (e + 3 < E) q.w = src[3];
                }
            }
            wr[v] = q;
        }
    };
    auto stash = [&](int buf) {
#pragma unroll
        for (int v = 0; v < XV; ++v) {
            const int lin = v * SC_THREADS + tid;
            const int tok = lin / (SC_TK / 8), ii = (lin % (SC_TK / 8)) * 8;
            const uint32_t w4[4] = {xr[v].x, xr[v].y, xr[v].z, xr[v].w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                xs[buf][ii + 2 * q][tok ^ ((ii / 8) * SWZ)] = bf16_lo(w4[q]);
                xs[buf][ii + 2 * q + 1][tok ^ ((ii / 8) * SWZ)] = bf16_hi(w4[q]);
            }
        }
#pragma unroll
        for (int v = 0; v < WV; ++v) {
            const int lin = v * SC_THREADS + tid;
            *reinterpret_cast<float4*>(&ws[buf][lin / (TE / 4)][(lin % (TE / 4)) * 4]) = wr[v];
        }
    };

    fetch(0);
    stash(0);
    __syncthreads();
    int buf = 0;
    for (int i0 = 0; i0 < d; i0 += SC_TK) {
        const bool more = i0 + SC_TK < d;
        if (more) fetch(i0 + SC_TK);
        // Past-the-end i (d not a multiple of the slab) multiplies zeros: fma(0, 0, acc) = acc, exact.
#pragma unroll
        for (int kk = 0; kk < SC_TK; ++kk) {
            unsigned long long xp[RT / 2], wp[RE];
#pragma unroll
            for (int a = 0; a < RT / 4; ++a) {
                const float4 v = *reinterpret_cast<const float4*>(&xs[buf][kk][(tt + 4 * a) ^ ((kk / 8) * SWZ)]);
                xp[2 * a] = pack_f32x2(v.x, v.y);
                xp[2 * a + 1] = pack_f32x2(v.z, v.w);
            }
            if constexpr (RT % 4 == 2) {
                const float2 v = *reinterpret_cast<const float2*>(&xs[buf][kk][(tt + RT - 2) ^ ((kk / 8) * SWZ)]);
                xp[RT / 2 - 1] = pack_f32x2(v.x, v.y);
            }
#pragma unroll
            for (int b = 0; b < RE / 4; ++b) {
                const float4 v = *reinterpret_cast<const float4*>(&ws[buf][kk][te + EG * b]);
                wp[4 * b] = pack_f32x2(v.x, v.x);
                wp[4 * b + 1] = pack_f32x2(v.y, v.y);
                wp[4 * b + 2] = pack_f32x2(v.z, v.z);
                wp[4 * b + 3] = pack_f32x2(v.w, v.w);
            }
#pragma unroll
            for (int a = 0; a < RT / 2; ++a)
#pragma unroll
                for (int b = 0; b < RE; ++b) fma_f32x2(acc[a][b], xp[a], wp[b]);
        }
        if (more) stash(buf ^ 1);
        __syncthreads();
        buf ^= 1;
    }
#pragma unroll
    for (int a = 0; a < RT / 2; ++a) {
        float lo[RE], hi[RE];
#pragma unroll
        for (int b = 0; b < RE; ++b) unpack_f32x2(acc[a][b], lo[b], hi[b]);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int t = t0 + tt + 2 * a + h;
            if (t >= T) continue;
#pragma unroll
            for (int b = 0; b < RE; b += 4) {
                const float v0 = h ? hi[b] : lo[b], v1 = h ? hi[b + 1] : lo[b + 1];
                const float v2 = h ? hi[b + 2] : lo[b + 2], v3 = h ? hi[b + 3] : lo[b + 3];
                const int e = e0 + te + EG * (b / 4);
                float* dst = z + (size_t)t * E + e;
                if (w_vec && e + 3 < E) {
                    *reinterpret_cast<float4*>(dst) = make_float4(v0, v1, v2, v3);
                } else {
                    if (e < E) dst[0] = v0;
                    if (e + 1 < E) dst[1] = v1;
                    if (e + 2 < E) dst[2] = v2;
                    if (e + 3 < E) dst[3] = v3;
                }
            }
        }
    }
}

// Tile choice: the largest tile that still gives every SM a few CTAs.
template <int RT, int RE, int TK>
inline void launch_route_score(const bf16* x, const float* W_r, float* z, int T, int d, int E, cudaStream_t st) {
    dim3 grid(ceil_div(T, 16 * RT), ceil_div(E, 8 * RE));
    route_score_kernel<RT, RE, TK><<<grid, SC_THREADS, 0, st>>>(x, W_r, z, T, d, E);
}
inline void route_score(const bf16* x, const float* W_r, float* z, int T, int d, int E, int sm_count,
                        cudaStream_t st) {
    const long long big = (long long)ceil_div(T, 128) * ceil_div(E, 64);
    const long long mid = (long long)ceil_div(T, 64) * ceil_div(E, 32);
    if (big >= 2ll * sm_count) launch_route_score<8, 8, 16>(x, W_r, z, T, d, E, st);
    else if (2 * mid >= sm_count) launch_route_score<4, 4, 32>(x, W_r, z, T, d, E, st);
    else launch_route_score<2, 4, 32>(x, W_r, z, T, d, E, st);
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
    float my_z = 0.0f;     // lane j keeps the gate logit and the id of the j-th pick (k <= 32, checked on the host)
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
        if (j == lane) {
            my_e = best;
            my_z = zg[best];
        }
    }
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
}

// ---------------------------------------------------------------------------------------------
// Router backward (selection held fixed).  With g_j = s_j / sum_l s_l over a token's k selected
// experts (s = softmax over all E, whose common denominator cancels, or s = sigmoid):
//   softmax:  dz_j = g_j (dgate_j - sum_l g_l dgate_l)
//   sigmoid:  dz_j = (dgate_j - sum_l g_l dgate_l) / S * s_j (1 - s_j),   S = sum_l s_l
// dz is zero at every expert that was not selected.  Then dW_r = x^T dz, dX += dz W_r^T and, for a
// bias added before the score, dbias = column sums of dz.
// ---------------------------------------------------------------------------------------------

// One warp per token: lane j < k owns the j-th selected expert.  Writes dz per assignment and, in
// expert-contiguous row order (row = perm_row[assignment]), the copy that the dW_r kernel reads.
__global__ void __launch_bounds__(256) route_bwd_dz_kernel(const float* __restrict__ logits,
                                                           const float* __restrict__ bias,
                                                           const int32_t* __restrict__ idx,
                                                           const float* __restrict__ gate,
                                                           const float* __restrict__ dgate,
                                                           const int32_t* __restrict__ perm_row,
                                                           float* __restrict__ dz_sel, float* __restrict__ dz_row,
                                                           int T, int E, int k, int score_fn, int bias_mode) {
    const int lane = threadIdx.x % 32;
    const int t = blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
    if (t >= T) return;
    const bool act = lane < k;
    const size_t a = (size_t)t * k + lane;
    float g = 0.0f, dg = 0.0f, zz = 0.0f;
    if (act) {
        const int e = idx[a];
        g = gate[a];
        dg = dgate[a];
        zz = logits[(size_t)t * E + e];
        if (bias_mode == 2) zz += bias[e];
    }
    float dot = g * dg;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
    float dz;
    if (score_fn == 0) {
        dz = g * (dg - dot);
    } else {
        const float s = act ? sigmoidf_acc(zz) : 0.0f;
        float S = s;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) S += __shfl_xor_sync(0xffffffffu, S, off);
        dz = (dg - dot) / S * s * (1.0f - s);
    }
    if (act) {
        dz_sel[a] = dz;
        const int32_t p = perm_row[a];
        if (p >= 0) dz_row[p] = dz;
    }
}

// dW_r[i,e] = sum over the rows p of expert e (ascending) of Xp[p,i] * dz_row[p].  Block (i-chunk, e):
// 128 threads, eight columns i each (16-byte loads); Xp rows are read once, coalesced, two rows in
// flight per thread.  Deterministic (no atomics).
__global__ void __launch_bounds__(128) route_bwd_dwr_kernel(const bf16* __restrict__ Xp,
                                                            const float* __restrict__ dz_row,
                                                            const int32_t* __restrict__ offsets,
                                                            float* __restrict__ dW_r, float* __restrict__ dbias,
                                                            int d, int E) {
    const int e = blockIdx.y;
    const int i = (blockIdx.x * 128 + threadIdx.x) * 8;
    const int p0 = offsets[e], p1 = offsets[e + 1];
    if (i < d) {
        float a[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) a[q] = 0.0f;
        auto add = [&](const uint4& v, float w) {
            a[0] = fmaf(bf16_lo(v.x), w, a[0]); a[1] = fmaf(bf16_hi(v.x), w, a[1]);
            a[2] = fmaf(bf16_lo(v.y), w, a[2]); a[3] = fmaf(bf16_hi(v.y), w, a[3]);
            a[4] = fmaf(bf16_lo(v.z), w, a[4]); a[5] = fmaf(bf16_hi(v.z), w, a[5]);
            a[6] = fmaf(bf16_lo(v.w), w, a[6]); a[7] = fmaf(bf16_hi(v.w), w, a[7]);
        };
        int p = p0;
        for (; p + 1 < p1; p += 2) {
            const uint4 v0 = __ldcs(reinterpret_cast<const uint4*>(Xp + (size_t)p * d + i));
            const uint4 v1 = __ldcs(reinterpret_cast<const uint4*>(Xp + (size_t)(p + 1) * d + i));
            add(v0, dz_row[p]);
            add(v1, dz_row[p + 1]);
        }
        if (p < p1) add(__ldcs(reinterpret_cast<const uint4*>(Xp + (size_t)p * d + i)), dz_row[p]);
#pragma unroll
        for (int q = 0; q < 8; ++q) dW_r[(size_t)(i + q) * E + e] = a[q];
    }
    if (dbias && blockIdx.x == 0 && threadIdx.x == 0) {
        float sb = 0.0f;
        for (int p = p0; p < p1; ++p) sb += dz_row[p];
        dbias[e] = sb;
    }
}

// W_r^T [E,d] from W_r [d,E] (32 x 32 tiles through shared memory): gives the dX kernel contiguous rows.
__global__ void __launch_bounds__(256) transpose_f32_kernel(const float* __restrict__ in, float* __restrict__ out,
                                                            int rows, int cols) {
    __shared__ float tile[32][33];
    const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    const int tx = threadIdx.x % 32, ty = threadIdx.x / 32;
    for (int r = ty; r < 32; r += 8)
        if (r0 + r < rows && c0 + tx < cols) tile[r][tx] = in[(size_t)(r0 + r) * cols + c0 + tx];
    __syncthreads();
    for (int c = ty; c < 32; c += 8)
        if (c0 + c < cols && r0 + tx < rows) out[(size_t)(c0 + c) * rows + r0 + tx] = tile[tx][c];
}

// dX[t,:] += dz[t,:] W_r^T = sum_j dz[t,j] * W_r^T[e_j,:]: one CTA per token walks its k selected rows
// of W_r^T (contiguous, L2-resident) four columns per thread; dX is read, updated in fp32 and rounded
// back to bf16.  d is a multiple of 8.
__global__ void __launch_bounds__(256) route_bwd_dx_kernel(const float* __restrict__ W_rT,
                                                           const int32_t* __restrict__ idx,
                                                           const float* __restrict__ dz_sel, bf16* __restrict__ dX,
                                                           int T, int d, int E, int k) {
    __shared__ int32_t es[32];
    __shared__ float dzs[32];
    const int t = blockIdx.x;
    if (threadIdx.x < k) {
        es[threadIdx.x] = idx[(size_t)t * k + threadIdx.x];
        dzs[threadIdx.x] = dz_sel[(size_t)t * k + threadIdx.x];
    }
    __syncthreads();
    for (int i = threadIdx.x * 4; i < d; i += 256 * 4) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int j = 0; j < k; ++j) {
            const float4 w = *reinterpret_cast<const float4*>(W_rT + (size_t)es[j] * d + i);
            const float s = dzs[j];
            acc.x = fmaf(s, w.x, acc.x); acc.y = fmaf(s, w.y, acc.y);
            acc.z = fmaf(s, w.z, acc.z); acc.w = fmaf(s, w.w, acc.w);
        }
        uint2* px = reinterpret_cast<uint2*>(dX + (size_t)t * d + i);
        uint2 v = *px;
        v.x = pack_bf16x2(bf16_lo(v.x) + acc.x, bf16_hi(v.x) + acc.y);
        v.y = pack_bf16x2(bf16_lo(v.y) + acc.z, bf16_hi(v.y) + acc.w);
        *px = v;
    }
}

}  // namespace mop
