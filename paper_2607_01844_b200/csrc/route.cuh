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
// Fast scoring path: logits on the tensor cores, the contract's chain only where it can matter.
//
// 1. W_r (fp32) is split into three bf16 pieces, hi + mid + lo = W_r to 2^-24 relative (each
//    residual is exact in fp32), and x (bf16) is multiplied by the pieces on the tensor cores: z~
//    (route_score_pair_kernel; the K loop is summed in segments of 192, all three pieces, so that the
//    truncating accumulation inside the tensor core stays short; the segments are added in fp32 registers).
//    Every product is exact; what separates z~ from the contract's logit z (one fp32 fused
//    multiply-add per i, i ascending) is the rounding of the two summations.  Each rounding is at most
//    u = 2^-24 of a partial sum, and the partial sums of a logit grow like a random walk towards
//    ||x|| ||w|| / sqrt(d) for data without a common direction: d roundings give a standard deviation of
//    u ||x|| ||w|| / sqrt(6) per summation, whatever d.  The selection relies on
//        |z~ - z|  <=  eps_z(t) = 24 u ||x_t||_2 max_e ||W_r[:,e]||_2        (40 standard deviations).
//    This is a model, not a worst case (which is d u ||x|| ||w||): the realised maximum over millions
//    of logits is 3 to 6.2 u ||x|| ||w|| on every shape tried, the tests assert it, and every logit that
//    the kernel re-evaluates is compared with half the bound as it runs (mop_route_stats).
//    In key space a logit error e moves sigmoid(z) + b by at most (s (1 - s) + e / 8) e + 4e-7; approximate
//    keys are formed with the fast sigmoid, whose own error (below 1e-6) is added to that.
// 2. Screening pass, one warp per token: the k largest approximate keys, every key with the interval that
//    holds its exact value.  If the intervals of adjacent picks are disjoint and no other expert's
//    interval reaches the weakest pick, the exact keys have the same order and the token is done
//    (more than nine tenths of the tokens).  The others are listed.  Resolving pass, one warp per listed
//    token: it evaluates the contract's chain (__fmaf_rn, i ascending, W_r read through its transposed
//    copy) for the experts in doubt, whose intervals become points and whose keys are the contract's,
//    writes those logits over z~, and selects again, until nothing that matters overlaps.  Indices and
//    their order are then those of the exact path.
// 3. Gates are ratios of scores, not an order: a pick keeps its approximate logit unless that could move
//    its gate by more than 5e-6 relative (score far from saturation), in which case its chain is
//    evaluated too; the gates then agree with the exact path's to 1e-6 + 1e-5 g.
// ---------------------------------------------------------------------------------------------

// W_r [d,E] -> three bf16 pieces [3,d,E], the transposed copy W_r^T [E,d] (32 x 32 tiles through shared
// memory) and, per 32-row slab, the partial squared column norms (summed by route_wnorm_kernel).
__global__ void __launch_bounds__(256) route_prep_kernel(const float* __restrict__ W_r, bf16* __restrict__ pieces,
                                                         float* __restrict__ W_rT, float* __restrict__ colsq,
                                                         int d, int E) {
    __shared__ float tile[32][33];
    const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    const int tx = threadIdx.x % 32, ty = threadIdx.x / 32;
    const size_t n = (size_t)d * E;
    for (int r = ty; r < 32; r += 8) {
        float w = 0.0f;
        if (r0 + r < d && c0 + tx < E) {
            const size_t i = (size_t)(r0 + r) * E + c0 + tx;
            w = W_r[i];
            const bf16 hi = __float2bfloat16_rn(w);
            const float r1 = w - __bfloat162float(hi);          // exact
            const bf16 mid = __float2bfloat16_rn(r1);
            const float r2 = r1 - __bfloat162float(mid);        // exact
            pieces[i] = hi;
            pieces[n + i] = mid;
            pieces[2 * n + i] = __float2bfloat16_rn(r2);
        }
        tile[r][tx] = w;
    }
    __syncthreads();
    for (int c = ty; c < 32; c += 8)
        if (c0 + c < E && r0 + tx < d) W_rT[(size_t)(c0 + c) * d + r0 + tx] = tile[tx][c];
    if (ty == 0 && c0 + tx < E) {
        float sq = 0.0f;
        for (int r = 0; r < 32; ++r) sq = fmaf(tile[r][tx], tile[r][tx], sq);
        colsq[(size_t)blockIdx.y * E + c0 + tx] = sq;
    }
}

// Squared column norms ||W_r[:,e]||^2 from the slab partials: one warp per expert, fixed order (reproducible).
__global__ void __launch_bounds__(256) route_wnorm_kernel(const float* __restrict__ colsq, float* __restrict__ wsq,
                                                          int slabs, int E) {
    const int lane = threadIdx.x % 32;
    const int e = blockIdx.x * 8 + threadIdx.x / 32;
    if (e >= E) return;
    float sq = 0.0f;
    for (int s = lane; s < slabs; s += 32) sq += colsq[(size_t)s * E + e];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, off);
    if (lane == 0) wsq[e] = sq;
}

// ||x_t||_2 per token: one warp per row, 16-byte loads.
__global__ void __launch_bounds__(256) route_xnorm_kernel(const bf16* __restrict__ x, float* __restrict__ xnorm, int T,
                                                          int d) {
    const int lane = threadIdx.x % 32;
    const int t = blockIdx.x * 8 + threadIdx.x / 32;
    if (t >= T) return;
    const uint4* row = reinterpret_cast<const uint4*>(x + (size_t)t * d);
    float sq = 0.0f;
    for (int v = lane; v < d / 8; v += 32) {
        const uint4 q = __ldg(row + v);
        const uint32_t w4[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float a = bf16_lo(w4[j]), b = bf16_hi(w4[j]);
            sq = fmaf(a, a, sq);
            sq = fmaf(b, b, sq);
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, off);
    if (lane == 0) xnorm[t] = sqrtf(sq);
}

constexpr int SELF_WARPS = 2;     // warps per block of the fast selection (a warp that re-evaluates takes ~20 us)
constexpr float ROUTE_EPS_C = 24.0f;      // order:  |z~ - z| <= C 2^-24 ||x_t|| max_e ||W_r[:,e]||  (see below)
constexpr float ROUTE_EPS_GATE_C = 6.0f;  // gates:  the same with the largest error seen, not a bound (a tolerance, not an order)
constexpr float ROUTE_GATE_REL = 5e-6f;   // a pick whose gate could be off by more than this (relative) gets its chain
constexpr int SELF_XCHUNK = 512;  // elements of the token's row staged per step of the exact chains
constexpr int SELF_CAND = 4;      // chains evaluated side by side (one lane each), their W_r^T rows staged in shared memory
constexpr int SELF_WPITCH = SELF_XCHUNK + 4;   // row pitch of the staged W_r^T chunks: lanes read different banks
constexpr int SELF_SMEM_FLOATS = SELF_XCHUNK + SELF_CAND * SELF_WPITCH;   // per warp, besides the 2 E logit / list words

// Order-preserving map of a finite float to an unsigned integer (-0 counts as +0, as in a float comparison).
__device__ __forceinline__ uint32_t key_ord(float f) {
    uint32_t u = __float_as_uint(f);
    if (u == 0x80000000u) u = 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// k selection rounds over keys held in registers: lane l owns the experts e = l + 32 q, q < Q, key kv[q].
// A round is two warp reductions (largest key among the lanes' best untaken keys, then the lowest expert id
// among the lanes that hold it) and a rescan of the winner's own keys.  Lane j < k keeps the j-th pick: its
// expert, its key and the logit its gate is computed from; `taken` marks this lane's picked experts.
// Same order as route_select_kernel: larger key first, equal keys by lower id.
template <int Q>
__device__ __forceinline__ void select_rounds_reg(const float (&kv)[Q], uint32_t invalid, const float* zg, int k, int lane,
                                                  int& my_e, float& my_key, float& my_z, uint32_t& taken) {
    taken = 0;
    my_e = -1; my_key = 0.0f; my_z = 0.0f;
    float bk = 0.0f; int bq = -1;
    auto rescan = [&]() {
        bq = -1; bk = 0.0f;
        const uint32_t off = taken | invalid;
#pragma unroll
        for (int q = 0; q < Q; ++q)
            if (!((off >> q) & 1u) && (bq < 0 || kv[q] > bk)) { bq = q; bk = kv[q]; }
    };
    rescan();
    for (int j = 0; j < k; ++j) {
        const uint32_t mine = bq >= 0 ? key_ord(bk) : 0u;            // 0 lies below the image of every finite key
        const uint32_t top = __reduce_max_sync(0xffffffffu, mine);
        const int cand = (bq >= 0 && mine == top) ? lane + 32 * bq : 0x7fffffff;
        const int win = __reduce_min_sync(0xffffffffu, cand);
        const float wkey = __shfl_sync(0xffffffffu, bk, win & 31);
        if ((win & 31) == lane) { taken |= 1u << (win >> 5); rescan(); }
        if (j == lane) { my_e = win; my_key = wkey; my_z = zg[win]; }
    }
}

__device__ __forceinline__ float route_key(float zz, float b, int score_fn, int bias_mode) {
    return (score_fn == 1 && bias_mode == 1) ? __fadd_rn(sigmoid_contract(zz), b) : zz;
}
// Key of an approximate logit: the sigmoid by the fast exponential and division.  Against the contract's sequence it is
// off by less than 1e-6 (exponential: 2 + 1.173 |z| ulp, times the slope s (1 - s): at most 8e-8; division 2 ulp;
// the contract's own polynomial 2e-7), which key_error adds to the interval of such a key.
constexpr float ROUTE_FAST_KEY_ERR = 1e-6f;
__device__ __forceinline__ float route_key_approx(float zz, float b, int score_fn, int bias_mode) {
    return (score_fn == 1 && bias_mode == 1) ? sigmoidf_fast(zz) + b : zz;
}

// Bound on the error of an approximate key whose logit is off by at most ez (a little slack covers its own rounding).
__device__ __forceinline__ float key_error(float zz, float ez, int score_fn, int bias_mode) {
    if (!(score_fn == 1 && bias_mode == 1)) return ez;                   // the key is the logit itself
    const float s = sigmoidf_fast(zz);
    return 1.001f * (s * (1.0f - s) + 0.125f * ez) * ez + 4e-7f + ROUTE_FAST_KEY_ERR;   // |s''| <= 0.1
}

// One token, one warp.  RESOLVE = false: the screening pass; it returns false, writing nothing, as soon as some
// order or gate is in doubt.  RESOLVE = true: evaluates the chains in doubt until everything is settled.
// Lane l holds the keys of the experts l + 32 q in registers (Q = ceil(E / 32) rounded up to a supported size).
// zg: E floats (logits); clist: E ints, xs, ws: staging of the chains (RESOLVE only).
template <bool RESOLVE, int Q>
__device__ __forceinline__ bool route_token(int t, int lane, float* zg, int32_t* clist, float* xs, float* ws,
                                            float* __restrict__ z, const float* __restrict__ z1,
                                            const float* __restrict__ bias,
                                            const bf16* __restrict__ x, const float* __restrict__ W_rT,
                                            const float* __restrict__ xnorm, float wmax, int32_t* __restrict__ idx,
                                            float* __restrict__ gate, int32_t* __restrict__ stats, int d, int E, int k,
                                            int score_fn, int bias_mode) {
    float* zrow = z + (size_t)t * E;
    float kv[Q];
    uint32_t invalid = 0;                            // slots q of this lane beyond E
#pragma unroll
    for (int q = 0; q < Q; ++q) {
        const int e = lane + 32 * q;
        kv[q] = 0.0f;
        if (e < E) {
            float zz = zrow[e];
            if (z1) {                                // the logit GEMM left two partial sums over K: add, keep the sum
                zz += z1[(size_t)t * E + e];
                zrow[e] = zz;
            }
            const float b = bias_mode ? bias[e] : 0.0f;
            if (bias_mode == 2) zz = __fadd_rn(zz, b);
            kv[q] = route_key_approx(zz, b, score_fn, bias_mode);
            zg[e] = zz;
        } else {
            invalid |= 1u << q;
        }
    }
    __syncwarp();
    // Bound of this token's logit error (see above).
    const float scale = 5.9604645e-8f * xnorm[t] * wmax;
    const float ez = ROUTE_EPS_C * scale, ez_gate = ROUTE_EPS_GATE_C * scale;
    uint32_t exact = 0;                              // this lane's experts that carry the chain's logit
    int my_e; float my_key, my_z; uint32_t taken;
    int n_chains = 0, n_bad = 0;
    for (int iter = 0; iter <= k + 1; ++iter) {
        select_rounds_reg<Q>(kv, invalid, zg, k, lane, my_e, my_key, my_z, taken);
        // interval [lo, hi] that holds the exact key of each pick (a point once the chain was evaluated)
        const bool pick = lane < k;
        const uint32_t owner_exact = __shfl_sync(0xffffffffu, exact, pick ? (my_e & 31) : 0);
        const uint32_t pick_exact = pick ? (owner_exact >> (my_e >> 5)) & 1u : 1u;
        const float my_err = (pick && !pick_exact) ? key_error(my_z, ez, score_fn, bias_mode) : 0.0f;
        const float lo = pick ? my_key - my_err : INFINITY, hi = pick ? my_key + my_err : -INFINITY;
        const float next_hi = __shfl_down_sync(0xffffffffu, hi, 1), prev_lo = __shfl_up_sync(0xffffffffu, lo, 1);
        // a pick is in doubt if it may swap with a neighbour (NaN compares unsure: inputs must be finite)
        bool doubt = pick && ((lane + 1 < k && !(lo > next_hi)) || (lane > 0 && !(prev_lo > hi)));
        float lo_min = lo;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) lo_min = fminf(lo_min, __shfl_xor_sync(0xffffffffu, lo_min, off));
        // outsiders that could reach the weakest pick, and the picks they could reach.  Nearly all of them
        // fail already with the largest error any key can have (slope 1/4), which costs no transcendental.
        const float err_any = (score_fn == 1 && bias_mode == 1)
                                  ? 1.001f * (0.25f + 0.125f * ez) * ez + 4e-7f + ROUTE_FAST_KEY_ERR : ez;
        float out_hi = -INFINITY;
        int n_c = 0;
        bool any_cand = false;
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            const int e = lane + 32 * q;
            bool cand = false;
            if (!(((taken | invalid) >> q) & 1u) && !(kv[q] + err_any < lo_min)) {
                const bool ex = (exact >> q) & 1u;
                const float h = kv[q] + (ex ? 0.0f : key_error(zg[e], ez, score_fn, bias_mode));
                if (!(h < lo_min)) { out_hi = fmaxf(out_hi, h); cand = !ex; }
            }
            if constexpr (RESOLVE) {
                const uint32_t m = __ballot_sync(0xffffffffu, cand);
                if (m) {
                    if (cand) clist[n_c + __popc(m & ((1u << lane) - 1u))] = e;
                    n_c += __popc(m);
                }
            } else {
                any_cand |= cand;
            }
        }
        if constexpr (!RESOLVE) {
            if (__any_sync(0xffffffffu, any_cand)) return false;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) out_hi = fmaxf(out_hi, __shfl_xor_sync(0xffffffffu, out_hi, off));
        if (pick && !(lo > out_hi)) doubt = true;
        // gates: d g / g = (1 - s) dz for a sigmoid score, at most dz for a softmax over the picks
        if (pick && !pick_exact) {
            const float sens = (score_fn == 1) ? 1.0f - sigmoidf_fast(my_z) : 1.0f;
            if (sens * ez_gate > ROUTE_GATE_REL) doubt = true;
        }
        // picks in doubt whose logit is still approximate join the list
        const bool need = doubt && !pick_exact;
        const uint32_t m = __ballot_sync(0xffffffffu, need);
        if constexpr (!RESOLVE) {
            if (m) return false;
            break;
        }
        if (need) clist[n_c + __popc(m & ((1u << lane) - 1u))] = my_e;
        n_c += __popc(m);
        if (n_c == 0) break;                         // every order that matters is settled (exact ties go by id)
        __syncwarp();
        for (int c0 = 0; c0 < n_c; c0 += SELF_CAND) {
            const int nc = min(SELF_CAND, n_c - c0);
            const bool mine = lane < nc;
            const int e = mine ? clist[c0 + lane] : 0;
            float acc = 0.0f;
            // All lanes fetch: the token's chunk (16 bytes per lane) and the same chunk of every candidate's row
            // of W_r^T (lane l: 16-byte pieces l, l + 32, ... of the nc rows laid end to end).  The fetch of chunk
            // i + 1 is in flight while the chains run over chunk i.
            constexpr int WV = SELF_CAND * SELF_XCHUNK / 4 / 32;      // 16-byte pieces of W per lane and chunk
            constexpr int XV = SELF_XCHUNK / 8 / 32;                  // 16-byte pieces of x per lane and chunk
            uint4 xq[XV];
            float4 wq[WV];
            auto fetch = [&](int i0) {
                const int n = min(SELF_XCHUNK, d - i0);              // a multiple of 8
#pragma unroll
                for (int u = 0; u < XV; ++u)
                    if (lane + 32 * u < n / 8)
                        xq[u] = __ldg(reinterpret_cast<const uint4*>(x + (size_t)t * d + i0) + lane + 32 * u);
#pragma unroll
                for (int u = 0; u < WV; ++u) {
                    const int v = lane + 32 * u, c = v / (SELF_XCHUNK / 4), j = v % (SELF_XCHUNK / 4);
                    if (c < nc && 4 * j < n)
                        wq[u] = __ldg(reinterpret_cast<const float4*>(W_rT + (size_t)clist[c0 + c] * d + i0) + j);
                }
            };
            fetch(0);
            for (int i0 = 0; i0 < d; i0 += SELF_XCHUNK) {
                const int n = min(SELF_XCHUNK, d - i0);
                __syncwarp();
                // x stays bf16 in shared memory (16 bytes = 8 elements per load in the chains: every shared-memory
                // instruction of a warp costs a wavefront however few lanes take part, and the chains of all
                // resident warps together are bound by those wavefronts when most tokens are listed)
#pragma unroll
                for (int u = 0; u < XV; ++u) reinterpret_cast<uint4*>(xs)[lane + 32 * u] = xq[u];
#pragma unroll
                for (int u = 0; u < WV; ++u) {
                    const int v = lane + 32 * u, c = v / (SELF_XCHUNK / 4), j = v % (SELF_XCHUNK / 4);
                    if (c < nc) *reinterpret_cast<float4*>(ws + c * SELF_WPITCH + 4 * j) = wq[u];
                }
                __syncwarp();
                if (i0 + SELF_XCHUNK < d) fetch(i0 + SELF_XCHUNK);
                if (mine) {
                    // the contract's chain: one fused multiply-add per i, i ascending
                    const float* wrow = ws + lane * SELF_WPITCH;
#pragma unroll 4
                    for (int i = 0; i < n; i += 8) {
                        const float4 w0 = *reinterpret_cast<const float4*>(wrow + i);
                        const float4 w1 = *reinterpret_cast<const float4*>(wrow + i + 4);
                        const uint4 xv = *reinterpret_cast<const uint4*>(reinterpret_cast<const bf16*>(xs) + i);
                        acc = __fmaf_rn(bf16_lo(xv.x), w0.x, acc);
                        acc = __fmaf_rn(bf16_hi(xv.x), w0.y, acc);
                        acc = __fmaf_rn(bf16_lo(xv.y), w0.z, acc);
                        acc = __fmaf_rn(bf16_hi(xv.y), w0.w, acc);
                        acc = __fmaf_rn(bf16_lo(xv.z), w1.x, acc);
                        acc = __fmaf_rn(bf16_hi(xv.z), w1.y, acc);
                        acc = __fmaf_rn(bf16_lo(xv.w), w1.z, acc);
                        acc = __fmaf_rn(bf16_hi(xv.w), w1.w, acc);
                    }
                }
            }
            float newkey = 0.0f;
            if (mine) {
                if (fabsf(zrow[e] - acc) > 0.5f * ez) ++n_bad;       // the model of the error is checked as we go
                zrow[e] = acc;                       // the exact logit replaces the approximate one
                const float b = bias_mode ? bias[e] : 0.0f;
                const float zz = (bias_mode == 2) ? __fadd_rn(acc, b) : acc;
                newkey = route_key(zz, b, score_fn, bias_mode);      // the contract's key
                zg[e] = zz;
            }
            // the evaluated experts' keys go to their owner lanes, which mark them exact
            for (int j = 0; j < nc; ++j) {
                const int ej = clist[c0 + j];
                const float kj = __shfl_sync(0xffffffffu, newkey, j);
                if ((ej & 31) == lane) {
                    exact |= 1u << (ej >> 5);
#pragma unroll
                    for (int q = 0; q < Q; ++q)
                        if (q == (ej >> 5)) kv[q] = kj;
                }
            }
        }
        n_chains += n_c;
        __syncwarp();
    }
    if (RESOLVE && stats && n_chains > 0) {          // statistics only: no result depends on them
        n_bad = __reduce_add_sync(0xffffffffu, n_bad);
        if (lane == 0) { atomicAdd(stats, 1); atomicAdd(stats + 1, n_chains); if (n_bad) atomicAdd(stats + 2, n_bad); }
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
    return true;
}

// Largest column norm of W_r, from the squared norms: every lane returns it.
__device__ __forceinline__ float route_wmax(const float* __restrict__ wsq, int E, int lane) {
    float wmax2 = 0.0f;
    for (int e = lane; e < E; e += 32) wmax2 = fmaxf(wmax2, wsq[e]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) wmax2 = fmaxf(wmax2, __shfl_xor_sync(0xffffffffu, wmax2, off));
    return sqrtf(wmax2);
}

// Screening pass: every token, one warp each, little shared memory (high occupancy).  Tokens whose approximate
// keys settle everything are finished here; the others are listed for the resolving pass.  The list's order
// depends on timing, no result does.
constexpr int SCREEN_WARPS = 4;
template <int Q>
__global__ void __launch_bounds__(SCREEN_WARPS * 32) route_screen_kernel(
    float* __restrict__ z, const float* __restrict__ z1, const float* __restrict__ bias,
    const float* __restrict__ xnorm, const float* __restrict__ wsq, int32_t* __restrict__ idx, float* __restrict__ gate,
    int32_t* __restrict__ todo, int32_t* __restrict__ n_todo, int T, int d, int E, int k, int score_fn, int bias_mode) {
    extern __shared__ float sel_smem[];
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int t = blockIdx.x * SCREEN_WARPS + warp;
    if (t >= T) return;
    const float wmax = route_wmax(wsq, E, lane);
    const bool done = route_token<false, Q>(t, lane, sel_smem + (size_t)warp * E, nullptr, nullptr, nullptr, z, z1, bias,
                                            nullptr, nullptr, xnorm, wmax, idx, gate, nullptr, d, E, k, score_fn, bias_mode);
    if (!done && lane == 0) todo[atomicAdd(n_todo, 1)] = t;
}

// Resolving pass: the listed tokens, one warp each, with the staging memory of the chains.
template <int Q>
__global__ void __launch_bounds__(SELF_WARPS * 32) route_resolve_kernel(
    float* __restrict__ z, const float* __restrict__ bias, const bf16* __restrict__ x, const float* __restrict__ W_rT,
    const float* __restrict__ xnorm, const float* __restrict__ wsq, int32_t* __restrict__ idx,
    float* __restrict__ gate, const int32_t* __restrict__ todo, const int32_t* __restrict__ n_todo,
    int32_t* __restrict__ stats, int d, int E, int k, int score_fn, int bias_mode) {
    extern __shared__ float sel_smem[];
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int n = *n_todo;
    if ((int)blockIdx.x * SELF_WARPS >= n) return;
    float* zg = sel_smem + (size_t)warp * (2 * E + SELF_SMEM_FLOATS);
    int32_t* clist = reinterpret_cast<int32_t*>(zg + E);   // experts whose exact logit is needed
    float* xs = zg + 2 * E;                                 // a chunk of the token's row, fp32
    float* ws = xs + SELF_XCHUNK;                           // the same chunk of up to SELF_CAND rows of W_r^T
    const float wmax = route_wmax(wsq, E, lane);
    for (int i = blockIdx.x * SELF_WARPS + warp; i < n; i += gridDim.x * SELF_WARPS) {
        route_token<true, Q>(todo[i], lane, zg, clist, xs, ws, z, nullptr, bias, x, W_rT, xnorm, wmax, idx, gate, stats, d,
                             E, k, score_fn, bias_mode);
        __syncwarp();
    }
}

// The two passes for the smallest supported Q >= ceil(E / 32).
template <int Q>
inline void route_select_fast_q(float* z, const float* z1, const float* bias, const bf16* x, const float* W_rT, const float* xnorm,
                                const float* wsq, int32_t* idx, float* gate, int32_t* todo, int32_t* n_todo,
                                int32_t* stats, int T, int d, int E, int k, int score_fn, int bias_mode, int pass,
                                int resolve_blocks, cudaStream_t st) {
    if (pass == 0) {
        route_screen_kernel<Q><<<ceil_div(T, SCREEN_WARPS), SCREEN_WARPS * 32, (size_t)SCREEN_WARPS * E * sizeof(float), st>>>(
            z, z1, bias, xnorm, wsq, idx, gate, todo, n_todo, T, d, E, k, score_fn, bias_mode);
    } else {
        const size_t smem = (size_t)SELF_WARPS * (2 * E + SELF_SMEM_FLOATS) * sizeof(float);
        route_resolve_kernel<Q><<<resolve_blocks, SELF_WARPS * 32, smem, st>>>(z, bias, x, W_rT, xnorm, wsq, idx, gate, todo,
                                                                                n_todo, stats, d, E, k, score_fn, bias_mode);
    }
}
// Blocks of the resolving pass that are resident at once: its grid.  Every warp then walks its share of the list;
// a larger grid would run in waves of whole walks.
template <int Q>
inline int route_resolve_resident_q(int E, int sm_count) {
    int nb = 0;
    const size_t smem = (size_t)SELF_WARPS * (2 * E + SELF_SMEM_FLOATS) * sizeof(float);
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, route_resolve_kernel<Q>, SELF_WARPS * 32, smem) != cudaSuccess || nb < 1)
        nb = 1;
    return nb * sm_count;
}
inline int route_resolve_resident(int E, int sm_count) {
    const int q = ceil_div(E, 32);
    if (q <= 2) return route_resolve_resident_q<2>(E, sm_count);
    if (q <= 4) return route_resolve_resident_q<4>(E, sm_count);
    if (q <= 8) return route_resolve_resident_q<8>(E, sm_count);
    if (q <= 12) return route_resolve_resident_q<12>(E, sm_count);
    if (q <= 16) return route_resolve_resident_q<16>(E, sm_count);
    return route_resolve_resident_q<32>(E, sm_count);
}
inline void route_select_fast(float* z, const float* z1, const float* bias, const bf16* x, const float* W_rT, const float* xnorm,
                              const float* wsq, int32_t* idx, float* gate, int32_t* todo, int32_t* n_todo, int32_t* stats,
                              int T, int d, int E, int k, int score_fn, int bias_mode, int pass, int resolve_blocks,
                              cudaStream_t st) {
    const int q = ceil_div(E, 32);
#define MOP_ROUTE_Q(QQ)                                                                                                 \
    route_select_fast_q<QQ>(z, z1, bias, x, W_rT, xnorm, wsq, idx, gate, todo, n_todo, stats, T, d, E, k, score_fn, bias_mode, \
                            pass, resolve_blocks, st)
    if (q <= 2) MOP_ROUTE_Q(2);
    else if (q <= 4) MOP_ROUTE_Q(4);
    else if (q <= 8) MOP_ROUTE_Q(8);
    else if (q <= 12) MOP_ROUTE_Q(12);
    else if (q <= 16) MOP_ROUTE_Q(16);
    else MOP_ROUTE_Q(32);
#undef MOP_ROUTE_Q
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
