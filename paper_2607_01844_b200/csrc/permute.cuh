// Count / prefix-sum permutation of token-expert assignments into expert-contiguous rows, and the
// row movers (scatter x -> Xp, k-row combine Yp -> Y).  No atomics anywhere: the order inside an
// expert is the assignment id, fixed by a two-level (warp segment, expert) prefix sum.
#pragma once
#include "common.cuh"

namespace mop {

constexpr int PERM_SEG = 512;    // assignments walked by one warp ("unit")
constexpr int PERM_WARPS = 4;    // warps per block in the histogram / rank kernels

// Histogram per unit: partial[u][e] = number of assignments of unit u that go to expert e.
__global__ void __launch_bounds__(PERM_WARPS * 32) perm_hist_kernel(const int32_t* __restrict__ idx,
                                                                    int32_t* __restrict__ partial, int M, int E) {
    extern __shared__ int32_t perm_smem[];
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    int32_t* cnt = perm_smem + (size_t)warp * E;
    const int unit = blockIdx.x * PERM_WARPS + warp;
    const int a0 = unit * PERM_SEG;
    if (a0 >= M) return;
    for (int e = lane; e < E; e += 32) cnt[e] = 0;
    __syncwarp();
    for (int it = 0; it < PERM_SEG / 32; ++it) {
        const int a = a0 + it * 32 + lane;
        int e = (a < M) ? idx[a] : -1;
        if (e < 0 || e >= E) e = -1;
        const uint32_t same = __match_any_sync(0xffffffffu, e);
        if (e >= 0 && lane == __ffs(same) - 1) cnt[e] += __popc(same);
        __syncwarp();
    }
    for (int e = lane; e < E; e += 32) partial[(size_t)unit * E + e] = cnt[e];
}

// Scan on one block: counts, offsets (exclusive scan over experts) and, in place of partial[u][e], the first
// row of unit u inside expert e; thread e owns expert e (strided if E > blockDim).  Used when there is nothing
// to permute (it still writes counts and offsets); otherwise perm_scan_cols_kernel + perm_rank_kernel do this.
__global__ void __launch_bounds__(1024) perm_scan_kernel(int32_t* __restrict__ partial, int32_t* __restrict__ counts,
                                                         int32_t* __restrict__ offsets, int units, int E) {
    extern __shared__ int32_t scan_smem[];  // E + 1
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
        int32_t run = 0;
        for (int u = 0; u < units; ++u) {
            const int32_t c = partial[(size_t)u * E + e];
            partial[(size_t)u * E + e] = run;
            run += c;
        }
        counts[e] = run;
        scan_smem[e] = run;
    }
    __syncthreads();
    if (threadIdx.x < 32) {
        // exclusive scan over E by one warp, 32 experts per step
        int32_t carry = 0;
        for (int e0 = 0; e0 < E; e0 += 32) {
            const int e = e0 + threadIdx.x;
            const int32_t c = (e < E) ? scan_smem[e] : 0;
            int32_t inc = c;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int32_t o = __shfl_up_sync(0xffffffffu, inc, off);
                if ((int)threadIdx.x >= off) inc += o;
            }
            if (e < E) scan_smem[e] = carry + inc - c;
            carry += __shfl_sync(0xffffffffu, inc, 31);
        }
        if (threadIdx.x == 0) scan_smem[E] = carry;
    }
    __syncthreads();
    for (int e = threadIdx.x; e <= E; e += blockDim.x) offsets[e] = scan_smem[e];
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
        const int32_t o = scan_smem[e];
        for (int u = 0; u < units; ++u) partial[(size_t)u * E + e] += o;
    }
}

// Column scan, spread over the GPU: a block owns 32 experts (a lane each: coalesced 128-byte rows of
// partial[u][.]) and its eight warps own eight contiguous ranges of units.  In place of partial[u][e]: the
// number of rows of expert e in the units before u; counts[e] = the expert's total.  Fixed order, no atomics.
constexpr int PSCAN_WARPS = 8;
__global__ void __launch_bounds__(PSCAN_WARPS * 32) perm_scan_cols_kernel(int32_t* __restrict__ partial,
                                                                          int32_t* __restrict__ counts, int units,
                                                                          int E) {
    __shared__ int32_t tot[PSCAN_WARPS][32];
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int e = blockIdx.x * 32 + lane;
    const int per = (units + PSCAN_WARPS - 1) / PSCAN_WARPS;
    const int u0 = min(units, warp * per), u1 = min(units, u0 + per);
    int32_t run = 0;
    if (e < E)
        for (int u = u0; u < u1; ++u) {
            const int32_t c = partial[(size_t)u * E + e];
            partial[(size_t)u * E + e] = run;
            run += c;
        }
    tot[warp][lane] = run;
    __syncthreads();
    int32_t before = 0, total = 0;
#pragma unroll
    for (int w = 0; w < PSCAN_WARPS; ++w) {
        if (w < warp) before += tot[w][lane];
        total += tot[w][lane];
    }
    if (e < E) {
        if (before)
            for (int u = u0; u < u1; ++u) partial[(size_t)u * E + e] += before;
        if (warp == 0) counts[e] = total;
    }
}

// Rank: second walk over the same segments; perm_row[a] = offsets[e] + base[u][e] + rank inside the unit.
// Every block scans counts[] into the experts' offsets for itself (E <= 1024 words of shared memory);
// block 0 also writes them out.
__global__ void __launch_bounds__(PERM_WARPS * 32) perm_rank_kernel(const int32_t* __restrict__ idx,
                                                                    const int32_t* __restrict__ base,
                                                                    const int32_t* __restrict__ counts,
                                                                    int32_t* __restrict__ offsets,
                                                                    int32_t* __restrict__ perm_row,
                                                                    int32_t* __restrict__ row_src, int M, int E) {
    extern __shared__ int32_t perm_smem[];
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    int32_t* off = perm_smem + (size_t)PERM_WARPS * E;   // E + 1 words
    for (int e = threadIdx.x; e < E; e += blockDim.x) off[e] = counts[e];
    __syncthreads();
    if (warp == 0) {
        // exclusive scan over E by one warp, 32 experts per step
        int32_t carry = 0;
        for (int e0 = 0; e0 < E; e0 += 32) {
            const int e = e0 + lane;
            const int32_t c = (e < E) ? off[e] : 0;
            int32_t inc = c;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int32_t v = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += v;
            }
            if (e < E) off[e] = carry + inc - c;
            carry += __shfl_sync(0xffffffffu, inc, 31);
        }
        if (lane == 0) off[E] = carry;
    }
    __syncthreads();
    if (blockIdx.x == 0)
        for (int e = threadIdx.x; e <= E; e += blockDim.x) offsets[e] = off[e];
    int32_t* run = perm_smem + (size_t)warp * E;
    const int unit = blockIdx.x * PERM_WARPS + warp;
    const int a0 = unit * PERM_SEG;
    if (a0 >= M) return;
    for (int e = lane; e < E; e += 32) run[e] = base[(size_t)unit * E + e] + off[e];
    __syncwarp();
    const uint32_t lt = (1u << lane) - 1u;
    for (int it = 0; it < PERM_SEG / 32; ++it) {
        const int a = a0 + it * 32 + lane;
        int e = (a < M) ? idx[a] : -1;
        if (e < 0 || e >= E) e = -1;
        const uint32_t same = __match_any_sync(0xffffffffu, e);
        int32_t p = -1;
        if (e >= 0) p = run[e] + __popc(same & lt);
        __syncwarp();
        if (e >= 0 && lane == __ffs(same) - 1) run[e] += __popc(same);
        __syncwarp();
        if (a < M) {
            perm_row[a] = p;
            if (p >= 0) row_src[p] = a;
        }
    }
}

// Small layers: histogram, scan and rank in ONE block (the three launches above cost more than their work when
// there are only a few units).  Warp w owns the units w, w + 32, ...; cnt[u][e] lives in shared memory, first as
// the unit's histogram, then as the first row of unit u inside expert e.  Same tables as the three-kernel path.
constexpr int PERM_SMALL_MAX_UNITS = 8;       // beyond that the three parallel kernels are faster (measured at 48 units)
constexpr int PERM_SMALL_MAX_WORDS = 10240;     // units * E words of shared memory (40 KiB)
__global__ void __launch_bounds__(1024) perm_small_kernel(const int32_t* __restrict__ idx, int32_t* __restrict__ counts,
                                                          int32_t* __restrict__ offsets, int32_t* __restrict__ perm_row,
                                                          int32_t* __restrict__ row_src, int M, int E, int units) {
    extern __shared__ int32_t perm_smem[];
    int32_t* cnt = perm_smem;                      // [units][E]
    int32_t* off = perm_smem + (size_t)units * E;  // [E + 1]
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    for (int i = threadIdx.x; i < units * E; i += blockDim.x) cnt[i] = 0;
    __syncthreads();
    for (int u = warp; u < units; u += 32) {
        int32_t* c = cnt + (size_t)u * E;
        for (int it = 0; it < PERM_SEG / 32; ++it) {
            const int a = u * PERM_SEG + it * 32 + lane;
            int e = (a < M) ? idx[a] : -1;
            if (e < 0 || e >= E) e = -1;
            const uint32_t same = __match_any_sync(0xffffffffu, e);
            if (e >= 0 && lane == __ffs(same) - 1) c[e] += __popc(same);
            __syncwarp();
        }
    }
    __syncthreads();
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
        int32_t run = 0;
        for (int u = 0; u < units; ++u) {
            const int32_t c = cnt[(size_t)u * E + e];
            cnt[(size_t)u * E + e] = run;
            run += c;
        }
        counts[e] = run;
        off[e] = run;
    }
    __syncthreads();
    if (warp == 0) {
        int32_t carry = 0;
        for (int e0 = 0; e0 < E; e0 += 32) {
            const int e = e0 + lane;
            const int32_t c = (e < E) ? off[e] : 0;
            int32_t inc = c;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int32_t v = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += v;
            }
            if (e < E) off[e] = carry + inc - c;
            carry += __shfl_sync(0xffffffffu, inc, 31);
        }
        if (lane == 0) off[E] = carry;
    }
    __syncthreads();
    for (int e = threadIdx.x; e <= E; e += blockDim.x) offsets[e] = off[e];
    const uint32_t lt = (1u << lane) - 1u;
    for (int u = warp; u < units; u += 32) {
        int32_t* run = cnt + (size_t)u * E;
        for (int e = lane; e < E; e += 32) run[e] += off[e];
        __syncwarp();
        for (int it = 0; it < PERM_SEG / 32; ++it) {
            const int a = u * PERM_SEG + it * 32 + lane;
            int e = (a < M) ? idx[a] : -1;
            if (e < 0 || e >= E) e = -1;
            const uint32_t same = __match_any_sync(0xffffffffu, e);
            int32_t p = -1;
            if (e >= 0) p = run[e] + __popc(same & lt);
            __syncwarp();
            if (e >= 0 && lane == __ffs(same) - 1) run[e] += __popc(same);
            __syncwarp();
            if (a < M) {
                perm_row[a] = p;
                if (p >= 0) row_src[p] = a;
            }
        }
    }
}
inline bool perm_small_fits(int units, int E) {
    return units > 0 && units <= PERM_SMALL_MAX_UNITS && (long long)units * E <= PERM_SMALL_MAX_WORDS;
}

// Scatter rows: one warp per token reads x[t,:] once (16-byte vectors, coalesced) and writes it to
// its k destination rows.  Used for x -> Xp and for dY -> dYp.
__global__ void __launch_bounds__(256) scatter_rows_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst,
                                                           const int32_t* __restrict__ perm_row, int T, int k,
                                                           int vec_per_row) {
    const int warps_per_block = blockDim.x / 32;
    const int lane = threadIdx.x % 32;
    for (int t = blockIdx.x * warps_per_block + threadIdx.x / 32; t < T; t += gridDim.x * warps_per_block) {
        int32_t myrow = -1;
        if (lane < k) myrow = perm_row[(size_t)t * k + lane];  // k <= 32 checked on the host
        const uint4* s = src + (size_t)t * vec_per_row;
        for (int c0 = 0; c0 < vec_per_row; c0 += 128) {
            uint4 v[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int c = c0 + q * 32 + lane;
                if (c < vec_per_row) v[q] = __ldg(s + c);
            }
            for (int j = 0; j < k; ++j) {
                const int32_t p = __shfl_sync(0xffffffffu, myrow, j);
                if (p < 0) continue;
                uint4* o = dst + (size_t)p * vec_per_row;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int c = c0 + q * 32 + lane;
                    if (c < vec_per_row) __stcs(o + c, v[q]);
                }
            }
        }
    }
}

// Combine: Y[t,:] = bf16(sum_j Yp[perm_row[t*k+j],:]) with the k-row sum kept in fp32 registers,
// j ascending.  One warp per token, 16-byte vectors.
__global__ void __launch_bounds__(256) combine_rows_kernel(const uint4* __restrict__ Yp,
                                                           const int32_t* __restrict__ perm_row,
                                                           uint4* __restrict__ Y, int T, int k, int vec_per_row) {
    const int warps_per_block = blockDim.x / 32;
    const int lane = threadIdx.x % 32;
    for (int t = blockIdx.x * warps_per_block + threadIdx.x / 32; t < T; t += gridDim.x * warps_per_block) {
        int32_t myrow = -1;
        if (lane < k) myrow = perm_row[(size_t)t * k + lane];
        for (int c0 = 0; c0 < vec_per_row; c0 += 64) {
            float acc[2][8];
#pragma unroll
            for (int q = 0; q < 2; ++q)
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[q][i] = 0.0f;
            for (int j = 0; j < k; ++j) {
                const int32_t p = __shfl_sync(0xffffffffu, myrow, j);
                if (p < 0) continue;
                const uint4* r = Yp + (size_t)p * vec_per_row;
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    const int c = c0 + q * 32 + lane;
                    if (c < vec_per_row) {
                        const uint4 v = __ldcs(r + c);
                        acc[q][0] += bf16_lo(v.x); acc[q][1] += bf16_hi(v.x);
                        acc[q][2] += bf16_lo(v.y); acc[q][3] += bf16_hi(v.y);
                        acc[q][4] += bf16_lo(v.z); acc[q][5] += bf16_hi(v.z);
                        acc[q][6] += bf16_lo(v.w); acc[q][7] += bf16_hi(v.w);
                    }
                }
            }
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int c = c0 + q * 32 + lane;
                if (c < vec_per_row) {
                    uint4 o;
                    o.x = pack_bf16x2(acc[q][0], acc[q][1]);
                    o.y = pack_bf16x2(acc[q][2], acc[q][3]);
                    o.z = pack_bf16x2(acc[q][4], acc[q][5]);
                    o.w = pack_bf16x2(acc[q][6], acc[q][7]);
                    Y[(size_t)t * vec_per_row + c] = o;
                }
            }
        }
    }
}

// Scatter rows with the whole source row in registers (VPL 16-byte vectors per lane, rows of up to 512 VPL
// bytes): the row is read once and each of its k copies is written as one contiguous run, which DRAM takes
// better than pieces of 2 KiB interleaved over k rows (random 2 KiB pieces: 4.4 TB/s at T = 16384, d = 7168).
template <int VPL>
__global__ void __launch_bounds__(256) scatter_rows_reg_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst,
                                                               const int32_t* __restrict__ perm_row, int T, int k,
                                                               int vec_per_row) {
    const int warps_per_block = blockDim.x / 32;
    const int lane = threadIdx.x % 32;
    for (int t = blockIdx.x * warps_per_block + threadIdx.x / 32; t < T; t += gridDim.x * warps_per_block) {
        int32_t myrow = -1;
        if (lane < k) myrow = perm_row[(size_t)t * k + lane];  // k <= 32 checked on the host
        const uint4* s = src + (size_t)t * vec_per_row;
        uint4 v[VPL];
#pragma unroll
        for (int q = 0; q < VPL; ++q) {
            const int c = q * 32 + lane;
            if (c < vec_per_row) v[q] = __ldg(s + c);
        }
        for (int j = 0; j < k; ++j) {
            const int32_t p = __shfl_sync(0xffffffffu, myrow, j);
            if (p < 0) continue;
            uint4* o = dst + (size_t)p * vec_per_row;
#pragma unroll
            for (int q = 0; q < VPL; ++q) {
                const int c = q * 32 + lane;
                if (c < vec_per_row) __stcs(o + c, v[q]);
            }
        }
    }
}

// Combine with longer runs per row: the row is walked in segments of 32 SEG vectors (3.5 or 4 KiB); for every
// segment the k rows are read one after the other, the next row's vectors in flight while the current ones are
// added.  Same sums in the same order as combine_rows_kernel (j ascending, fp32), so the same bits.
template <int SEG>
__global__ void __launch_bounds__(256) combine_rows_seg_kernel(const uint4* __restrict__ Yp,
                                                               const int32_t* __restrict__ perm_row,
                                                               uint4* __restrict__ Y, int T, int k, int vec_per_row) {
    const int warps_per_block = blockDim.x / 32;
    const int lane = threadIdx.x % 32;
    for (int t = blockIdx.x * warps_per_block + threadIdx.x / 32; t < T; t += gridDim.x * warps_per_block) {
        int32_t myrow = -1;
        if (lane < k) myrow = perm_row[(size_t)t * k + lane];
        for (int c0 = 0; c0 < vec_per_row; c0 += 32 * SEG) {
            float acc[SEG][8];
#pragma unroll
            for (int q = 0; q < SEG; ++q)
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[q][i] = 0.0f;
            uint4 a[SEG], b[SEG];
            auto load = [&](uint4 (&buf)[SEG], int j) -> bool {
                const int32_t p = __shfl_sync(0xffffffffu, myrow, j);
                if (p < 0) return false;
                const uint4* r = Yp + (size_t)p * vec_per_row + c0 + lane;
#pragma unroll
                for (int q = 0; q < SEG; ++q)
                    if (c0 + q * 32 + lane < vec_per_row) buf[q] = __ldcs(r + q * 32);
                return true;
            };
            auto add = [&](const uint4 (&buf)[SEG]) {
#pragma unroll
                for (int q = 0; q < SEG; ++q) {
                    if (c0 + q * 32 + lane < vec_per_row) {
                        const uint4 v = buf[q];
                        acc[q][0] += bf16_lo(v.x); acc[q][1] += bf16_hi(v.x);
                        acc[q][2] += bf16_lo(v.y); acc[q][3] += bf16_hi(v.y);
                        acc[q][4] += bf16_lo(v.z); acc[q][5] += bf16_hi(v.z);
                        acc[q][6] += bf16_lo(v.w); acc[q][7] += bf16_hi(v.w);
                    }
                }
            };
            bool va = load(a, 0), vb = false;
            for (int j = 0; j < k; j += 2) {
                if (j + 1 < k) vb = load(b, j + 1);
                if (va) add(a);
                if (j + 2 < k) va = load(a, j + 2);
                if (j + 1 < k && vb) add(b);
            }
#pragma unroll
            for (int q = 0; q < SEG; ++q) {
                const int c = c0 + q * 32 + lane;
                if (c < vec_per_row) {
                    uint4 o;
                    o.x = pack_bf16x2(acc[q][0], acc[q][1]);
                    o.y = pack_bf16x2(acc[q][2], acc[q][3]);
                    o.z = pack_bf16x2(acc[q][4], acc[q][5]);
                    o.w = pack_bf16x2(acc[q][6], acc[q][7]);
                    Y[(size_t)t * vec_per_row + c] = o;
                }
            }
        }
    }
}

// Launchers: the register-row forms for rows of up to 16 KiB, the chunked kernels otherwise.
inline void launch_scatter_rows(const uint4* src, uint4* dst, const int32_t* perm_row, int T, int k, int vec_per_row,
                                int sm_count, cudaStream_t st) {
    const int blocks = min(ceil_div(T, 8), sm_count * 8);
    if (blocks <= 0) return;
    if (vec_per_row <= 32 * 8) scatter_rows_reg_kernel<8><<<blocks, 256, 0, st>>>(src, dst, perm_row, T, k, vec_per_row);
    else if (vec_per_row <= 32 * 16) scatter_rows_reg_kernel<16><<<blocks, 256, 0, st>>>(src, dst, perm_row, T, k, vec_per_row);
    else if (vec_per_row <= 32 * 28) scatter_rows_reg_kernel<28><<<blocks, 256, 0, st>>>(src, dst, perm_row, T, k, vec_per_row);
    else if (vec_per_row <= 32 * 32) scatter_rows_reg_kernel<32><<<blocks, 256, 0, st>>>(src, dst, perm_row, T, k, vec_per_row);
    else scatter_rows_kernel<<<blocks, 256, 0, st>>>(src, dst, perm_row, T, k, vec_per_row);
}
inline void launch_combine_rows(const uint4* Yp, const int32_t* perm_row, uint4* Y, int T, int k, int vec_per_row,
                                int sm_count, cudaStream_t st) {
    const int blocks = min(ceil_div(T, 8), sm_count * 8);
    if (blocks <= 0) return;
    // short rows (d < 4096) keep the chunked kernel: measured faster there (more warps per SM)
    if (vec_per_row >= 32 * 16 && vec_per_row % (32 * 7) == 0)
        combine_rows_seg_kernel<7><<<blocks, 256, 0, st>>>(Yp, perm_row, Y, T, k, vec_per_row);
    else if (vec_per_row >= 32 * 16) combine_rows_seg_kernel<8><<<blocks, 256, 0, st>>>(Yp, perm_row, Y, T, k, vec_per_row);
    else combine_rows_kernel<<<blocks, 256, 0, st>>>(Yp, perm_row, Y, T, k, vec_per_row);
}

// dgate[a] = sum over n-tiles of the partial dot products written by the dgrad-down epilogue
// (row p = perm_row[a]; fixed order, so the result is reproducible).
__global__ void dgate_reduce_kernel(const float* __restrict__ part, const int32_t* __restrict__ perm_row,
                                    float* __restrict__ dgate, int M, int ntiles) {
    const int a = blockIdx.x * blockDim.x + threadIdx.x;
    if (a >= M) return;
    const int32_t p = perm_row[a];
    float s = 0.0f;
    if (p >= 0)
        for (int n = 0; n < ntiles; ++n) s += part[(size_t)n * M + p];
    dgate[a] = s;
}

// ---------------------------------------------------------------------------------------------
// Expert-chunked layer (only a fraction of the expert-contiguous buffers is live at a time).
// Chunk i of C takes the experts [eb(i), eb(i+1)) where eb(i) is the first expert whose first row is
// at or past ceil(i M / C): C chunks of at most ceil(M / C) + (rows of one expert) rows each.
// ---------------------------------------------------------------------------------------------

// Tables of one chunk: off_c[e] = first row of expert e inside the chunk's buffers (experts outside the
// chunk get no rows), row_src_c[r] = assignment of chunk row r, perm_c[a] = chunk row of assignment a or -1.
// bounds[0] = first row of the chunk in the whole layer, bounds[1] = its rows.
__global__ void __launch_bounds__(256) chunk_tables_kernel(const int32_t* __restrict__ offsets,
                                                           const int32_t* __restrict__ row_src,
                                                           const int32_t* __restrict__ perm_row,
                                                           int32_t* __restrict__ off_c, int32_t* __restrict__ row_src_c,
                                                           int32_t* __restrict__ perm_c, int32_t* __restrict__ bounds,
                                                           int E, int M, int chunk, int n_chunks) {
    __shared__ int32_t s_lo, s_hi;
    if (threadIdx.x == 0) {
        const long long t0 = ((long long)chunk * M + n_chunks - 1) / n_chunks;
        const long long t1 = ((long long)(chunk + 1) * M + n_chunks - 1) / n_chunks;
        int e0 = 0, e1 = 0;
        while (e0 < E && offsets[e0] < t0) ++e0;          // E <= 1024: a short serial search
        e1 = e0;
        if (chunk + 1 == n_chunks) e1 = E;
        else while (e1 < E && offsets[e1] < t1) ++e1;
        s_lo = offsets[e0];
        s_hi = offsets[e1];
    }
    __syncthreads();
    const int lo = s_lo, hi = s_hi;
    const int gtid = blockIdx.x * blockDim.x + threadIdx.x, gsz = gridDim.x * blockDim.x;
    if (gtid == 0) { bounds[0] = lo; bounds[1] = hi - lo; }
    for (int e = gtid; e <= E; e += gsz) off_c[e] = min(max(offsets[e], lo), hi) - lo;
    for (int r = gtid; r < hi - lo; r += gsz) row_src_c[r] = row_src[lo + r];
    for (int a = gtid; a < M; a += gsz) {
        const int32_t p = perm_row[a];
        perm_c[a] = (p >= lo && p < hi) ? p - lo : -1;
    }
}

// Xp_c[r,:] = x[row_src_c[r] / k, :] for the rows of a chunk (one warp per row, 16-byte vectors).
__global__ void __launch_bounds__(256) gather_rows_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst,
                                                          const int32_t* __restrict__ row_src_c,
                                                          const int32_t* __restrict__ bounds, int k, int vec_per_row) {
    const int rows = bounds[1];
    const int lane = threadIdx.x % 32, wpb = blockDim.x / 32;
    for (int r = blockIdx.x * wpb + threadIdx.x / 32; r < rows; r += gridDim.x * wpb) {
        const uint4* s = src + (size_t)(row_src_c[r] / k) * vec_per_row;
        uint4* o = dst + (size_t)r * vec_per_row;
        for (int c = lane; c < vec_per_row; c += 32) __stcs(o + c, __ldg(s + c));
    }
}

// Accumulating combine: acc[t,:] (+)= sum_j Yp_c[perm_c[t*k+j], :] over the token's rows inside the chunk
// (fp32, j ascending; chunks are added in chunk order, so the result is reproducible).  first: acc is
// written, not read; last: the sum is rounded once to bf16 into out instead of going back to acc.
__global__ void __launch_bounds__(256) combine_acc_kernel(const uint4* __restrict__ Yp_c,
                                                          const int32_t* __restrict__ perm_c, float4* __restrict__ acc,
                                                          uint4* __restrict__ out, int T, int k, int vec_per_row,
                                                          int first, int last) {
    const int wpb = blockDim.x / 32, lane = threadIdx.x % 32;
    for (int t = blockIdx.x * wpb + threadIdx.x / 32; t < T; t += gridDim.x * wpb) {
        int32_t myrow = -1;
        if (lane < k) myrow = perm_c[(size_t)t * k + lane];
        const bool any = __any_sync(0xffffffffu, myrow >= 0);
        if (!any && !first && !last) continue;              // nothing of this token in the chunk
        for (int c = lane; c < vec_per_row; c += 32) {
            float a[8];
            float4* ap = acc + ((size_t)t * vec_per_row + c) * 2;
            if (first) {
#pragma unroll
                for (int i = 0; i < 8; ++i) a[i] = 0.0f;
            } else {
                const float4 a0 = ap[0], a1 = ap[1];
                a[0] = a0.x; a[1] = a0.y; a[2] = a0.z; a[3] = a0.w; a[4] = a1.x; a[5] = a1.y; a[6] = a1.z; a[7] = a1.w;
            }
            for (int j = 0; j < k; ++j) {
                const int32_t p = __shfl_sync(0xffffffffu, myrow, j);
                if (p < 0) continue;
                const uint4 v = __ldcs(Yp_c + (size_t)p * vec_per_row + c);
                a[0] += bf16_lo(v.x); a[1] += bf16_hi(v.x); a[2] += bf16_lo(v.y); a[3] += bf16_hi(v.y);
                a[4] += bf16_lo(v.z); a[5] += bf16_hi(v.z); a[6] += bf16_lo(v.w); a[7] += bf16_hi(v.w);
            }
            if (last) {
                uint4 o;
                o.x = pack_bf16x2(a[0], a[1]); o.y = pack_bf16x2(a[2], a[3]);
                o.z = pack_bf16x2(a[4], a[5]); o.w = pack_bf16x2(a[6], a[7]);
                out[(size_t)t * vec_per_row + c] = o;
            } else {
                ap[0] = make_float4(a[0], a[1], a[2], a[3]);
                ap[1] = make_float4(a[4], a[5], a[6], a[7]);
            }
        }
    }
}

// dgate of the assignments that lie inside the chunk (others are left alone).
__global__ void dgate_reduce_chunk_kernel(const float* __restrict__ part, const int32_t* __restrict__ perm_c,
                                          float* __restrict__ dgate, int M, int rows_pitch, int ntiles) {
    const int a = blockIdx.x * blockDim.x + threadIdx.x;
    if (a >= M) return;
    const int32_t p = perm_c[a];
    if (p < 0) return;
    float s = 0.0f;
    for (int n = 0; n < ntiles; ++n) s += part[(size_t)n * rows_pitch + p];
    dgate[a] = s;
}

// Zero the weight gradients of the experts that received no row (the chunked backward writes only experts with rows).
__global__ void __launch_bounds__(256) zero_empty_experts_kernel(const int32_t* __restrict__ offsets,
                                                                float4* __restrict__ dWg, float4* __restrict__ dWu,
                                                                float4* __restrict__ dWd, size_t vec_per_expert) {
    const int e = blockIdx.y;
    if (offsets[e + 1] > offsets[e]) return;
    const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < vec_per_expert; i += (size_t)gridDim.x * blockDim.x) {
        dWg[e * vec_per_expert + i] = z;
        dWu[e * vec_per_expert + i] = z;
        dWd[e * vec_per_expert + i] = z;
    }
}

}  // namespace mop
