// "Tokens on N" two-CTA grouped GEMMs for the forward pass: the MMA computes the TRANSPOSED product
//     D^T [weight rows (M = 256 across the CTA pair) x tokens (N <= 256)] = W^T-tile * Xp^T
// so that the ragged dimension (an expert's token count) sits on the MMA's N, whose granularity is
// 16, instead of on M, whose granularity is 128: an expert with 171 rows costs one N = 176 tile
// instead of two 128-row tiles.  The weights are the "A" operand (each CTA of the pair holds its
// own 128 weight rows), the tokens the "B" operand (each CTA loads half of the tile's token rows),
// tcgen05.mma.cta_group::2 multiplies, and each CTA's TMEM receives [its 128 weight rows x N].
//
//   TN_F1  G^T|U^T: a CTA's 128 weight rows are 64 gate columns followed by the 64 matching up
//          columns of W_gate / W_up, so G and U of one (f, token) land in the same CTA (TMEM lanes
//          l and l + 64); the epilogue exchanges U through shared memory, applies SwiGLU and
//          writes H (+ G, U stash) back in token-major layout.
//   TN_F2  O^T = W_down^T-tile * H^T, gate applied per token column, Yp written token-major.
//   TN_F1G as TN_F1, but the token operand is gathered straight from the unpermuted x [T, d]: every
//          lane of the producer warp owns four token rows of the tile and fetches them per K block
//          with one TMA gather4 copy, so the expert-contiguous copy Xp never exists (the
//          single-GPU form of keeping only a fraction of the routed inputs live, Section 3.3).
//          The TMA unit retires these 4-row copies far more slowly than one 128-row box (about
//          60 ns each on B200), so this form trades time for memory and is opt-in.
//   TN_B4  dXp^T = W_gate[e] dG^T + W_up[e] dU^T: the weights are read K-major ([E, d, f] as it
//          lies in memory, rows of d on M), two K phases into one accumulator, dXp token-major.
//   TN_B2  dHu^T = W_down[e] dYp^T (weights K-major, rows of f on M); the epilogue turns each
//          32 x 32 block token-major through shared memory and then runs the SwiGLU backward on
//          16-byte runs of the stash: dG, dU, gate*H out, and one dgate partial per 32 columns of f.
//
// The epilogue transposes 32 x 32 blocks through shared memory so that global stores are 64-byte
// row segments.  Barrier protocol, bounded waits and teardown as in the pair kernel.
#pragma once
#include "gemm_tc2.cuh"

namespace mop {

enum : int { TN_F1 = 0, TN_F2 = 1, TN_F1G = 2, TN_B4 = 3, TN_B2 = 4 };

constexpr int TN_STAGES = 3;
constexpr int TN_BK = 128;                           // K per pipeline stage: two 64-wide swizzle spans
constexpr int TN_SUB_BYTES = 128 * 64 * 2;           // 16 KiB: 128 rows x 64 K (or one 64-wide MN chunk x 128 K)
constexpr int TN_A_BYTES = 2 * TN_SUB_BYTES;         // 32 KiB: this CTA's 128 weight rows x 128 K
constexpr int TN_B_BYTES = 2 * TN_SUB_BYTES;         // up to 128 token rows (half of N = 256) x 128 K
constexpr int TN_STAGE_BYTES = TN_A_BYTES + TN_B_BYTES;
constexpr int TN_EPI_BYTES = 4 * 8192;               // per epilogue warp: transposition buffers
constexpr int TN_SMEM_BYTES = TN_STAGES * TN_STAGE_BYTES + 1024 /*align*/ + TC_BAR_BYTES + TN_EPI_BYTES;
constexpr int TN_THREADS = 192;
constexpr int TN_BOX_ROWS = 128;                     // token rows per TMA box (one box per stage)

struct TnArgs {
    const int4* ttiles;       // {expert, first row, rows (1..256), 0} per token tile
    const int32_t* n_ttiles;  // device scalar
    int tiles_m;              // weight-row tiles per token tile (each 256 rows; F1: 128 columns of f)
    int kblocks;              // K / 128 rounded up
    int Mw;                   // weight rows in total (F1: f; F2: d)
    const int32_t* row_src;   // F1G: assignment index t*k + j of every expert-contiguous row
    int topk;                 // F1G: k (token of a row = row_src / k)
    int32_t* status;
    EpiArgs ep;
};

// Token tiles: an expert's rows are cut into ceil(rows/256) nearly equal tiles.
__device__ __forceinline__ void tn_build_ttiles_body(const int32_t* __restrict__ offsets, int E,
                                                     int4* __restrict__ tiles, int32_t* __restrict__ n_tiles,
                                                     int32_t* scan) {
    const int e = threadIdx.x;
    int cnt = 0, off = 0;
    if (e < E) { off = offsets[e]; cnt = offsets[e + 1] - off; }
    const int nt = (cnt + 255) / 256;
    scan[e] = nt;
    __syncthreads();
    for (int s = 1; s < 1024; s <<= 1) {
        const int v = (e >= s) ? scan[e - s] : 0;
        __syncthreads();
        scan[e] += v;
        __syncthreads();
    }
    const int first = scan[e] - nt;
    const int sz = nt ? (((cnt + nt - 1) / nt + 15) & ~15) : 0;
    // .w = position of the tile within its expert | number of tiles of the expert << 16
    for (int i = 0; i < nt; ++i) tiles[first + i] = make_int4(e, off + i * sz, min(sz, cnt - i * sz), i | (nt << 16));
    if (e == 1023) *n_tiles = scan[1023];
}
__global__ void __launch_bounds__(1024) tn_build_ttiles_kernel(const int32_t* __restrict__ offsets, int E,
                                                               int4* __restrict__ tiles,
                                                               int32_t* __restrict__ n_tiles) {
    __shared__ int32_t scan[1025];
    tn_build_ttiles_body(offsets, E, tiles, n_tiles, scan);
}
// Both tables in one launch (block 0: 128-row tiles of the tokens-on-M kernels, block 1: token tiles).
__global__ void __launch_bounds__(1024) build_both_tiles_kernel(const int32_t* __restrict__ offsets, int E,
                                                                int4* __restrict__ mtiles, int32_t* __restrict__ n_mtiles,
                                                                int4* __restrict__ ttiles, int32_t* __restrict__ n_ttiles) {
    __shared__ int32_t scan[1025];
    if (blockIdx.x == 0) tc_build_mtiles_body(offsets, E, mtiles, n_mtiles, scan);
    else tn_build_ttiles_body(offsets, E, ttiles, n_ttiles, scan);
}

// Four rows of a [rows, cols] bf16 tensor (map box {64, 1}) -> 4 x 128 bytes at dst, swizzled like a tile box.
__device__ __forceinline__ void tma2_gather4(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int r0, int r1,
                                             int r2, int r3) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cta.global.tile::gather4.mbarrier::complete_tx::bytes.cta_group::2 [%0], "
        "[%1, {%3, %4, %5, %6, %7}], [%2];" ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(r0), "r"(r1), "r"(r2), "r"(r3)
        : "memory");
}

__device__ __forceinline__ void bar_pair_sync(int id) { asm volatile("bar.sync %0, 64;" ::"r"(id) : "memory"); }

// 32 tokens x 32 features staged as bf16 [token][feature] -> 64-byte row segments in global memory
__device__ __forceinline__ void tn_write_rows(bf16* __restrict__ dst, int ldo, const uint16_t* st, int row0,
                                              int rows_left, int col0, int lane) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int tok = 8 * i + (lane >> 2), part = lane & 3;
        const uint4 v = *reinterpret_cast<const uint4*>(st + tok * 32 + part * 8);
        if (tok < rows_left) *reinterpret_cast<uint4*>(dst + (size_t)(row0 + tok) * ldo + col0 + part * 8) = v;
    }
}

__device__ __forceinline__ uint16_t bf16_bits(float v) {
    return __bfloat16_as_ushort(__float2bfloat16_rn(v));
}

template <int KIND>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(TN_THREADS, 1)
tn_gemm_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmA1,
               const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmB1, const TnArgs args) {
    constexpr int S = TN_STAGES;
    extern __shared__ uint8_t tc_smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S * TN_STAGE_BYTES);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * S + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    uint8_t* epi_smem = smem + S * TN_STAGE_BYTES + TC_BAR_BYTES;

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const uint32_t rank = cluster_ctarank();
    const bool leader = rank == 0;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bar_base = smem_u32(bars);
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (S + s); };
    auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * S + b); };
    auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * S + 2 + b); };

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 8); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tma_prefetch_desc(&tmA0); tma_prefetch_desc(&tmB);
        if (KIND != TN_F2) tma_prefetch_desc(&tmA1);
        if (KIND == TN_B4) tma_prefetch_desc(&tmB1);
    }
    if (warp == 1) tmem2_alloc(smem_u32(tmem_slot), 512);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int total_tiles = (*args.n_ttiles) * args.tiles_m;
    const int nkb = (KIND == TN_B4 ? 2 : 1) * args.kblocks;   // K blocks per tile (B4: two phases)
    const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
    // work tile t -> token tile t / tiles_m (its expert, first row, rows) and weight-row tile t % tiles_m
    struct Tile { int e, row0, rows, nmma, mt; };
    // Within an expert the token tiles vary fastest: the clusters that run at the same time on
    // neighbouring work tiles then share one weight tile (the large operand) through L2.
    auto decode = [&](int t) {
        const int q = t / args.tiles_m;
        int4 m = __ldg(args.ttiles + q);
        const int nt = m.w >> 16;
        Tile ti;
        ti.mt = t % args.tiles_m;
        if (nt > 1) {
            const int first = q - (m.w & 0xffff);                 // first token tile of this expert
            const int l = t - first * args.tiles_m;               // position among the expert's work tiles
            ti.mt = l / nt;
            m = __ldg(args.ttiles + first + l % nt);
        }
        ti.e = m.x; ti.row0 = m.y; ti.rows = m.z; ti.nmma = (m.z + 15) & ~15;
        return ti;
    };

    if (warp == 0 && KIND == TN_F1G) {
        // ============================================ TMA producer with row gather (both CTAs, whole warp)
        int stage = 0; uint32_t phase = 0; bool alive = true;
        Tile nxt = decode(min(cluster_id, max(total_tiles - 1, 0)));
        for (int t = cluster_id; t < total_tiles && alive; t += n_clusters) {
            const Tile ti = nxt;
            if (t + n_clusters < total_tiles) nxt = decode(t + n_clusters);
            const int half = ti.nmma >> 1;                             // token rows per CTA (multiple of 8)
            const int ngroups = half >> 2;                             // gather4 copies per K block (<= 32)
            const int brow0 = ti.row0 + (int)rank * half;
            const int last = ti.row0 + ti.rows - 1;                    // padding rows repeat the last valid one
            int tok[4] = {0, 0, 0, 0};
            if (lane < ngroups) {
#pragma unroll
                for (int j = 0; j < 4; ++j) tok[j] = __ldg(args.row_src + min(brow0 + 4 * lane + j, last)) / args.topk;
            }
            const uint32_t tx = 2u * (TN_A_BYTES + 2u * (uint32_t)half * 128u);
            for (int kb = 0; kb < args.kblocks; ++kb) {
                if (!mbar_wait_warp(empty_bar(stage), phase ^ 1u, abort_flag, args.status, STATUS_WAIT_EMPTY, lane)) {
                    alive = false; break;
                }
                const uint32_t fb = full_bar(stage) & T2_PEER_MASK;
                const uint32_t sA = smem_base + stage * TN_STAGE_BYTES;
                const uint32_t sB = sA + TN_A_BYTES;
                const int k0 = kb * TN_BK;
                if (lane == 0) {
                    if (leader) mbar_expect_tx(full_bar(stage), tx);
                    const int f0 = ti.mt * 128 + 64 * (int)rank;
                    tma2_load_4d(sA, &tmA0, fb, 0, k0, f0 >> 6, ti.e);
                    tma2_load_4d(sA + TN_SUB_BYTES, &tmA1, fb, 0, k0, f0 >> 6, ti.e);
                }
                if (lane < ngroups) {
                    tma2_gather4(sB + lane * 512, &tmB, fb, k0, tok[0], tok[1], tok[2], tok[3]);
                    tma2_gather4(sB + TN_SUB_BYTES + lane * 512, &tmB, fb, k0 + 64, tok[0], tok[1], tok[2], tok[3]);
                }
                __syncwarp();
                if (++stage == S) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 0) {
        // ===================================================================== TMA producer (both CTAs)
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0; bool alive = true;
            const uint64_t pol_w = l2_policy_evict_last();
            Tile nxt = decode(min(cluster_id, max(total_tiles - 1, 0)));
            for (int t = cluster_id; t < total_tiles && alive; t += n_clusters) {
                const Tile ti = nxt;
                if (t + n_clusters < total_tiles) nxt = decode(t + n_clusters);
                const int half = ti.nmma >> 1;                         // token rows per CTA
                const int nbox = (half + TN_BOX_ROWS - 1) / TN_BOX_ROWS;
                const int brow0 = ti.row0 + (int)rank * half;
                const uint32_t tx = 2u * (TN_A_BYTES + 2u * (uint32_t)nbox * TN_BOX_ROWS * 128u);
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, args.status, STATUS_WAIT_EMPTY)) {
                        alive = false; break;
                    }
                    const uint32_t fb = full_bar(stage) & T2_PEER_MASK;
                    if (leader) mbar_expect_tx(full_bar(stage), tx);
                    const uint32_t sA = smem_base + stage * TN_STAGE_BYTES;
                    const uint32_t sB = sA + TN_A_BYTES;
                    const int ph = (KIND == TN_B4 && kb >= args.kblocks) ? 1 : 0;   // B4: gate phase, then up phase
                    const int k0 = (kb - ph * args.kblocks) * TN_BK;
                    if constexpr (KIND == TN_B4 || KIND == TN_B2) {
                        // K-major weights: this CTA's 128 weight rows, two boxes of 64 columns of K
                        const int m0 = ti.mt * 256 + 128 * (int)rank;
                        tma2_load_3d(sA, ph ? &tmA1 : &tmA0, fb, k0, m0, ti.e);
                        tma2_load_3d(sA + TN_SUB_BYTES, ph ? &tmA1 : &tmA0, fb, k0 + 64, m0, ti.e);
                        tma2_load_2d(sB, ph ? &tmB1 : &tmB, fb, k0, brow0);
                        tma2_load_2d(sB + TN_SUB_BYTES, ph ? &tmB1 : &tmB, fb, k0 + 64, brow0);
                        if (++stage == S) { stage = 0; phase ^= 1u; }
                        continue;
                    }
                    if constexpr (KIND != TN_F2) {
                        // 64 gate columns, then the 64 matching up columns (N-major weights [E, d, f])
                        const int f0 = ti.mt * 128 + 64 * (int)rank;
                        tma2_load_4d_hint(sA, &tmA0, fb, 0, k0, f0 >> 6, ti.e, pol_w);
                        tma2_load_4d_hint(sA + TN_SUB_BYTES, &tmA1, fb, 0, k0, f0 >> 6, ti.e, pol_w);
                    } else {
                        const int m0 = ti.mt * 256 + 128 * (int)rank;
                        tma2_load_4d_hint(sA, &tmA0, fb, 0, k0, m0 >> 6, ti.e, pol_w);   // two chunks in one copy
                    }
                    tma2_load_2d(sB, &tmB, fb, k0, brow0);
                    tma2_load_2d(sB + TN_SUB_BYTES, &tmB, fb, k0 + 64, brow0);
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ===================================================================== MMA issuer (leader CTA)
        // One thread runs the whole loop (wait, fence, four MMAs, commit): per K block nothing but
        // these instructions stands between two groups of MMAs, so the tensor pipe's queue stays fed.
        if (leader && lane == 0) {
            constexpr bool A_KMAJOR = (KIND == TN_B4 || KIND == TN_B2);
            // descriptors without the start address: A is M-major (N-major weights) or K-major, B is K-major
            // A M-major: the two 64-wide chunks are TN_SUB_BYTES apart and hold 128 K rows each (2 KiB per
            // K = 16); K-major operands: two 64-K sub-tiles TN_SUB_BYTES apart, 32 bytes per K = 16 inside one
            const uint64_t desc_a = smem_desc(0, A_KMAJOR ? 0 : TN_SUB_BYTES, 1024);
            const uint64_t desc_b = smem_desc(0, 0, 1024);
            int stage = 0; uint32_t phase = 0; int it = 0; bool alive = true;
            Tile nxt = decode(min(cluster_id, max(total_tiles - 1, 0)));
            for (int t = cluster_id; t < total_tiles && alive; t += n_clusters) {
                const Tile ti = nxt;
                if (t + n_clusters < total_tiles) nxt = decode(t + n_clusters);
                // M = 256 over the pair, N = this tile's tokens
                const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((A_KMAJOR ? 0u : 1u) << 15) |
                                       ((uint32_t)(ti.nmma >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
                const int buf = it & 1;
                const uint32_t tphase = (uint32_t)(it >> 1) & 1u;
                if (!mbar_wait(tempty_bar(buf), tphase ^ 1u, abort_flag, args.status, STATUS_WAIT_TMEM_EMPTY)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)buf * 256;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag, args.status, STATUS_WAIT_FULL)) {
                        alive = false; break;
                    }
                    tc_fence_after();
                    const uint32_t sA = smem_base + stage * TN_STAGE_BYTES;
                    const uint64_t da = desc_a | (uint64_t)((sA & 0x3ffffu) >> 4);
                    const uint64_t db = desc_b | (uint64_t)(((sA + TN_A_BYTES) & 0x3ffffu) >> 4);
#pragma unroll
                    for (int k8 = 0; k8 < TN_BK / 16; ++k8) {
                        const uint32_t kmaj = (uint32_t)((k8 >> 2) * (TN_SUB_BYTES >> 4) + (k8 & 3) * 2);
                        umma2_bf16(d_tmem, da + (A_KMAJOR ? kmaj : (uint32_t)(k8 * (2048 >> 4))), db + kmaj, idesc,
                                   (kb | k8) != 0 ? 1u : 0u);
                    }
                    umma2_commit_both(empty_bar(stage));
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
                if (!alive) break;
                umma2_commit_both(tfull_bar(buf));
                ++it;
            }
        }
    } else {
        // ===================================================================== epilogue (4 warps, both CTAs)
        const int quarter = warp & 3;                 // TMEM lanes 32*quarter .. +31
        uint8_t* wbuf = epi_smem + quarter * 8192;    // this warp's staging
        int it = 0;
        Tile nxt = decode(min(cluster_id, max(total_tiles - 1, 0)));
        for (int t = cluster_id; t < total_tiles; t += n_clusters) {
            const Tile ti = nxt;
            if (t + n_clusters < total_tiles) nxt = decode(t + n_clusters);
            const int buf = it & 1;
            const uint32_t tphase = (uint32_t)(it >> 1) & 1u;
            // F2: the gates of the tile's tokens (two dependent loads each) are fetched before the wait for the
            // accumulator, so that their latency is hidden behind the main loop instead of paid per 32 tokens
            float gpre[8];
            if constexpr (KIND == TN_F2) {
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int tk = 32 * j + lane;
                    gpre[j] = tk < ti.rows ? args.ep.gate[args.ep.row_src[ti.row0 + tk]] : 0.0f;
                }
            }
            bool ready = mbar_wait_warp(tfull_bar(buf), tphase, abort_flag, args.status, STATUS_WAIT_TMEM_FULL, lane);
            // the gate warp and its up warp meet at a named barrier below: they give up together or not at all
            if constexpr (KIND == TN_F1 || KIND == TN_F1G) ready = bar_vote_all(1 + (quarter & 1), 64, ready);
            if (!ready) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)buf * 256;
            float v[32];

            if constexpr (KIND == TN_F1 || KIND == TN_F1G) {
                // Lanes 0..63 of the CTA hold gate rows, lanes 64..127 the matching up rows: warp q (gate)
                // and warp q + 2 (up) own the same 32 f columns.  Per chunk of 32 tokens they swap halves
                // through shared memory (the gate warp hands over G of tokens 16..31, the up warp U of
                // tokens 0..15), so each evaluates SwiGLU for 16 tokens and writes 16 rows of H.
                const bool is_up = quarter >= 2;
                const int fcol = ti.mt * 128 + 64 * (int)rank + 32 * (quarter & 1);   // first f of this warp
                const bool f_ok = fcol < args.Mw;
                float* my_x = reinterpret_cast<float*>(wbuf);                                  // 16 x 33 fp32
                const float* peer_x = reinterpret_cast<const float*>(epi_smem + (quarter ^ 2) * 8192);
                uint16_t* hb = reinterpret_cast<uint16_t*>(wbuf + 2176);                       // 16 x 32 bf16: H
                uint16_t* sb = reinterpret_cast<uint16_t*>(wbuf + 3200);                       // 32 x 32 bf16: stash
                bf16* stash_out = is_up ? args.ep.out2 : args.ep.out1;
                const int t_own = is_up ? 16 : 0;
                const int pair_bar = 1 + (quarter & 1);
#pragma unroll 1
                for (int c = 0; c < ti.nmma; c += 32) {
                    tmem_ld32(taddr + c, v);
                    const int rows_left = ti.rows - c;
#pragma unroll
                    for (int i = 0; i < 16; ++i) my_x[i * 33 + lane] = is_up ? v[i] : v[16 + i];
                    if (stash_out) {
#pragma unroll
                        for (int tk = 0; tk < 32; ++tk) sb[tk * 32 + lane] = bf16_bits(v[tk]);
                    }
                    bar_pair_sync(pair_bar);     // both halves are in shared memory
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float other = peer_x[i * 33 + lane];
                        const float mine = is_up ? v[16 + i] : v[i];
                        const float g = is_up ? other : mine, u = is_up ? mine : other;
                        hb[i * 32 + lane] = bf16_bits(g * sigmoidf_fast(g) * u);
                    }
                    __syncwarp();
                    if (f_ok) {
#pragma unroll
                        for (int i = 0; i < 2; ++i) {     // 16 tokens x 32 features of H: 64-byte row segments
                            const int tok = 8 * i + (lane >> 2), part = lane & 3;
                            const uint4 hv = *reinterpret_cast<const uint4*>(hb + tok * 32 + part * 8);
                            if (t_own + tok < rows_left)
                                *reinterpret_cast<uint4*>(args.ep.out0 + (size_t)(ti.row0 + c + t_own + tok) * args.ep.ldo +
                                                          fcol + part * 8) = hv;
                        }
                        if (stash_out) tn_write_rows(stash_out, args.ep.ldo, sb, ti.row0 + c, rows_left, fcol, lane);
                    }
                    bar_pair_sync(pair_bar);     // the partner has read this warp's half
                }
            } else if constexpr (KIND == TN_B2) {
                const int fcol = ti.mt * 256 + 128 * (int)rank + 32 * quarter;      // first f column of this warp
                const bool f_ok = fcol < args.Mw;
                float* fbuf = reinterpret_cast<float*>(wbuf);                       // 32 tokens x 33 fp32
                const int part = lane & 3;
#pragma unroll 1
                for (int c = 0; c < ti.nmma; c += 32) {
                    const int rows_left = ti.rows - c;
                    // the stash (G, U, H: 16 bytes each per lane and sub-block) is requested first, so that its
                    // latency overlaps the TMEM read and the transposition below
                    uint4 gq[4], uq[4], hq[4];
                    float gate[4];
                    bool ok[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int tok = 8 * i + (lane >> 2);
                        ok[i] = f_ok && tok < rows_left;
                        gate[i] = 0.0f;
                        if (ok[i]) {
                            const int row = ti.row0 + c + tok;
                            const size_t o = (size_t)row * args.ep.ldo + fcol + part * 8;
                            gq[i] = *reinterpret_cast<const uint4*>(args.ep.in0 + o);
                            uq[i] = *reinterpret_cast<const uint4*>(args.ep.in1 + o);
                            hq[i] = *reinterpret_cast<const uint4*>(args.ep.in2 + o);
                            gate[i] = args.ep.gate[args.ep.row_src[row]];
                        }
                    }
                    tmem_ld32(taddr + c, v);
#pragma unroll
                    for (int tk = 0; tk < 32; ++tk) fbuf[tk * 33 + lane] = v[tk];
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int tok = 8 * i + (lane >> 2);
                        float dot = 0.0f;
                        if (ok[i]) {
                            const uint32_t gw[4] = {gq[i].x, gq[i].y, gq[i].z, gq[i].w};
                            const uint32_t uw[4] = {uq[i].x, uq[i].y, uq[i].z, uq[i].w};
                            const uint32_t hw[4] = {hq[i].x, hq[i].y, hq[i].z, hq[i].w};
                            float dG[8], dU[8], gH[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const float G = (j & 1) ? bf16_hi(gw[j >> 1]) : bf16_lo(gw[j >> 1]);
                                const float U = (j & 1) ? bf16_hi(uw[j >> 1]) : bf16_lo(uw[j >> 1]);
                                const float H = (j & 1) ? bf16_hi(hw[j >> 1]) : bf16_lo(hw[j >> 1]);
                                const float dhu = fbuf[tok * 33 + part * 8 + j];
                                dot = fmaf(dhu, H, dot);
                                const float dh = gate[i] * dhu;
                                const float sg = sigmoidf_fast(G);
                                dG[j] = dh * U * sg * (1.0f + G * (1.0f - sg));
                                dU[j] = dh * (G * sg);
                                gH[j] = gate[i] * H;
                            }
                            const size_t o = (size_t)(ti.row0 + c + tok) * args.ep.ldo + fcol + part * 8;
                            store_bf16_run<8>(args.ep.out0 + o, dG);
                            store_bf16_run<8>(args.ep.out1 + o, dU);
                            store_bf16_run<8>(args.ep.out2 + o, gH);
                        }
                        dot += __shfl_xor_sync(0xffffffffu, dot, 1);
                        dot += __shfl_xor_sync(0xffffffffu, dot, 2);
                        if (ok[i] && part == 0)
                            args.ep.part[(size_t)(fcol >> 5) * args.ep.M_total + ti.row0 + c + tok] = dot;
                    }
                    __syncwarp();
                }
            } else {
                const int mcol = ti.mt * 256 + 128 * (int)rank + 32 * quarter;      // first output column of this warp
                const bool m_ok = mcol < args.Mw;
                uint16_t* st0 = reinterpret_cast<uint16_t*>(wbuf);
#pragma unroll
                for (int j8 = 0; j8 < 8; ++j8) {
                    const int c = 32 * j8;
                    if (c >= ti.nmma) break;
                    tmem_ld32(taddr + c, v);
                    const int rows_left = ti.rows - c;
                    // gate of token (c + lane), handed round by shuffle
                    const float gmine = (KIND == TN_F2) ? gpre[j8] : 1.0f;
#pragma unroll
                    for (int tk = 0; tk < 32; ++tk) {
                        const float g = __shfl_sync(0xffffffffu, gmine, tk);
                        st0[tk * 32 + lane] = bf16_bits(g * v[tk]);
                    }
                    __syncwarp();
                    if (m_ok) tn_write_rows(args.ep.out0, args.ep.ldo, st0, ti.row0 + c, rows_left, mcol, lane);
                    __syncwarp();
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(tempty_bar(buf) & T2_PEER_MASK);
            ++it;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) __nanosleep(1000);
        __syncthreads();
    }
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem2_dealloc(tmem_base, 512);
    }
}

// ------------------------------------------------------------------------------------------ host
inline mop_status tn_init() {
    if (cudaFuncSetAttribute(tn_gemm_kernel<TN_F1>, cudaFuncAttributeMaxDynamicSharedMemorySize, TN_SMEM_BYTES) !=
            cudaSuccess ||
        cudaFuncSetAttribute(tn_gemm_kernel<TN_F2>, cudaFuncAttributeMaxDynamicSharedMemorySize, TN_SMEM_BYTES) !=
            cudaSuccess ||
        cudaFuncSetAttribute(tn_gemm_kernel<TN_F1G>, cudaFuncAttributeMaxDynamicSharedMemorySize, TN_SMEM_BYTES) !=
            cudaSuccess ||
        cudaFuncSetAttribute(tn_gemm_kernel<TN_B4>, cudaFuncAttributeMaxDynamicSharedMemorySize, TN_SMEM_BYTES) !=
            cudaSuccess ||
        cudaFuncSetAttribute(tn_gemm_kernel<TN_B2>, cudaFuncAttributeMaxDynamicSharedMemorySize, TN_SMEM_BYTES) !=
            cudaSuccess)
        return MOP_ERR_CUDA;
    return MOP_OK;
}

inline mop_status build_both_tiles(TcPlan* p, const int32_t* offsets, int32_t* mtiles, int32_t* ttiles, cudaStream_t st) {
    p->prof->begin("build_tiles", st);
    build_both_tiles_kernel<<<2, 1024, 0, st>>>(offsets, p->s.E, reinterpret_cast<int4*>(mtiles + 64), mtiles,
                                                reinterpret_cast<int4*>(ttiles + 64), ttiles);
    p->prof->end(st);
    return cudaGetLastError() == cudaSuccess ? MOP_OK : MOP_ERR_CUDA;
}
inline mop_status tn_build_tiles(TcPlan* p, const int32_t* offsets, int32_t* tiles, cudaStream_t st) {
    p->prof->begin("tn_build_ttiles", st);
    tn_build_ttiles_kernel<<<1, 1024, 0, st>>>(offsets, p->s.E, reinterpret_cast<int4*>(tiles + 64), tiles);
    p->prof->end(st);
    return cudaGetLastError() == cudaSuccess ? MOP_OK : MOP_ERR_CUDA;
}

inline TnArgs tn_base_args(int32_t* tiles, int32_t* status) {
    TnArgs g{};
    g.ttiles = reinterpret_cast<const int4*>(tiles + 64);
    g.n_ttiles = tiles;
    g.status = status;
    return g;
}

// Up-projection + SwiGLU on the tokens-on-N kernel (`tiles` holds the token-tile table).
inline mop_status tn_up_swiglu(TcPlan* p, const TcFwdArgs& a, int32_t* tiles, int32_t* status, cudaStream_t st) {
    const mop_moe_shape& s = p->s;
    const uint64_t M = tc_rows(p);
    CUtensorMap mXp, mWg, mWu;
    if (!tc_map_2d(p, &mXp, a.Xp, M, s.d, TN_BOX_ROWS) || !tc_map_chunked_3d(p, &mWg, a.W_gate, s.E, s.d, s.f, 1, 128) ||
        !tc_map_chunked_3d(p, &mWu, a.W_up, s.E, s.d, s.f, 1, 128))
        return MOP_ERR_CUDA;
    TnArgs g = tn_base_args(tiles, status);
    g.tiles_m = ceil_div(s.f, 128); g.kblocks = ceil_div(s.d, TN_BK); g.Mw = s.f;
    g.ep.out0 = a.H; g.ep.out1 = a.G_save; g.ep.out2 = a.U_save; g.ep.ldo = s.f; g.ep.M_total = (int)M;
    p->prof->begin("gemm_up_swiglu", st);
    tn_gemm_kernel<TN_F1><<<p->sm_count & ~1, TN_THREADS, TN_SMEM_BYTES, st>>>(mWg, mWu, mXp, mXp, g);
    p->prof->end(st);
    return cudaGetLastError() == cudaSuccess ? MOP_OK : MOP_ERR_CUDA;
}

// Up-projection + SwiGLU reading its token rows straight from the unpermuted x (no Xp, no stash).
inline mop_status tn_up_swiglu_gather(TcPlan* p, const bf16* x, const TcFwdArgs& a, int32_t* tiles, int32_t* status,
                                      cudaStream_t st) {
    const mop_moe_shape& s = p->s;
    CUtensorMap mX, mWg, mWu;
    if (!tc_map_2d(p, &mX, x, s.T, s.d, 1) || !tc_map_chunked_3d(p, &mWg, a.W_gate, s.E, s.d, s.f, 1, 128) ||
        !tc_map_chunked_3d(p, &mWu, a.W_up, s.E, s.d, s.f, 1, 128))
        return MOP_ERR_CUDA;
    TnArgs g = tn_base_args(tiles, status);
    g.tiles_m = ceil_div(s.f, 128); g.kblocks = ceil_div(s.d, TN_BK); g.Mw = s.f;
    g.row_src = a.row_src; g.topk = s.k;
    g.ep.out0 = a.H; g.ep.ldo = s.f; g.ep.M_total = s.T * s.k;
    p->prof->begin("gemm_up_swiglu_gather", st);
    tn_gemm_kernel<TN_F1G><<<p->sm_count & ~1, TN_THREADS, TN_SMEM_BYTES, st>>>(mWg, mWu, mX, mX, g);
    p->prof->end(st);
    return cudaGetLastError() == cudaSuccess ? MOP_OK : MOP_ERR_CUDA;
}

// Down-projection + gate on the tokens-on-N kernel.
inline mop_status tn_down_gate(TcPlan* p, const TcFwdArgs& a, int32_t* tiles, int32_t* status, cudaStream_t st) {
    const mop_moe_shape& s = p->s;
    const uint64_t M = tc_rows(p);
    CUtensorMap mH, mWd;
    if (!tc_map_2d(p, &mH, a.H, M, s.f, TN_BOX_ROWS) || !tc_map_chunked_3d(p, &mWd, a.W_down, s.E, s.f, s.d, 2, 128))
        return MOP_ERR_CUDA;
    TnArgs g = tn_base_args(tiles, status);
    g.tiles_m = ceil_div(s.d, 256); g.kblocks = ceil_div(s.f, TN_BK); g.Mw = s.d;
    g.ep.out0 = a.Yp; g.ep.gate = a.gate; g.ep.row_src = a.row_src; g.ep.ldo = s.d; g.ep.M_total = (int)M;
    p->prof->begin("gemm_down_gate", st);
    tn_gemm_kernel<TN_F2><<<p->sm_count & ~1, TN_THREADS, TN_SMEM_BYTES, st>>>(mWd, mWd, mH, mH, g);
    p->prof->end(st);
    return cudaGetLastError() == cudaSuccess ? MOP_OK : MOP_ERR_CUDA;
}

// Data gradient of the up-projection on the tokens-on-N kernel: dXp = dG W_gate^T + dU W_up^T.
inline mop_status tn_dgrad_gate_up(TcPlan* p, const TcBwdArgs& a, int32_t* tiles, int32_t* status, cudaStream_t st) {
    const mop_moe_shape& s = p->s;
    const uint64_t M = tc_rows(p);
    CUtensorMap mWg, mWu, mdG, mdU;
    if (!tc_map_3d(p, &mWg, a.W_gate, s.E, s.d, s.f, 128) || !tc_map_3d(p, &mWu, a.W_up, s.E, s.d, s.f, 128) ||
        !tc_map_2d(p, &mdG, a.dG, M, s.f, TN_BOX_ROWS) || !tc_map_2d(p, &mdU, a.dU, M, s.f, TN_BOX_ROWS))
        return MOP_ERR_CUDA;
    TnArgs g = tn_base_args(tiles, status);
    g.tiles_m = ceil_div(s.d, 256); g.kblocks = ceil_div(s.f, TN_BK); g.Mw = s.d;
    g.ep.out0 = a.dXp; g.ep.ldo = s.d; g.ep.M_total = (int)M;
    p->prof->begin("gemm_dgrad_gate_up", st);
    tn_gemm_kernel<TN_B4><<<p->sm_count & ~1, TN_THREADS, TN_SMEM_BYTES, st>>>(mWg, mWu, mdG, mdU, g);
    p->prof->end(st);
    return cudaGetLastError() == cudaSuccess ? MOP_OK : MOP_ERR_CUDA;
}

// Data gradient of the down-projection with the SwiGLU backward on the tokens-on-N kernel.
// Writes one dgate partial per 32 columns of f (part[f / 32][row]).
inline mop_status tn_dgrad_down(TcPlan* p, const TcBwdArgs& a, int32_t* tiles, int32_t* status, cudaStream_t st) {
    const mop_moe_shape& s = p->s;
    const uint64_t M = tc_rows(p);
    CUtensorMap mWd, mdYp;
    if (!tc_map_3d(p, &mWd, a.W_down, s.E, s.f, s.d, 128) || !tc_map_2d(p, &mdYp, a.dYp, M, s.d, TN_BOX_ROWS))
        return MOP_ERR_CUDA;
    TnArgs g = tn_base_args(tiles, status);
    g.tiles_m = ceil_div(s.f, 256); g.kblocks = ceil_div(s.d, TN_BK); g.Mw = s.f;
    g.ep.out0 = a.dG; g.ep.out1 = a.dU; g.ep.out2 = a.gH; g.ep.in0 = a.G_save; g.ep.in1 = a.U_save; g.ep.in2 = a.H;
    g.ep.gate = a.gate; g.ep.row_src = a.row_src; g.ep.part = a.part; g.ep.ldo = s.f; g.ep.M_total = (int)M;
    p->prof->begin("gemm_dgrad_down_dswiglu", st);
    tn_gemm_kernel<TN_B2><<<p->sm_count & ~1, TN_THREADS, TN_SMEM_BYTES, st>>>(mWd, mWd, mdYp, mdYp, g);
    p->prof->end(st);
    return cudaGetLastError() == cudaSuccess ? MOP_OK : MOP_ERR_CUDA;
}

}  // namespace mop
