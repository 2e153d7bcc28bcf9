// Router logits on the tensor cores: z~ = x (W_hi + W_mid + W_lo), the three bf16 pieces of the fp32
// router weights W_r (Section 3.1: z = x W_r), as one two-CTA kernel (tcgen05.mma.cta_group::2).
//
// A pair of CTAs computes 256 tokens x up to 256 experts.  What bounds this GEMM on one CTA is the
// L2 -> shared memory traffic (E is small, so a tile of W is as large as a tile of x), hence:
//   * every 64-wide K block of x is fetched ONCE per pair tile (16 KiB per CTA) and multiplied with
//     that block of all three pieces before it is released: x and W travel through separate rings
//     (3 slots of x, 9 slots of W pieces, 16 KiB each), so that about 160 KiB of copies stay in
//     flight while one piece is being multiplied;
//   * each CTA fetches only its half of the experts' columns (the pair MMA reads both halves).
// Per K block a CTA thus receives 16 + 3 x 16 KiB for 3 x 512 tensor-pipe cycles (42 bytes per
// cycle; the one-CTA 128 x 256 tile needed 96).
//
// The K loop is summed in segments of RS_SEG K blocks (192 of K, all pieces): the tensor core
// accumulates a segment into a fresh accumulator (its additions truncate), the eight epilogue warps
// add the finished segment to fp32 registers with round-to-nearest while the next one runs in the
// other accumulator.  Over 36 updates per segment the truncation bias stays below the rounding noise
// of the fp32 reference chain; over the whole of K = 7168 x 3 it would reach 2e-4.
//
// Experts are split into tiles of 256 columns; a last tile of at most 128 columns runs an N = 128
// instruction.  Tiles of one block of tokens are neighbours in the schedule, so x is read from DRAM
// once.  No tile table: rows and columns follow from the tile index.  Waits are bounded as in the
// other tensor-core kernels; no TMA multicast is used.
#pragma once
#include "gemm_tc2.cuh"

namespace mop {

constexpr int RS_SA = 3;                    // slots of x (128 rows x 64 of K per CTA)
constexpr int RS_SB = 9;                    // slots of W pieces (64 of K x up to 128 columns per CTA)
constexpr int RS_SLOT = 16384;
constexpr int RS_SEG = 3;                   // K blocks per accumulation segment
constexpr int RS_EPI_WARPS = 8;
constexpr int RS_THREADS = 64 + 32 * RS_EPI_WARPS;
constexpr int RS_SMEM_BYTES = (RS_SA + RS_SB) * RS_SLOT + 1024 /*align*/ + TC_BAR_BYTES;

struct RsArgs {
    float* z;          // [T, E] fp32 logits (device)
    float* z1;         // splits == 2: the sum over the second half of K goes here (the selection adds the two)
    int splits;        // 1 or 2 halves of the K loop per tile, as separate units of work
    int T, d, E;
    int32_t* status;
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(RS_THREADS, 1)
route_score_pair_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW2,
                        const __grid_constant__ CUtensorMap tmW1, const RsArgs args) {
    extern __shared__ uint8_t tc_smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (RS_SA + RS_SB) * RS_SLOT);
    // bars: fullA[SA] (leader's are used), emptyA[SA] (both), fullB[SB] (leader's), emptyB[SB] (both),
    //       tmem_full[2] (both), tmem_empty[2] (leader's)
    constexpr int NBARS = 2 * RS_SA + 2 * RS_SB + 4;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + NBARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const uint32_t rank = cluster_ctarank();
    const bool leader = rank == 0;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bar_base = smem_u32(bars);
    auto fullA = [&](int s) { return bar_base + 8u * s; };
    auto emptyA = [&](int s) { return bar_base + 8u * (RS_SA + s); };
    auto fullB = [&](int s) { return bar_base + 8u * (2 * RS_SA + s); };
    auto emptyB = [&](int s) { return bar_base + 8u * (2 * RS_SA + RS_SB + s); };
    auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * RS_SA + 2 * RS_SB + b); };
    auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * RS_SA + 2 * RS_SB + 2 + b); };
    auto slotA = [&](int s) { return smem_base + (uint32_t)s * RS_SLOT; };
    auto slotB = [&](int s) { return smem_base + (uint32_t)(RS_SA + s) * RS_SLOT; };

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2 * RS_SA + 2 * RS_SB; ++s) mbar_init(bar_base + 8u * s, 1);
        for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 2 * RS_EPI_WARPS); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tma_prefetch_desc(&tmX); tma_prefetch_desc(&tmW2); tma_prefetch_desc(&tmW1);
    }
    if (warp == 1) tmem2_alloc(smem_u32(tmem_slot), 512);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();          // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int kblocks = args.d / TC_BK;
    const int tiles_n = (args.E + 255) / 256, tiles_m = (args.T + 255) / 256;
    const int total_tiles = tiles_m * tiles_n * args.splits;
    const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
    // columns of n-tile nt: 256, or 128 for a last tile of at most 128 columns
    auto tile_cols = [&](int nt) { return (args.E - 256 * nt <= 128) ? 128 : 256; };
    // Unit of work t -> block of tokens, n-tile, half of K.  The 256-column tiles come first and the narrow last
    // ones after them (they cost half as much: the round-robin over the pairs then ends evenly); the halves of K of
    // one tile are neighbours, and so are the tiles of one block of tokens: x is read from DRAM once.
    const int wide_n = tiles_n - (tile_cols(tiles_n - 1) == 128 ? 1 : 0);
    const int wide_units = tiles_m * wide_n * args.splits;
    struct Unit { int mt, nt, kb0, kb1; float* out; };
    auto decode = [&](int t) {
        Unit u;
        int r, nn, n_first;
        if (t < wide_units) { r = t; nn = wide_n; n_first = 0; }
        else { r = t - wide_units; nn = tiles_n - wide_n; n_first = wide_n; }
        const int ks = r % args.splits;
        r /= args.splits;
        u.mt = r / nn;
        u.nt = n_first + (r - u.mt * nn);
        const int per = (kblocks + args.splits - 1) / args.splits;
        u.kb0 = ks * per;
        u.kb1 = min(kblocks, u.kb0 + per);
        u.out = ks ? args.z1 : args.z;
        return u;
    };

    if (warp == 0) {
        // ===================================================================== TMA producer (both CTAs)
        if (lane == 0) {
            int sa = 0, sb = 0; uint32_t pa = 0, pb = 0; bool alive = true;
            for (int t = cluster_id; t < total_tiles && alive; t += n_clusters) {
                const Unit u = decode(t);
                const int nt = u.nt;
                const int row0 = u.mt * 256 + 128 * (int)rank;        // past T: the copy fills zeros
                const int half_cols = tile_cols(nt) >> 1;             // this CTA's columns: 64 or 128
                const int chunk0 = (nt * 256 + (int)rank * half_cols) >> 6;
                const CUtensorMap* mw = half_cols == 128 ? &tmW2 : &tmW1;
                for (int kb = u.kb0; kb < u.kb1 && alive; ++kb) {
                    if (!mbar_wait(emptyA(sa), pa ^ 1u, abort_flag, args.status, STATUS_WAIT_EMPTY)) { alive = false; break; }
                    if (leader) mbar_expect_tx(fullA(sa), 2 * RS_SLOT);
                    tma2_load_2d(slotA(sa), &tmX, fullA(sa) & T2_PEER_MASK, kb * TC_BK, row0);
                    if (++sa == RS_SA) { sa = 0; pa ^= 1u; }
                    for (int ph = 0; ph < 3; ++ph) {
                        if (!mbar_wait(emptyB(sb), pb ^ 1u, abort_flag, args.status, STATUS_WAIT_EMPTY)) { alive = false; break; }
                        if (leader) mbar_expect_tx(fullB(sb), 2 * half_cols * TC_BK * 2);
                        // chunked map {64 columns, d rows, E/64 chunks, 3 pieces}
                        tma2_load_4d(slotB(sb), mw, fullB(sb) & T2_PEER_MASK, 0, kb * TC_BK, chunk0, ph);
                        if (++sb == RS_SB) { sb = 0; pb ^= 1u; }
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ===================================================================== MMA issuer (leader CTA)
        if (leader && lane == 0) {
            // kind::f16, bf16 x bf16 -> fp32, A K-major, B N-major, M = 256 over the pair; N per tile
            constexpr uint32_t idesc0 = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(256 >> 4) << 24);
            const uint64_t desc_a = smem_desc(0, 0, 1024);
            const uint64_t desc_b = smem_desc(0, TC_CHUNK_BYTES, 1024);
            constexpr uint32_t b_step = 2048 >> 4;      // 16 rows of K, 128 bytes each
            int sa = 0, sb = 0; uint32_t pa = 0, pb = 0; int it = 0; bool alive = true;
            for (int t = cluster_id; t < total_tiles && alive; t += n_clusters) {
                const Unit u = decode(t);
                const uint32_t idesc = idesc0 | ((uint32_t)(tile_cols(u.nt) >> 3) << 17);
                if (!mbar_wait(tempty_bar(it & 1), ((uint32_t)(it >> 1) & 1u) ^ 1u, abort_flag, args.status,
                               STATUS_WAIT_TMEM_EMPTY)) break;
                tc_fence_after();
                uint32_t d_tmem = tmem_base + (uint32_t)(it & 1) * TC_BN;
                int kseg = 0;                            // K block inside the segment
                for (int kb = u.kb0; kb < u.kb1 && alive; ++kb) {
                    if (!mbar_wait(fullA(sa), pa, abort_flag, args.status, STATUS_WAIT_FULL)) { alive = false; break; }
                    const uint64_t da = desc_a | (uint64_t)((slotA(sa) & 0x3ffffu) >> 4);
                    for (int ph = 0; ph < 3; ++ph) {
                        if (!mbar_wait(fullB(sb), pb, abort_flag, args.status, STATUS_WAIT_FULL)) { alive = false; break; }
                        tc_fence_after();
                        const uint64_t db = desc_b | (uint64_t)((slotB(sb) & 0x3ffffu) >> 4);
#pragma unroll
                        for (int k4 = 0; k4 < TC_BK / 16; ++k4)
                            umma2_bf16(d_tmem, da + k4 * 2, db + k4 * b_step, idesc, (kseg | ph | k4) != 0 ? 1u : 0u);
                        umma2_commit_both(emptyB(sb));
                        if (++sb == RS_SB) { sb = 0; pb ^= 1u; }
                    }
                    if (!alive) break;
                    umma2_commit_both(emptyA(sa));
                    if (++sa == RS_SA) { sa = 0; pa ^= 1u; }
                    if (++kseg == RS_SEG && kb + 1 < u.kb1) {
                        // segment done: hand this accumulator to the epilogue and go on in the other one
                        umma2_commit_both(tfull_bar(it & 1));
                        ++it;
                        kseg = 0;
                        if (!mbar_wait(tempty_bar(it & 1), ((uint32_t)(it >> 1) & 1u) ^ 1u, abort_flag, args.status,
                                       STATUS_WAIT_TMEM_EMPTY)) { alive = false; break; }
                        tc_fence_after();
                        d_tmem = tmem_base + (uint32_t)(it & 1) * TC_BN;
                    }
                }
                if (!alive) break;
                umma2_commit_both(tfull_bar(it & 1));
                ++it;
            }
        }
    } else {
        // ===================================================================== epilogue (8 warps, both CTAs)
        const int quarter = warp & 3;            // TMEM lanes 32*quarter .. +31 belong to this warp
        const int half = (warp - 2) >> 2;        // columns [128*half, 128*half + 128) of the tile
        int it = 0;
        bool ok = true;
        for (int t = cluster_id; t < total_tiles && ok; t += n_clusters) {
            const Unit u = decode(t);
            const int mt = u.mt, nt = u.nt;
            const int nseg = (u.kb1 - u.kb0 + RS_SEG - 1) / RS_SEG;
            const bool active = half * 128 < tile_cols(nt);
            float sum[4][32];
#pragma unroll
            for (int g = 0; g < 4; ++g)
#pragma unroll
                for (int i = 0; i < 32; ++i) sum[g][i] = 0.0f;
            for (int sg = 0; sg < nseg; ++sg) {
                const int b = it & 1;
                if (!mbar_wait_warp(tfull_bar(b), (uint32_t)(it >> 1) & 1u, abort_flag, args.status, STATUS_WAIT_TMEM_FULL,
                                    lane)) { ok = false; break; }
                tc_fence_after();
                if (active) {
                    const uint32_t ta = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)b * TC_BN + half * 128;
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        float part[32];
                        tmem_ld32(ta + 32 * g, part);
#pragma unroll
                        for (int i = 0; i < 32; ++i) sum[g][i] += part[i];
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(tempty_bar(b) & T2_PEER_MASK);
                ++it;
            }
            if (!ok) break;
            const int row = mt * 256 + 128 * (int)rank + quarter * 32 + lane;
            if (active && row < args.T) {
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    const int col = nt * 256 + half * 128 + 32 * g;
                    if (col < args.E) epi_f32<32>(u.out + (size_t)row * args.E + col, sum[g], 0);
                }
            }
        }
    }

    // ------------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) __nanosleep(1000);
        __syncthreads();
    }
    cluster_sync_all();          // neither CTA leaves while the other may still signal its barriers
    if (warp == 1) {
        tc_fence_after();
        tmem2_dealloc(tmem_base, 512);
    }
}

inline mop_status rs_init() {
    return cudaFuncSetAttribute(route_score_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, RS_SMEM_BYTES) ==
                   cudaSuccess ? MOP_OK : MOP_ERR_CUDA;
}

// Halves of K as separate units pay when the tiles leave many pairs idle or end unevenly (config 5: 32 wide and 32
// narrow tiles on 74 pairs: the last pair finishes after 0.75 instead of 1 tile time); the makespan of the
// kernel's round-robin is computed for both and the shorter one taken.
inline int rs_pick_splits(int T, int d, int E, int n_clusters) {
    const int tiles_m = (T + 255) / 256, tiles_n = (E + 255) / 256;
    const bool narrow_last = E - 256 * (tiles_n - 1) <= 128;
    const int wide_n = tiles_n - (narrow_last ? 1 : 0);
    if (d / TC_BK < 2 * RS_SEG || n_clusters < 1) return 1;
    double best = 0.0;
    int pick = 1;
    for (int splits = 1; splits <= 2; ++splits) {
        const int wide = tiles_m * wide_n * splits, total = tiles_m * tiles_n * splits;
        double worst = 0.0;
        for (int c = 0; c < n_clusters && c < total; ++c) {
            double sum = 0.0;
            for (int t = c; t < total; t += n_clusters) sum += (t < wide ? 1.0 : 0.5) / splits;
            worst = sum > worst ? sum : worst;
        }
        worst += 0.03 * (splits - 1);     // a second partial sum costs a little in the selection
        if (splits == 1 || worst < 0.9 * best) { best = worst; pick = splits; }
    }
    return pick;
}

// x: [T, d] bf16; pieces: [3, d, E] bf16; z, z1: [T, E] fp32 (all device).  d and E multiples of 64.
// Returns in *used_splits whether the logits are z (1) or z + z1 (2).
inline mop_status rs_launch(const TcPlan* p, const char* name, const void* x, const void* pieces, float* z, float* z1,
                            int T, int d, int E, int32_t* status, int* used_splits, cudaStream_t st) {
    CUtensorMap mX, mW2, mW1;
    if (!tc_map_2d(p, &mX, x, T, d, 128) || !tc_map_chunked_3d(p, &mW2, pieces, 3, d, E, 2) ||
        !tc_map_chunked_3d(p, &mW1, pieces, 3, d, E, 1))
        return MOP_ERR_CUDA;
    const int grid = p->sm_count & ~1;
    RsArgs a{};
    a.z = z; a.z1 = z1; a.T = T; a.d = d; a.E = E; a.status = status;
    a.splits = z1 ? rs_pick_splits(T, d, E, grid / 2) : 1;
    *used_splits = a.splits;
    p->prof->begin(name, st);
    route_score_pair_kernel<<<grid, RS_THREADS, RS_SMEM_BYTES, st>>>(mX, mW2, mW1, a);
    p->prof->end(st);
    return cudaGetLastError() == cudaSuccess ? MOP_OK : MOP_ERR_CUDA;
}

}  // namespace mop
