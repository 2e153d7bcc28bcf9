// Two-CTA tensor-core grouped GEMMs (tcgen05.mma.cta_group::2) for the kinds whose rows are token
// rows (F1, F2, B2, B4).  A cluster of two CTAs on neighbouring SMs computes a 256 x 256 tile: each
// CTA loads its own 128 rows of A and HALF of the B tile (128 of the 256 N columns), the leader CTA
// issues one MMA of M=256, N=256, K=16 that reads both CTAs' shared memory, and each CTA's TMEM
// receives its own 128 x 256 accumulator.  Per output element this halves the B bytes that cross
// L2 -> SM and shared memory, which is what bounds the one-CTA kernel; the smaller stage (32 KiB)
// also allows six pipeline stages instead of four.
//
// Synchronisation: TMA loads of both CTAs complete on the LEADER's "full" barrier (the loads carry
// .cta_group::2 and the barrier address has the CTA-rank bit cleared); the leader's commits are
// multicast to the "empty" and "accumulator full" barriers of both CTAs; the epilogue warps of both
// CTAs arrive on the leader's "accumulator empty" barrier.  No TMA multicast is used anywhere.
// Every wait is bounded as in the one-CTA kernel.
#pragma once
#include "gemm_tc.cuh"

namespace mop {

constexpr int T2_STAGES = 6;
constexpr int T2_A_BYTES = TC_BM * TC_BK * 2;        // 16 KiB: this CTA's 128 rows of A
constexpr int T2_B_BYTES = 128 * TC_BK * 2;          // 16 KiB: this CTA's 128 N columns of B
constexpr int T2_STAGE_BYTES = T2_A_BYTES + T2_B_BYTES;
constexpr int T2_SMEM_BYTES = T2_STAGES * T2_STAGE_BYTES + 1024 /*align*/ + TC_BAR_BYTES;
constexpr int T2_THREADS = 192;
constexpr uint32_t T2_PEER_MASK = 0xFEFFFFFFu;       // clears the CTA-rank bit of a shared::cluster address

// ------------------------------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tma2_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], "
        "[%2];" ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tma2_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, "
        "%5}], [%2];" ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
        : "memory");
}
__device__ __forceinline__ void tma2_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z,
                                             int w) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, "
        "%5, %6}], [%2];" ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z), "r"(w)
        : "memory");
}
// the same copy with an L2 eviction policy
__device__ __forceinline__ void tma2_load_4d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y,
                                                  int z, int w, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], "
        "[%1, {%3, %4, %5, %6}], [%2], %7;" ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z), "r"(w), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void tmem2_alloc(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem2_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma2_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                           uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(
            d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// commit to the barrier at this shared-memory offset in BOTH CTAs of the pair
__device__ __forceinline__ void umma2_commit_both(uint32_t bar) {
    const uint16_t mask = 3;
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
        "h"(mask)
        : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Instruction descriptor of the pair: M = 256 across the two CTAs, N = 256.
__host__ __device__ constexpr uint32_t make_idesc2(bool b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn ? 1u : 0u) << 16) | ((uint32_t)(256 >> 3) << 17) |
           ((uint32_t)(256 >> 4) << 24);
}

// 256-row pair tiles of the ragged-M GEMMs: {expert, first row, rows in the pair (1..256), 0}.
__global__ void __launch_bounds__(1024) tc_build_pairtiles_kernel(const int32_t* __restrict__ offsets, int E,
                                                                  int4* __restrict__ tiles,
                                                                  int32_t* __restrict__ n_tiles) {
    __shared__ int32_t scan[1025];
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
    for (int i = 0; i < nt; ++i) tiles[first + i] = make_int4(e, off + i * 256, min(256, cnt - i * 256), 0);
    if (e == 1023) *n_tiles = scan[1023];
}

// Mixed schedule: the full 256-row pairs of every expert go to the two-CTA kernel, the remaining
// rows (< 256 per expert, as one or two 128-row tiles) to the one-CTA kernel, so that pairing adds
// no padding.  One launch builds both lists.
__global__ void __launch_bounds__(1024) tc_build_mixed_kernel(const int32_t* __restrict__ offsets, int E,
                                                              int4* __restrict__ pair_tiles,
                                                              int32_t* __restrict__ n_pairs,
                                                              int4* __restrict__ single_tiles,
                                                              int32_t* __restrict__ n_singles) {
    __shared__ int32_t scan_p[1024], scan_s[1024];
    const int e = threadIdx.x;
    int cnt = 0, off = 0;
    if (e < E) { off = offsets[e]; cnt = offsets[e + 1] - off; }
    const int np = cnt / 256;
    const int rem = cnt - 256 * np;
    const int ns = (rem + TC_BM - 1) / TC_BM;
    scan_p[e] = np; scan_s[e] = ns;
    __syncthreads();
    for (int s = 1; s < 1024; s <<= 1) {
        const int vp = (e >= s) ? scan_p[e - s] : 0, vs = (e >= s) ? scan_s[e - s] : 0;
        __syncthreads();
        scan_p[e] += vp; scan_s[e] += vs;
        __syncthreads();
    }
    const int fp = scan_p[e] - np, fs = scan_s[e] - ns;
    for (int i = 0; i < np; ++i) pair_tiles[fp + i] = make_int4(e, off + i * 256, 256, 0);
    for (int i = 0; i < ns; ++i)
        single_tiles[fs + i] = make_int4(e, off + 256 * np + i * TC_BM, min(TC_BM, rem - i * TC_BM), 0);
    if (e == 1023) { *n_pairs = scan_p[1023]; *n_singles = scan_s[1023]; }
}

// ------------------------------------------------------------------------------------------ kernel
template <int KIND>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(T2_THREADS, 1)
tc_gemm2_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmA1,
                const __grid_constant__ CUtensorMap tmB0, const __grid_constant__ CUtensorMap tmB1,
                const TcArgs args) {
    using Tr = TcTraits<KIND>;
    static_assert(!Tr::RAGGED_K, "token-row kinds only");
    constexpr int S = T2_STAGES;
    extern __shared__ uint8_t tc_smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S * T2_STAGE_BYTES);
    // bars: [0,S) full (leader's are used), [S,2S) empty (both), tmem_full[2] (both), tmem_empty[2] (leader's)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * S + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

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
        tma_prefetch_desc(&tmA0); tma_prefetch_desc(&tmB0);
        if (Tr::PHASES == 2) tma_prefetch_desc(&tmA1);
        if (Tr::DUAL_B || Tr::PHASES == 2) tma_prefetch_desc(&tmB1);
    }
    if (warp == 1) tmem2_alloc(smem_u32(tmem_slot), 512);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();          // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int total_tiles = (*args.n_mtiles) * args.tiles_n;
    const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
    auto decode = [&](int t) {
        TileInfo ti;
        int mt, nt;
        if (args.m_fastest) { const int nm = __ldg(args.n_mtiles); nt = t / nm; mt = t - nt * nm; }
        else { mt = t / args.tiles_n; nt = t - mt * args.tiles_n; }
        const int4 m = __ldg(args.mtiles + mt);
        ti.e = m.x; ti.row0 = m.y + 128 * (int)rank; ti.rows = min(128, max(0, m.z - 128 * (int)rank));
        ti.m0 = 0; ti.nt = nt; ti.skip = false;
        return ti;
    };

    if (warp == 0) {
        // ===================================================================== TMA producer (both CTAs)
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0; bool alive = true;
            TileInfo nxt = decode(min(cluster_id, max(total_tiles - 1, 0)));
            for (int t = cluster_id; t < total_tiles && alive; t += n_clusters) {
                const TileInfo ti = nxt;
                if (t + n_clusters < total_tiles) nxt = decode(t + n_clusters);
                const int n0 = ti.nt * Tr::N_PER_TILE + (KIND == TC_VP ? args.n_base : 0);
                const int nkb = Tr::PHASES * args.kblocks;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, args.status, STATUS_WAIT_EMPTY)) {
                        alive = false; break;
                    }
                    const uint32_t fb = full_bar(stage) & T2_PEER_MASK;    // the leader's barrier
                    if (leader) mbar_expect_tx(full_bar(stage), 2 * T2_STAGE_BYTES);
                    const uint32_t sA = smem_base + stage * T2_STAGE_BYTES;
                    const uint32_t sB = sA + T2_A_BYTES;
                    const int ph = (Tr::PHASES == 2 && kb >= args.kblocks) ? 1 : 0;
                    const int k0 = (kb - ph * args.kblocks) * TC_BK;
                    tma2_load_2d(sA, ph ? &tmA1 : &tmA0, fb, k0, ti.row0);
                    if constexpr (!Tr::B_MN) {
                        // K-major weights: this CTA's 128 output columns are 128 rows of the [E, N, K] tensor
                        tma2_load_3d(sB, ph ? &tmB1 : &tmB0, fb, k0 + (KIND == TC_VX ? args.kb_base : 0), n0 + 128 * (int)rank,
                                     ti.e);
                    } else {
                        // N-major weights: two 64-wide column chunks; with two B tensors (gate | up) the
                        // leader holds the gate columns and the peer the up columns
                        const CUtensorMap* mp = (Tr::DUAL_B && rank) ? &tmB1 : &tmB0;
                        const int nb = Tr::DUAL_B ? n0 : n0 + 128 * (int)rank;
                        tma2_load_4d(sB, mp, fb, 0, k0, nb >> 6, ti.e);   // chunked map, two chunks per copy
                    }
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ===================================================================== MMA issuer (leader CTA)
        // one thread runs the whole loop (wait, fence, four MMAs, commit) with precomputed descriptors
        if (leader && lane == 0) {
            constexpr uint32_t idesc = make_idesc2(Tr::B_MN);
            const uint64_t desc_a = smem_desc(0, 0, 1024);
            const uint64_t desc_b = Tr::B_MN ? smem_desc(0, TC_CHUNK_BYTES, 1024) : smem_desc(0, 0, 1024);
            constexpr uint32_t b_step = (Tr::B_MN ? 2048 : 32) >> 4;
            int stage = 0; uint32_t phase = 0; int it = 0; bool alive = true;
            const int nkb = Tr::PHASES * args.kblocks;
            for (int t = cluster_id; t < total_tiles && alive; t += n_clusters) {
                const int buf = it & 1;
                const uint32_t tphase = (uint32_t)(it >> 1) & 1u;
                if (!mbar_wait(tempty_bar(buf), tphase ^ 1u, abort_flag, args.status, STATUS_WAIT_TMEM_EMPTY)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)buf * TC_BN;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag, args.status, STATUS_WAIT_FULL)) {
                        alive = false; break;
                    }
                    tc_fence_after();
                    const uint32_t sA = smem_base + stage * T2_STAGE_BYTES;
                    const uint64_t da = desc_a | (uint64_t)((sA & 0x3ffffu) >> 4);
                    const uint64_t db = desc_b | (uint64_t)(((sA + T2_A_BYTES) & 0x3ffffu) >> 4);
#pragma unroll
                    for (int k4 = 0; k4 < TC_BK / 16; ++k4)
                        umma2_bf16(d_tmem, da + k4 * 2, db + k4 * b_step, idesc, (kb | k4) != 0 ? 1u : 0u);
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
        const int quarter = warp & 3;
        const int r = quarter * 32 + lane;
        int it = 0;
        TileInfo nxt = decode(min(cluster_id, max(total_tiles - 1, 0)));
        for (int t = cluster_id; t < total_tiles; t += n_clusters) {
            const TileInfo ti = nxt;
            if (t + n_clusters < total_tiles) nxt = decode(t + n_clusters);
            const int buf = it & 1;
            const uint32_t tphase = (uint32_t)(it >> 1) & 1u;
            if (!mbar_wait_warp(tfull_bar(buf), tphase, abort_flag, args.status, STATUS_WAIT_TMEM_FULL, lane)) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)buf * TC_BN;
            tc_epilogue_rows<KIND>(args, taddr, r < ti.rows, ti.row0 + r,
                                   ti.nt * Tr::N_PER_TILE + (KIND == TC_VP ? args.n_base : 0), ti.nt);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(tempty_bar(buf) & T2_PEER_MASK);
            ++it;
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

// ------------------------------------------------------------------------------------------ host
template <int KIND>
inline mop_status tc2_set_smem() {
    return cudaFuncSetAttribute(tc_gemm2_kernel<KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize, T2_SMEM_BYTES) ==
                   cudaSuccess ? MOP_OK : MOP_ERR_CUDA;
}

inline mop_status tc2_init() {
    mop_status r;
    if ((r = tc2_set_smem<TC_F1>()) != MOP_OK) return r;
    if ((r = tc2_set_smem<TC_F2>()) != MOP_OK) return r;
    if ((r = tc2_set_smem<TC_B2>()) != MOP_OK) return r;
    if ((r = tc2_set_smem<TC_B4>()) != MOP_OK) return r;
    if ((r = tc2_set_smem<TC_VL>()) != MOP_OK) return r;
    if ((r = tc2_set_smem<TC_VP>()) != MOP_OK) return r;
    if ((r = tc2_set_smem<TC_VX>()) != MOP_OK) return r;
    return MOP_OK;
}

template <int KIND>
inline mop_status tc2_launch(const TcPlan* p, const char* name, const CUtensorMap& a0, const CUtensorMap& a1,
                             const CUtensorMap& b0, const CUtensorMap& b1, const TcArgs& args, cudaStream_t st) {
    p->prof->begin(name, st);
    const int grid = p->sm_count & ~1;   // whole pairs
    tc_gemm2_kernel<KIND><<<grid, T2_THREADS, T2_SMEM_BYTES, st>>>(a0, a1, b0, b1, args);
    p->prof->end(st);
    return cudaGetLastError() == cudaSuccess ? MOP_OK : MOP_ERR_CUDA;
}

inline mop_status tc2_build_mixed(const TcPlan* p, const int32_t* offsets, int32_t* tiles, int32_t* tiles2,
                                  cudaStream_t st) {
    p->prof->begin("tc_build_mixed_tiles", st);
    tc_build_mixed_kernel<<<1, 1024, 0, st>>>(offsets, p->s.E, reinterpret_cast<int4*>(tiles + 64), tiles,
                                              reinterpret_cast<int4*>(tiles2 + 64), tiles2);
    p->prof->end(st);
    return cudaGetLastError() == cudaSuccess ? MOP_OK : MOP_ERR_CUDA;
}

inline mop_status tc2_build_tiles(const TcPlan* p, const int32_t* offsets, int32_t* tiles, cudaStream_t st) {
    p->prof->begin("tc_build_pairtiles", st);
    tc_build_pairtiles_kernel<<<1, 1024, 0, st>>>(offsets, p->s.E, reinterpret_cast<int4*>(tiles + 64), tiles);
    p->prof->end(st);
    return cudaGetLastError() == cudaSuccess ? MOP_OK : MOP_ERR_CUDA;
}

}  // namespace mop
