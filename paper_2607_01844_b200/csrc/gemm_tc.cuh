// Tensor-core grouped GEMMs for sm_100a: tcgen05.mma with TMEM accumulators, operands staged by
// TMA into 128-byte-swizzled shared memory, one persistent warp-specialised CTA per SM.
//
// Every GEMM of the layer is one instantiation of tc_grouped_gemm_kernel<KIND>:
//   F1   [G|U] = Xp W_gate[e] | Xp W_up[e]        SwiGLU epilogue -> H (+ stash)      ragged M
//   F2   O     = H W_down[e]                      gate epilogue   -> Yp               ragged M
//   B2   dHu   = dYp W_down[e]^T                  SwiGLU-backward epilogue            ragged M
//   B4   dXp   = dG W_gate[e]^T + dU W_up[e]^T    (two K phases)  -> bf16             ragged M
//   WD   dW_down[e] = (gate H)_e^T dYp_e          fp32 store                          ragged K
//   WGU  dW_gate[e] = Xp_e^T dG_e, dW_up[e] = Xp_e^T dU_e  (a tile belongs to one of the two)  ragged K
//   VL   Y = X W_voc (never stored)               online log-sum-exp partials         dense M
//   VP   dY = g ([v = t] - exp(X W_voc - lse))     bf16, one block of vocabulary columns dense M
//   VX   dX += dY W_voc^T over that block          fp32 read-modify-write              dense M
// CTA tile 128 x 256 (one tcgen05.mma.cta_group::1 of M=128, N=256, K=16 per 32 bytes of K),
// K step 64 per pipeline stage, 4 stages, two 256-column accumulators in TMEM so that the
// epilogue of tile i overlaps the main loop of tile i+1.
//
// Roles: warp 0 = TMA producer, warp 1 = MMA issuer (owns TMEM), warps 2..5 = epilogue.
// Every mbarrier wait is bounded: on expiry the CTA records a code in the status word, raises a
// CTA-wide abort flag, lets its copies land, frees TMEM and returns.
#pragma once
#include <cuda.h>

#include "../../include/mop_moe.h"
#include "epilogue.cuh"

namespace mop {

enum : int { TC_F1 = 0, TC_F2 = 1, TC_B2 = 2, TC_B4 = 3, TC_WD = 4, TC_WGU = 5, TC_VL = 6, TC_VP = 7, TC_VX = 8 };

constexpr int TC_BM = 128, TC_BN = 256, TC_BK = 64;
constexpr int TC_A_BYTES = TC_BM * TC_BK * 2;   // 16 KiB
constexpr int TC_B_BYTES = TC_BN * TC_BK * 2;   // 32 KiB
constexpr int TC_STAGE_BYTES = TC_A_BYTES + TC_B_BYTES;
constexpr int TC_CHUNK_BYTES = 64 * TC_BK * 2;  // one 64-wide MN chunk of 64 K rows: 8 KiB
constexpr int TC_BAR_BYTES = 1024;                // barriers, TMEM slot, abort flag (keeps 1 KiB alignment)
constexpr long long TC_WAIT_CYCLES = 4000000000ll;  // about two seconds

template <int KIND>
struct TcTraits {
    static constexpr bool A_MN = (KIND == TC_WD || KIND == TC_WGU);   // A is M-contiguous in memory
    static constexpr bool B_MN = (KIND != TC_B2 && KIND != TC_B4 && KIND != TC_VX);   // B is N-contiguous in memory
    static constexpr bool DUAL_B = (KIND == TC_F1);                   // two B tensors, 128 columns each
    // Both weight gradients of the up-projection in one launch: the second half of an m-block's n-tiles takes
    // its B operand from the second tensor (dU) and writes the second output (dW_up).  A tile thus covers 256
    // columns (1 KiB per row) of ONE gradient: DRAM takes such a store stream faster than 2 x 512 bytes.
    static constexpr bool SEL_B = (KIND == TC_WGU);
    static constexpr bool RAGGED_K = A_MN;
    static constexpr bool B_WEIGHT = !RAGGED_K;                       // B is an [E, ., .] weight tensor
    static constexpr int PHASES = (KIND == TC_B4) ? 2 : 1;
    static constexpr int N_PER_TILE = DUAL_B ? 128 : 256;             // output columns per tensor per tile
    // Weight gradients have a short K loop (the expert's rows) and a 128 KiB fp32 tile to write, so
    // they run eight epilogue warps (two per TMEM lane quarter, 128 columns each).
    static constexpr int STAGES = RAGGED_K ? 3 : 4;
    static constexpr int EPI_WARPS = RAGGED_K ? 8 : 4;
    static constexpr int THREADS = 64 + 32 * EPI_WARPS;
    static constexpr int STORE_BYTES = RAGGED_K ? 4 * 16384 : 0;   // two 128-row x 32-column fp32 store boxes per half
    static constexpr int SMEM_BYTES = STAGES * TC_STAGE_BYTES + 1024 /*align*/ + TC_BAR_BYTES + STORE_BYTES;
};

struct TcArgs {
    const int32_t* offsets;
    const int4* mtiles;      // ragged M: {expert, first row, rows, 0} per 128-row tile
    const int32_t* n_mtiles; // device scalar
    int E;
    int tiles_n;             // n-tiles per row block
    int tiles_m_fixed;       // ragged K: m-tiles per expert
    int kblocks;             // ragged M: K / 64 (rounded up) per phase
    int Mfix, N;             // ragged K: output rows per expert; N = columns per output tensor
    int m_fastest;           // tile order: 1 = consecutive tiles walk the row tiles of one column block
    const int32_t* targets;  // VL, VP: target column per row
    float* ylab;             // VL: logit of the target column per row
    const float* row_lse;    // VP: log-sum-exp per row
    const float* row_g;      // VP: upstream weight per row
    int n_base;              // VP: first vocabulary column of the block (added to the tile's columns)
    int kb_base;             // VX: first vocabulary column of the block (added to B's K coordinate)
    int32_t* status;
    EpiArgs ep;
    float* outf1;            // WGU: second output tensor
    int keep_empty;          // weight gradients: leave the gradients of experts without rows untouched
};

// ------------------------------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
// Bounded wait.  Returns false if the CTA is aborting (this wait or another one ran out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                          int code, long long limit = TC_WAIT_CYCLES) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 32; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > limit) {
            *abort_flag = 1;
            atomicCAS(status, 0, code);
            return false;
        }
    }
}

// Barrier over `nthreads` threads (named barrier `id`) that also ANDs a predicate: every participant
// learns whether ALL of them arrived with ok.  Used where warps that took a bounded wait separately
// must agree on giving up before they meet at plain barriers (a warp that left alone would hang the rest).
__device__ __forceinline__ bool bar_vote_all(int id, int nthreads, bool ok) {
    uint32_t r;
    asm volatile(
        "{\n.reg .pred p, q;\nsetp.ne.b32 p, %3, 0;\nbar.red.and.pred q, %1, %2, p;\nselp.u32 %0, 1, 0, q;\n}"
        : "=r"(r)
        : "r"(id), "r"(nthreads), "r"(ok ? 1u : 0u)
        : "memory");
    return r != 0;
}

// Warp-uniform form: lane 0 waits, the outcome is broadcast, and every lane then observes the
// completed phase itself (so that its later reads are ordered after the barrier).
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                               int32_t* status, int code, int lane) {
    uint32_t ok = 1;
    if (lane == 0) ok = mbar_wait(bar, parity, abort_flag, status, code) ? 1u : 0u;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    if (ok) (void)mbar_try_wait(bar, parity);
    return ok != 0;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], "
        "[%2];" ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
        : "memory");
}
// L2 eviction policies for the weight-gradient kernels: their fp32 output stream (tens of GB, never
// re-read) would otherwise push the small operand set (an expert's rows, re-read by every tile of
// that expert) out of L2 between uses.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void tma_load_3d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y,
                                                 int z, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, "
        "{%3, %4, %5}], [%2], %6;" ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void tma_store_3d_hint(const CUtensorMap* map, uint32_t src, int x, int y, int z,
                                                  uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group.L2::cache_hint [%0, {%2, %3, %4}], [%1], %5;" ::"l"(
            map),
        "r"(src), "r"(x), "r"(y), "r"(z), "l"(policy)
        : "memory");
}
// shared -> global tile store (or fp32 add) of one box; completion is tracked by bulk groups
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int x, int y, int z) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(map),
                 "r"(src), "r"(x), "r"(y), "r"(z)
                 : "memory");
}
__device__ __forceinline__ void tma_reduce_add_3d(const CUtensorMap* map, uint32_t src, int x, int y, int z) {
    asm volatile("cp.reduce.async.bulk.tensor.3d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(
                     map),
                 "r"(src), "r"(x), "r"(y), "r"(z)
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void tma_store_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z,
                                            int w) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, "
        "%6}], [%2];" ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z), "r"(w)
        : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(
            d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 lanes x 32 consecutive fp32 columns: thread i of the warp gets lane (base lane + i).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Same load without the wait, so that several can be in flight; tmem_ld_wait then orders every
// later use of the destination registers after the wait.
__device__ __forceinline__ void tmem_ld32_nowait(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld_wait(float (&a)[32], float (&b)[32]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
    // empty statements that "modify" the registers: nothing that reads them can move above the wait
#pragma unroll
    for (int i = 0; i < 32; ++i) asm volatile("" : "+f"(a[i]), "+f"(b[i]));
}

__device__ __forceinline__ void tmem_ld_wait4(float (&a)[32], float (&b)[32], float (&c)[32], float (&d)[32]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) asm volatile("" : "+f"(a[i]), "+f"(b[i]), "+f"(c[i]), "+f"(d[i]));
}

// Shared-memory matrix descriptor, 128-byte swizzle, version 1 (Blackwell).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3ffffu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32;
    d |= (uint64_t)1 << 46;   // descriptor version
    d |= (uint64_t)2 << 61;   // SWIZZLE_128B
    return d;
}

// Instruction descriptor: fp32 accumulate, bf16 operands, M=128, N=256, operand majors.
__host__ __device__ constexpr uint32_t make_idesc(bool a_mn, bool b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
           ((uint32_t)(TC_BN >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
}

// Self-test of the bounded wait: one thread waits on a barrier that nothing will ever complete, with
// a short limit; the wait must give up, record its code in the status word and let the kernel end.
__global__ void tc_wait_selftest_kernel(int32_t* status, long long limit_cycles, int32_t* gave_up) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const bool ok = mbar_wait(smem_u32(&bar), 0, &abort_flag, status, STATUS_WAIT_FULL, limit_cycles);
        *gave_up = ok ? 0 : 1;
    }
}

// ------------------------------------------------------------------------------------------ tiles
struct TileInfo {
    int e, row0, rows;   // ragged M: first global row and valid rows; ragged K: first k row and k count
    int m0;              // ragged K: first output row of the tile inside the expert's matrix
    int nt;              // n-tile index
    int sel;             // SEL_B kinds: 1 = second B tensor and second output
    bool skip;           // nothing to multiply (expert without rows)
};

template <int KIND>
__device__ __forceinline__ TileInfo decode_tile(const TcArgs& a, int t) {
    TileInfo ti;
    ti.sel = 0;
    if constexpr (TcTraits<KIND>::RAGGED_K) {
        const int per_e = a.tiles_m_fixed * a.tiles_n;
        ti.e = t / per_e;
        const int r = t - ti.e * per_e;
        ti.m0 = (r / a.tiles_n) * TC_BM;
        ti.nt = r % a.tiles_n;
        if constexpr (TcTraits<KIND>::SEL_B) {
            const int half_n = a.tiles_n >> 1;
            if (ti.nt >= half_n) { ti.nt -= half_n; ti.sel = 1; }
        }
        ti.row0 = __ldg(a.offsets + ti.e);
        ti.rows = __ldg(a.offsets + ti.e + 1) - ti.row0;
        ti.skip = ti.rows <= 0;
    } else {
        int mt, nt;
        if (a.m_fastest) { const int nm = __ldg(a.n_mtiles); nt = t / nm; mt = t - nt * nm; }
        else { mt = t / a.tiles_n; nt = t - mt * a.tiles_n; }
        const int4 m = __ldg(a.mtiles + mt);
        ti.e = m.x; ti.row0 = m.y; ti.rows = m.z; ti.m0 = 0;
        ti.nt = nt;
        ti.skip = false;
    }
    return ti;
}

// 128-row tile list of the ragged-M GEMMs, built on the device from offsets (no host round trip).
__device__ __forceinline__ void tc_build_mtiles_body(const int32_t* __restrict__ offsets, int E,
                                                     int4* __restrict__ mtiles, int32_t* __restrict__ n_mtiles,
                                                     int32_t* scan) {
    const int e = threadIdx.x;
    int cnt = 0, off = 0;
    if (e < E) { off = offsets[e]; cnt = offsets[e + 1] - off; }
    const int nt = (cnt + TC_BM - 1) / TC_BM;
    scan[e] = nt;
    __syncthreads();
    // inclusive scan, Hillis-Steele over 1024 entries
    for (int s = 1; s < 1024; s <<= 1) {
        const int v = (e >= s) ? scan[e - s] : 0;
        __syncthreads();
        scan[e] += v;
        __syncthreads();
    }
    const int first = scan[e] - nt;
    for (int i = 0; i < nt; ++i) mtiles[first + i] = make_int4(e, off + i * TC_BM, min(TC_BM, cnt - i * TC_BM), 0);
    if (e == 1023) *n_mtiles = scan[1023];
}
__global__ void __launch_bounds__(1024) tc_build_mtiles_kernel(const int32_t* __restrict__ offsets, int E,
                                                               int4* __restrict__ mtiles,
                                                               int32_t* __restrict__ n_mtiles) {
    __shared__ int32_t scan[1025];
    tc_build_mtiles_body(offsets, E, mtiles, n_mtiles, scan);
}

// Epilogue of one 128 x 256 accumulator for the kinds whose rows are token rows: this thread owns
// row `grow` (valid iff row_ok) and walks the 256 columns in runs of 32.
template <int KIND>
__device__ __forceinline__ void tc_epilogue_rows(const TcArgs& args, uint32_t taddr, bool row_ok, int grow, int n0,
                                                 int nt) {
    float acc[32];
    if constexpr (KIND == TC_F1) {
        float acc2[32];
#pragma unroll 1
        for (int c = 0; c < 128; c += 32) {
            tmem_ld32(taddr + c, acc);
            tmem_ld32(taddr + 128 + c, acc2);
            if (row_ok && n0 + c < args.N) {
#pragma unroll
                for (int s = 0; s < 32; s += 8) {
                    float g8[8], u8[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) { g8[q] = acc[s + q]; u8[q] = acc2[s + q]; }
                    epi_swiglu<8>(args.ep, grow, n0 + c + s, g8, u8);
                }
            }
        }
    } else if constexpr (KIND == TC_F2 || KIND == TC_B2) {
        const float gate = row_ok ? args.ep.gate[args.ep.row_src[grow]] : 0.0f;
        float dot = 0.0f;
#pragma unroll 1
        for (int c = 0; c < TC_BN; c += 32) {
            tmem_ld32(taddr + c, acc);
            if (row_ok && n0 + c < args.N) {
#pragma unroll
                for (int s = 0; s < 32; s += 8) {
                    float a8[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) a8[q] = acc[s + q];
                    if constexpr (KIND == TC_F2) epi_gate<8>(args.ep, grow, n0 + c + s, gate, a8);
                    else dot += epi_dh<8>(args.ep, grow, n0 + c + s, gate, a8);
                }
            }
        }
        if (KIND == TC_B2 && row_ok) args.ep.part[(size_t)nt * args.ep.M_total + grow] = dot;
    } else if constexpr (KIND == TC_VL) {
        // Online log-sum-exp over this tile's 256 logits of the row (fp32 accumulators, never stored):
        // running maximum m and s = sum exp(y - m); the target's logit is picked up where it falls.
        float m = -INFINITY, ssum = 0.0f;
        const int tgt = row_ok ? args.targets[grow] - n0 : -1;
#pragma unroll 1
        for (int c = 0; c < TC_BN; c += 32) {
            tmem_ld32(taddr + c, acc);
            if (row_ok && n0 + c < args.N) {
                float cm = acc[0];
#pragma unroll
                for (int q = 1; q < 32; ++q) cm = fmaxf(cm, acc[q]);
                const float nm = fmaxf(m, cm);
                float part = 0.0f;
#pragma unroll
                for (int q = 0; q < 32; ++q) part += __expf(acc[q] - nm);
                ssum = ssum * __expf(m - nm) + part;
                m = nm;
                if (tgt >= c && tgt < c + 32) {
                    float y = 0.0f;
#pragma unroll
                    for (int q = 0; q < 32; ++q) y = (tgt - c == q) ? acc[q] : y;
                    args.ylab[grow] = y;
                }
            }
        }
        if (row_ok) {
            reinterpret_cast<float2*>(args.ep.part)[(size_t)nt * args.ep.M_total + grow] = make_float2(m, ssum);
        }
    } else if constexpr (KIND == TC_VP) {
        // Gradient of the log-likelihood with respect to the logits of this block of the vocabulary,
        // from the recomputed logits and the row's log-sum-exp; bf16, block-local columns.
        const float lse = row_ok ? args.row_lse[grow] : 0.0f;
        const float g = row_ok ? args.row_g[grow] : 0.0f;
        const int tgt = row_ok ? args.targets[grow] - n0 : -1;
#pragma unroll 1
        for (int c = 0; c < TC_BN; c += 32) {
            tmem_ld32(taddr + c, acc);
            if (row_ok && n0 + c < args.N) {
#pragma unroll
                for (int q = 0; q < 32; ++q) acc[q] = g * ((tgt - c == q ? 1.0f : 0.0f) - __expf(acc[q] - lse));
#pragma unroll
                for (int s = 0; s < 32; s += 8) {
                    float a8[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) a8[q] = acc[s + q];
                    store_bf16_run<8>(args.ep.out0 + (size_t)grow * args.ep.ldo + (n0 - args.n_base) + c + s, a8);
                }
            }
        }
    } else if constexpr (KIND == TC_VX) {
#pragma unroll 1
        for (int c = 0; c < TC_BN; c += 32) {
            tmem_ld32(taddr + c, acc);
            if (row_ok && n0 + c < args.N) epi_f32<32>(args.ep.outf + (size_t)grow * args.N + n0 + c, acc, args.ep.accumulate);
        }
    } else if constexpr (KIND == TC_B4) {
#pragma unroll 1
        for (int c = 0; c < TC_BN; c += 32) {
            tmem_ld32(taddr + c, acc);
            if (row_ok && n0 + c < args.N) {
#pragma unroll
                for (int s = 0; s < 32; s += 8) {
                    float a8[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) a8[q] = acc[s + q];
                    store_bf16_run<8>(args.ep.out0 + (size_t)grow * args.ep.ldo + n0 + c + s, a8);
                }
            }
        }
    }
}

// ------------------------------------------------------------------------------------------ kernel
template <int KIND>
__global__ void __launch_bounds__(TcTraits<KIND>::THREADS, 1)
tc_grouped_gemm_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmA1,
                       const __grid_constant__ CUtensorMap tmB0, const __grid_constant__ CUtensorMap tmB1,
                       const __grid_constant__ CUtensorMap tmO0, const __grid_constant__ CUtensorMap tmO1,
                       const TcArgs args) {
    using Tr = TcTraits<KIND>;
    constexpr int TC_STAGES = Tr::STAGES;
    extern __shared__ uint8_t tc_smem_raw[];
    // 1024-byte alignment: the swizzle pattern is a function of address bits 7..9
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + TC_STAGES * TC_STAGE_BYTES);
    // bars[0..S) full, [S..2S) empty, [2S..2S+2) tmem_full, [2S+2..2S+4) tmem_empty
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * TC_STAGES + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bar_base = smem_u32(bars);
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (TC_STAGES + s); };
    auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * TC_STAGES + b); };
    auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * TC_STAGES + 2 + b); };

    if (threadIdx.x == 0) {
        for (int s = 0; s < TC_STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), Tr::EPI_WARPS); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tma_prefetch_desc(&tmA0); tma_prefetch_desc(&tmB0);
        if (Tr::PHASES == 2) tma_prefetch_desc(&tmA1);
        if (Tr::DUAL_B || Tr::SEL_B || Tr::PHASES == 2) tma_prefetch_desc(&tmB1);
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    int total_tiles;
    if constexpr (Tr::RAGGED_K) total_tiles = args.E * args.tiles_m_fixed * args.tiles_n;
    else total_tiles = (*args.n_mtiles) * args.tiles_n;

    if (warp == 0) {
        // ===================================================================== TMA producer
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0; bool alive = true;
            const uint64_t keep = l2_policy_evict_last();
            (void)keep;
            // the next tile's descriptor is fetched one tile ahead so that its latency is hidden
            TileInfo nxt = decode_tile<KIND>(args, min((int)blockIdx.x, max(total_tiles - 1, 0)));
            for (int t = blockIdx.x; t < total_tiles && alive; t += gridDim.x) {
                const TileInfo ti = nxt;
                if (t + (int)gridDim.x < total_tiles) nxt = decode_tile<KIND>(args, t + gridDim.x);
                if (ti.skip) continue;
                const int n0 = ti.nt * Tr::N_PER_TILE + (KIND == TC_VP ? args.n_base : 0);
                const int nkb = Tr::RAGGED_K ? (ti.rows + TC_BK - 1) / TC_BK : Tr::PHASES * args.kblocks;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, args.status, STATUS_WAIT_EMPTY)) {
                        alive = false; break;
                    }
                    const uint32_t fb = full_bar(stage);
                    mbar_expect_tx(fb, TC_STAGE_BYTES);
                    const uint32_t sA = smem_base + stage * TC_STAGE_BYTES;
                    const uint32_t sB = sA + TC_A_BYTES;
                    const int ph = Tr::PHASES > 1 ? kb / args.kblocks : 0;
                    const int k0 = (kb - ph * args.kblocks) * TC_BK;
                    if constexpr (!Tr::A_MN) {
                        tma_load_2d(sA, (KIND == TC_B4 && ph) ? &tmA1 : &tmA0, fb, k0, ti.row0);
                    } else {
                        // chunked map {64, rows, cols/64}: both 64-wide column chunks in one copy
                        tma_load_3d_hint(sA, &tmA0, fb, 0, ti.row0 + kb * TC_BK, ti.m0 >> 6, keep);
                    }
                    if constexpr (!Tr::B_MN) {
                        tma_load_3d(sB, ph ? &tmB1 : &tmB0, fb, k0 + (KIND == TC_VX ? args.kb_base : 0), n0, ti.e);
                    } else {
                        // chunked maps {64, rows, cols/64 [, E]}: the 64-wide column chunks of the tile arrive
                        // chunk-major in one copy per tensor (four chunks, or two each of two tensors)
                        if constexpr (Tr::B_WEIGHT) {
                            tma_load_4d(sB, &tmB0, fb, 0, k0, n0 >> 6, ti.e);
                            if constexpr (Tr::DUAL_B) tma_load_4d(sB + 2 * TC_CHUNK_BYTES, &tmB1, fb, 0, k0, n0 >> 6, ti.e);
                        } else {
                            const int krow = ti.row0 + kb * TC_BK;
                            tma_load_3d_hint(sB, (Tr::SEL_B && ti.sel) ? &tmB1 : &tmB0, fb, 0, krow, n0 >> 6, keep);
                        }
                    }
                    if (++stage == TC_STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ===================================================================== MMA issuer
        constexpr uint32_t idesc = make_idesc(Tr::A_MN, Tr::B_MN);
        // MN-major operand: 64-wide chunks are TC_CHUNK_BYTES apart (leading offset), groups of
        // 8 K rows are 1024 bytes apart (stride offset); K-major: 8-row groups 1024 bytes apart.
        constexpr uint32_t mn_lbo = TC_CHUNK_BYTES, mn_sbo = 1024u;
        int stage = 0; uint32_t phase = 0; int it = 0; bool alive = true;
        TileInfo nxt = decode_tile<KIND>(args, min((int)blockIdx.x, max(total_tiles - 1, 0)));
        if constexpr (!Tr::RAGGED_K) {
            // Token-row kinds: one thread runs the whole issue loop (wait, fence, four MMAs, commit) with
            // descriptors that only need the stage's start address added, so the tensor pipe's queue stays fed.
            if (lane == 0) {
                const uint64_t desc_a = smem_desc(0, 0, 1024);
                const uint64_t desc_b = Tr::B_MN ? smem_desc(0, mn_lbo, mn_sbo) : smem_desc(0, 0, 1024);
                constexpr uint32_t b_step = (Tr::B_MN ? 2048 : 32) >> 4;
                const int nkb = Tr::PHASES * args.kblocks;
                for (int t = blockIdx.x; t < total_tiles && alive; t += gridDim.x) {
                    if (t + (int)gridDim.x < total_tiles) nxt = decode_tile<KIND>(args, t + gridDim.x);
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
                        const uint32_t sA = smem_base + stage * TC_STAGE_BYTES;
                        const uint64_t da = desc_a | (uint64_t)((sA & 0x3ffffu) >> 4);
                        const uint64_t db = desc_b | (uint64_t)(((sA + TC_A_BYTES) & 0x3ffffu) >> 4);
#pragma unroll
                        for (int k4 = 0; k4 < TC_BK / 16; ++k4)
                            umma_bf16(d_tmem, da + k4 * 2, db + k4 * b_step, idesc, (kb | k4) != 0 ? 1u : 0u);
                        umma_commit(empty_bar(stage));
                        if (++stage == TC_STAGES) { stage = 0; phase ^= 1u; }
                    }
                    if (!alive) break;
                    umma_commit(tfull_bar(buf));
                    ++it;
                }
            }
        } else
        for (int t = blockIdx.x; t < total_tiles && alive; t += gridDim.x) {
            const TileInfo ti = nxt;
            if (t + (int)gridDim.x < total_tiles) nxt = decode_tile<KIND>(args, t + gridDim.x);
            if (ti.skip) continue;
            const int buf = it & 1;
            const uint32_t tphase = (uint32_t)(it >> 1) & 1u;
            if (!mbar_wait_warp(tempty_bar(buf), tphase ^ 1u, abort_flag, args.status, STATUS_WAIT_TMEM_EMPTY, lane)) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)buf * TC_BN;
            const int nkb = Tr::RAGGED_K ? (ti.rows + TC_BK - 1) / TC_BK : Tr::PHASES * args.kblocks;
            for (int kb = 0; kb < nkb; ++kb) {
                if (!mbar_wait_warp(full_bar(stage), phase, abort_flag, args.status, STATUS_WAIT_FULL, lane)) {
                    alive = false; break;
                }
                tc_fence_after();
                const uint32_t sA = smem_base + stage * TC_STAGE_BYTES;
                const uint32_t sB = sA + TC_A_BYTES;
                int n_k4 = TC_BK / 16;                   // MMAs (16 rows of K each) of this block
                if constexpr (Tr::RAGGED_K) {
                    // K tail: rows past the expert's end belong to the next expert (or are zero fill).  Whole
                    // groups of 16 such rows are simply not multiplied; the rest of the last group (at most 15
                    // rows) is cleared in both operands (2 chunks of A and 4 of B, one after the other in the
                    // stage), so that nothing of a neighbour, not even an Inf or a NaN, reaches this gradient.
                    const int valid = ti.rows - kb * TC_BK;
                    if (valid < TC_BK) {
                        n_k4 = (valid + 15) >> 4;
                        uint8_t* base = smem + stage * TC_STAGE_BYTES;
                        const int n16 = (n_k4 * 16 - valid) * 8; // 16-byte vectors per chunk to clear
                        for (int i = lane; i < n16; i += 32) {
                            const int off = (valid + (i >> 3)) * 128 + (i & 7) * 16;
#pragma unroll
                            for (int ch = 0; ch < TC_STAGE_BYTES / TC_CHUNK_BYTES; ++ch)
                                *reinterpret_cast<uint4*>(base + ch * TC_CHUNK_BYTES + off) = make_uint4(0, 0, 0, 0);
                        }
                        if (n16 > 0) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        __syncwarp();
                    }
                }
                if (lane == 0) {
#pragma unroll
                    for (int k4 = 0; k4 < TC_BK / 16; ++k4) {
                        if (k4 >= n_k4) break;
                        const uint64_t ad = Tr::A_MN ? smem_desc(sA + k4 * 2048, mn_lbo, mn_sbo)
                                                     : smem_desc(sA + k4 * 32, 0, 1024);
                        const uint64_t bd = Tr::B_MN ? smem_desc(sB + k4 * 2048, mn_lbo, mn_sbo)
                                                     : smem_desc(sB + k4 * 32, 0, 1024);
                        umma_bf16(d_tmem, ad, bd, idesc, (kb | k4) != 0 ? 1u : 0u);
                    }
                    umma_commit(empty_bar(stage));
                }
                __syncwarp();
                if (++stage == TC_STAGES) { stage = 0; phase ^= 1u; }
            }
            if (!alive) break;
            if (lane == 0) umma_commit(tfull_bar(buf));
            __syncwarp();
            ++it;
        }
    } else {
        // ===================================================================== epilogue (4 warps)
        const int quarter = warp & 3;            // TMEM lanes 32*quarter .. +31 belong to this warp
        const int r = quarter * 32 + lane;       // row of the tile owned by this thread
        const int half = (warp - 2) >> 2;        // eight-warp epilogue: columns [128*half, 128*half + 128)
        int sbuf = 0;                            // weight gradients: store box in use
        int it = 0;
        TileInfo nxt = decode_tile<KIND>(args, min((int)blockIdx.x, max(total_tiles - 1, 0)));
        for (int t = blockIdx.x; t < total_tiles; t += gridDim.x) {
            const TileInfo ti = nxt;
            if (t + (int)gridDim.x < total_tiles) nxt = decode_tile<KIND>(args, t + gridDim.x);
            const int n0 = ti.nt * Tr::N_PER_TILE + (KIND == TC_VP ? args.n_base : 0);
            if constexpr (Tr::RAGGED_K) {
                if (ti.skip) {
                    // expert without rows: its gradient is zero (or unchanged when accumulating)
                    if (!args.ep.accumulate && !args.keep_empty && half == 0 && ti.m0 + r < args.Mfix) {
                        const size_t ro = ((size_t)ti.e * args.Mfix + ti.m0 + r) * args.N;
                        float* dst = (Tr::SEL_B && ti.sel) ? args.outf1 : args.ep.outf;
                        for (int c = 0; c < TC_BN; c += 4)
                            if (n0 + c < args.N) *reinterpret_cast<float4*>(dst + ro + n0 + c) = make_float4(0, 0, 0, 0);
                    }
                    continue;
                }
            }
            const int buf = it & 1;
            const uint32_t tphase = (uint32_t)(it >> 1) & 1u;
            bool ready = mbar_wait_warp(tfull_bar(buf), tphase, abort_flag, args.status, STATUS_WAIT_TMEM_FULL, lane);
            // the four warps of a column half meet at named barriers below: they give up together or not at all
            if constexpr (Tr::RAGGED_K) ready = bar_vote_all(1 + half, 128, ready);
            if (!ready) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)buf * TC_BN;
            const bool row_ok = Tr::RAGGED_K ? (ti.m0 + r < args.Mfix) : (r < ti.rows);
            const int grow = ti.row0 + r;        // ragged M: global row
            float acc[32];
            (void)acc;

            if constexpr (!Tr::RAGGED_K) {
                tc_epilogue_rows<KIND>(args, taddr, row_ok, grow, n0, ti.nt);
            } else {
                // Weight-gradient tile.  Each warp first reads its 32 rows x 128 columns from TMEM in one go and
                // hands the accumulator back, so that the MMA warp can run two tiles ahead of the stores.  Then
                // the four warps of a column half stage 128 rows x 32 fp32 columns in shared memory (128-byte
                // rows, 16-byte chunks XOR-swizzled by row: the layout of a 128B-swizzle tensor map,
                // conflict-free for one-row-per-lane writes) and one thread hands the 16 KiB box to TMA, which
                // writes whole 128-byte lines and clips rows >= Mfix and columns >= N.  Two boxes per half: one
                // is being read by the copy engine while the next one is staged.
                uint8_t* gbase = smem + TC_STAGES * TC_STAGE_BYTES + TC_BAR_BYTES + half * 32768;
                const CUtensorMap* mo = (Tr::SEL_B && ti.sel) ? &tmO1 : &tmO0;
                const bool issuer = (quarter == 0 && lane == 0);
                const uint64_t stream_out = l2_policy_evict_first();
                const int gbar = 1 + half;               // named barrier of this half's 128 threads
                float a0[32], a1[32], a2[32], a3[32];
                tmem_ld32_nowait(taddr + half * 128, a0);
                tmem_ld32_nowait(taddr + half * 128 + 32, a1);
                tmem_ld32_nowait(taddr + half * 128 + 64, a2);
                tmem_ld32_nowait(taddr + half * 128 + 96, a3);
                tmem_ld_wait4(a0, a1, a2, a3);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(tempty_bar(buf));
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    uint8_t* box = gbase + (sbuf & 1) * 16384;
                    uint8_t* rowp = box + (quarter * 32 + lane) * 128;
                    const float(&v)[32] = cc == 0 ? a0 : cc == 1 ? a1 : cc == 2 ? a2 : a3;
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        *reinterpret_cast<float4*>(rowp + ((j ^ (lane & 7)) << 4)) =
                            make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    // One barrier per step.  Before it the issuing thread makes sure that the box handed over one
                    // step ago has been read, so after it everyone may overwrite that box (the next step's).
                    if (issuer) tma_store_wait_read<0>();
                    asm volatile("bar.sync %0, 128;" ::"r"(gbar) : "memory");
                    if (issuer) {
                        const int gcol = n0 + half * 128 + 32 * cc;
                        if (gcol < args.N) {
                            if (args.ep.accumulate) tma_reduce_add_3d(mo, smem_u32(box), gcol, ti.m0, ti.e);
                            else tma_store_3d_hint(mo, smem_u32(box), gcol, ti.m0, ti.e, stream_out);
                        }
                        tma_store_commit();
                    }
                    ++sbuf;
                }
                ++it;
                continue;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(buf));
            ++it;
        }
        if (Tr::RAGGED_K && quarter == 0 && lane == 0) tma_store_wait_all();   // boxes read before the CTA exits
        (void)sbuf;
    }

    // ------------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // let copies that are still in flight land before the shared memory is released
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// Merge of the per-tile (max, sum) pairs of a row: lse = M + log sum_i s_i exp(m_i - M); the
// log-likelihood is the target's logit minus lse.  Fixed order: reproducible.
__global__ void vocab_lse_merge_kernel(const float2* __restrict__ part, const float* __restrict__ ylab,
                                       float* __restrict__ loss, float* __restrict__ lse, int N, int ntiles) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= N) return;
    float M = -INFINITY;
    for (int i = 0; i < ntiles; ++i) M = fmaxf(M, part[(size_t)i * N + n].x);
    float S = 0.0f;
    for (int i = 0; i < ntiles; ++i) {
        const float2 p = part[(size_t)i * N + n];
        S += p.y * expf(p.x - M);
    }
    const float l = M + logf(S);
    if (lse) lse[n] = l;
    loss[n] = ylab[n] - l;
}

// fp32 -> bf16 of a dense array (8 elements per thread; n a multiple of 8)
__global__ void f32_to_bf16_kernel(const float4* __restrict__ src, uint4* __restrict__ dst, size_t n8) {
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n8; i += (size_t)gridDim.x * blockDim.x) {
        const float4 a = src[2 * i], b = src[2 * i + 1];
        const float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
        store_bf16_run<8>(reinterpret_cast<bf16*>(dst + i), v);
    }
}

// ------------------------------------------------------------------------------------------ host
struct TcPlan {
    int sm_count;
    mop_moe_shape s;
    void* encode;   // cuTensorMapEncodeTiled
    int pairs;      // schedule of the token-row kinds (see gemm_host.cuh)
    long long rows_override;   // > 0: the row buffers of this call hold this many rows (an expert chunk), not T*k
    int fwd_tn;     // GEMMs on the tokens-on-N kernels: bit 0 up-projection, bit 1 down-projection, bit 2 dgrad of the up-projection, bit 3 dgrad of the down-projection
    Profiler* prof;
};

struct TcFwdArgs {
    const bf16* Xp; const int32_t* offsets; const int32_t* row_src; const float* gate;
    const bf16 *W_gate, *W_up, *W_down;
    bf16 *G_save, *U_save, *H, *Yp;
    const bf16* x_gather;   // non-null: the up-projection gathers its rows from x [T, d] and Xp is unused
};
struct TcBwdArgs {
    const bf16 *dYp, *Xp, *G_save, *U_save, *H;
    const int32_t* offsets; const int32_t* row_src; const float* gate;
    const bf16 *W_gate, *W_up, *W_down;
    bf16 *dG, *dU, *gH, *dXp; float* part;
    float *dW_gate, *dW_up, *dW_down; int accumulate;
    int keep_empty;   // experts without rows (in this call's offsets) keep their gradients: expert-chunked backward
};

inline bool tc_shape_supported(int d, int f) { return d % 64 == 0 && f % 64 == 0; }
inline uint64_t tc_rows(const TcPlan* p) {
    return p->rows_override > 0 ? (uint64_t)p->rows_override : (uint64_t)p->s.T * p->s.k;
}
inline size_t tc_tile_table_bytes(int M, int E) { return ((size_t)M / TC_BM + E + 8) * sizeof(int4) + 256; }

typedef CUresult (*tc_encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                 const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

template <int KIND>
inline mop_status tc_set_smem() {
    return cudaFuncSetAttribute(tc_grouped_gemm_kernel<KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                TcTraits<KIND>::SMEM_BYTES) == cudaSuccess
               ? MOP_OK : MOP_ERR_CUDA;
}

inline mop_status tc_plan_init(TcPlan* p, const mop_moe_shape& s, int sm_count, Profiler* prof) {
    p->sm_count = sm_count;
    p->prof = prof;
    p->s = s;
    p->rows_override = 0;
    cudaDriverEntryPointQueryResult q;
    void* fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn ||
        q != cudaDriverEntryPointSuccess)
        return MOP_ERR_CUDA;
    p->encode = fn;
    mop_status r;
    if ((r = tc_set_smem<TC_F1>()) != MOP_OK) return r;
    if ((r = tc_set_smem<TC_F2>()) != MOP_OK) return r;
    if ((r = tc_set_smem<TC_B2>()) != MOP_OK) return r;
    if ((r = tc_set_smem<TC_B4>()) != MOP_OK) return r;
    if ((r = tc_set_smem<TC_WD>()) != MOP_OK) return r;
    if ((r = tc_set_smem<TC_WGU>()) != MOP_OK) return r;
    if ((r = tc_set_smem<TC_VL>()) != MOP_OK) return r;
    if ((r = tc_set_smem<TC_VP>()) != MOP_OK) return r;
    if ((r = tc_set_smem<TC_VX>()) != MOP_OK) return r;
    return MOP_OK;
}

// 2-D map over a dense [rows, cols] bf16 matrix; box = {64 cols, box_rows}.
inline bool tc_map_2d(const TcPlan* p, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols,
                      uint32_t box_rows) {
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t es[2] = {1, 1};
    return reinterpret_cast<tc_encode_fn>(p->encode)(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base),
                                                     dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// 3-D map over a dense [E, rows, cols] bf16 tensor; box = {64 cols, box_rows, 1}.
inline bool tc_map_3d(const TcPlan* p, CUtensorMap* m, const void* base, uint64_t E, uint64_t rows, uint64_t cols,
                      uint32_t box_rows) {
    const cuuint64_t dims[3] = {cols, rows, E};
    const cuuint64_t strides[2] = {cols * 2, rows * cols * 2};
    const cuuint32_t box[3] = {64, box_rows, 1};
    const cuuint32_t es[3] = {1, 1, 1};
    return reinterpret_cast<tc_encode_fn>(p->encode)(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base),
                                                     dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Chunked maps for MN-major operands.  A dense [rows, cols] (or [E, rows, cols]) bf16 matrix is viewed
// as {64 columns, rows, cols/64 chunks [, E]} so that ONE copy brings `chunks` 64-wide column chunks
// of 64 rows each, chunk-major in shared memory: exactly the layout the MMA descriptor expects
// (chunk pitch 8 KiB, 128-byte swizzled rows).  cols must be a multiple of 64.
inline bool tc_map_chunked_2d(const TcPlan* p, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols,
                              uint32_t chunks) {
    const cuuint64_t dims[3] = {64, rows, cols / 64};
    const cuuint64_t strides[2] = {cols * 2, 128};
    const cuuint32_t box[3] = {64, 64, chunks};
    const cuuint32_t es[3] = {1, 1, 1};
    return reinterpret_cast<tc_encode_fn>(p->encode)(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base),
                                                     dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
inline bool tc_map_chunked_3d(const TcPlan* p, CUtensorMap* m, const void* base, uint64_t E, uint64_t rows,
                              uint64_t cols, uint32_t chunks, uint32_t box_rows = 64) {
    const cuuint64_t dims[4] = {64, rows, cols / 64, E};
    const cuuint64_t strides[3] = {cols * 2, 128, rows * cols * 2};
    const cuuint32_t box[4] = {64, box_rows, chunks, 1};
    const cuuint32_t es[4] = {1, 1, 1, 1};
    return reinterpret_cast<tc_encode_fn>(p->encode)(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base),
                                                     dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same views over a column block of a wider matrix: `cols` columns starting at `base`, rows
// `pitch` elements apart (pitch * element size and base must be multiples of 16 bytes).
inline bool tc_map_2d_pitch(const TcPlan* p, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols,
                            uint64_t pitch, uint32_t box_rows) {
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {pitch * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t es[2] = {1, 1};
    return reinterpret_cast<tc_encode_fn>(p->encode)(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base),
                                                     dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
inline bool tc_map_chunked_2d_pitch(const TcPlan* p, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols,
                                    uint64_t pitch, uint32_t chunks) {
    const cuuint64_t dims[3] = {64, rows, cols / 64};
    const cuuint64_t strides[2] = {pitch * 2, 128};
    const cuuint32_t box[3] = {64, 64, chunks};
    const cuuint32_t es[3] = {1, 1, 1};
    return reinterpret_cast<tc_encode_fn>(p->encode)(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base),
                                                     dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
inline bool tc_map_out_f32_pitch(const TcPlan* p, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols,
                                 uint64_t pitch) {
    const cuuint64_t dims[3] = {cols, rows, 1};
    const cuuint64_t strides[2] = {pitch * 4, rows * pitch * 4};
    const cuuint32_t box[3] = {32, 128, 1};
    const cuuint32_t es[3] = {1, 1, 1};
    return reinterpret_cast<tc_encode_fn>(p->encode)(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base),
                                                     dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                                                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 3-D map over a dense [E, rows, cols] fp32 tensor for stores; box = {32 cols, 128 rows, 1}.
inline bool tc_map_out_f32(const TcPlan* p, CUtensorMap* m, const void* base, uint64_t E, uint64_t rows,
                           uint64_t cols) {
    const cuuint64_t dims[3] = {cols, rows, E};
    const cuuint64_t strides[2] = {cols * 4, rows * cols * 4};
    const cuuint32_t box[3] = {32, 128, 1};
    const cuuint32_t es[3] = {1, 1, 1};
    return reinterpret_cast<tc_encode_fn>(p->encode)(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base),
                                                     dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                                                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int KIND>
inline mop_status tc_launch(const TcPlan* p, const char* name, const CUtensorMap& a0, const CUtensorMap& a1,
                            const CUtensorMap& b0, const CUtensorMap& b1, const CUtensorMap& o0, const CUtensorMap& o1,
                            const TcArgs& args, cudaStream_t st) {
    p->prof->begin(name, st);
    tc_grouped_gemm_kernel<KIND><<<p->sm_count, TcTraits<KIND>::THREADS, TcTraits<KIND>::SMEM_BYTES, st>>>(
        a0, a1, b0, b1, o0, o1, args);
    p->prof->end(st);
    return cudaGetLastError() == cudaSuccess ? MOP_OK : MOP_ERR_CUDA;
}

inline TcArgs tc_base_args(const TcPlan* p, const int32_t* offsets, int32_t* tiles, int32_t* status) {
    TcArgs a{};
    a.offsets = offsets;
    a.n_mtiles = tiles;                                   // first word of the table area
    a.mtiles = reinterpret_cast<const int4*>(tiles + 64); // entries start 256 bytes in
    a.E = p->s.E;
    a.status = status;
    return a;
}

inline mop_status tc_build_tiles(const TcPlan* p, const int32_t* offsets, int32_t* tiles, cudaStream_t st) {
    p->prof->begin("tc_build_mtiles", st);
    tc_build_mtiles_kernel<<<1, 1024, 0, st>>>(offsets, p->s.E, reinterpret_cast<int4*>(tiles + 64), tiles);
    p->prof->end(st);
    return cudaGetLastError() == cudaSuccess ? MOP_OK : MOP_ERR_CUDA;
}

}  // namespace mop
