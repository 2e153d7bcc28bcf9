// Host-side orchestration of the tensor-core grouped GEMMs: tensor maps, tile tables, launches.
#pragma once
#include "gemm_tc.cuh"
#include "gemm_tc2.cuh"
#include "gemm_tn.cuh"

namespace mop {

// Schedules of the token-row kinds (TcPlan::pairs): 0 = one-CTA kernel on 128-row tiles; 1 = two-CTA
// kernel on 256-row pairs (the last pair of an expert may be partly empty); 2 = mixed: full pairs on
// the two-CTA kernel, the remaining < 256 rows of each expert on the one-CTA kernel.
inline size_t tc_tables_bytes(int M, int E) { return 3 * tc_tile_table_bytes(M, E); }

inline mop_status tc_build_row_tiles(const TcPlan* p, const int32_t* offsets, int32_t* tiles, cudaStream_t st) {
    int32_t* tiles2 = tiles + tc_tile_table_bytes(p->s.T * p->s.k, p->s.E) / 4;
    if (p->pairs == 2) return tc2_build_mixed(p, offsets, tiles, tiles2, st);
    if (p->pairs == 1) return tc2_build_tiles(p, offsets, tiles, st);
    return tc_build_tiles(p, offsets, tiles, st);
}

// One token-row GEMM under the plan's schedule.  b0p/b1p are the B maps boxed for a pair CTA (128 N
// rows for K-major weights); b0/b1 those of the one-CTA kernel.
template <int KIND>
inline mop_status tc_rows_gemm(const TcPlan* p, const char* name, const char* name2, const CUtensorMap& a0,
                               const CUtensorMap& a1, const CUtensorMap& b0, const CUtensorMap& b1,
                               const CUtensorMap& b0p, const CUtensorMap& b1p, TcArgs g, int32_t* tiles,
                               cudaStream_t st, int* launches) {
    mop_status r;
    if (p->pairs >= 1) {
        if ((r = tc2_launch<KIND>(p, name2, a0, a1, b0p, b1p, g, st)) != MOP_OK) return r;
        ++*launches;
    }
    if (p->pairs != 1) {
        if (p->pairs == 2) {
            int32_t* tiles2 = tiles + tc_tile_table_bytes(p->s.T * p->s.k, p->s.E) / 4;
            g.n_mtiles = tiles2;
            g.mtiles = reinterpret_cast<const int4*>(tiles2 + 64);
        }
        if ((r = tc_launch<KIND>(p, name, a0, a1, b0, b1, a0, a0, g, st)) != MOP_OK) return r;
        ++*launches;
    }
    return MOP_OK;
}

inline mop_status tc_ffn_fwd_impl(TcPlan* p, const TcFwdArgs& a, int32_t* tiles, int32_t* status, cudaStream_t st,
                                  int* launches, bool with_down);

inline mop_status tc_ffn_fwd(TcPlan* p, const TcFwdArgs& a, int32_t* tiles, int32_t* status, cudaStream_t st,
                             int* launches) {
    return tc_ffn_fwd_impl(p, a, tiles, status, st, launches, true);
}
// Up-projection + SwiGLU alone (the backward's recomputation of G, U, H).
inline mop_status tc_up_only(TcPlan* p, const TcFwdArgs& a, int32_t* tiles, int32_t* status, cudaStream_t st,
                             int* launches) {
    return tc_ffn_fwd_impl(p, a, tiles, status, st, launches, false);
}

inline mop_status tc_ffn_fwd_impl(TcPlan* p, const TcFwdArgs& a, int32_t* tiles, int32_t* status, cudaStream_t st,
                                  int* launches, bool with_down) {
    const mop_moe_shape& s = p->s;
    const uint64_t M = tc_rows(p);
    mop_status r;
    // Tokens-on-N kernels: fwd_tn bit 0 = up-projection, bit 1 = down-projection (see tc_plan_policy)
    const bool gather = a.x_gather != nullptr;
    const bool tn_f1 = gather || (p->fwd_tn & 1), tn_f2 = p->fwd_tn & 2;
    int32_t* ttiles_fwd = tiles + 2 * (tc_tile_table_bytes(s.T * s.k, s.E) / 4);
    if ((tn_f1 != tn_f2) && p->pairs == 0) {   // one GEMM on each kind of kernel: both tables in one launch
        if ((r = build_both_tiles(p, a.offsets, tiles, ttiles_fwd, st)) != MOP_OK) return r;
        ++*launches;
    } else {
        if (tn_f1 || tn_f2) {
            if ((r = tn_build_tiles(p, a.offsets, ttiles_fwd, st)) != MOP_OK) return r;
            ++*launches;
        }
        if (!tn_f1 || !tn_f2) {
            if ((r = tc_build_row_tiles(p, a.offsets, tiles, st)) != MOP_OK) return r;
            ++*launches;
        }
    }
    // N-major weights as chunked maps: one-CTA tiles take 2 chunks per tensor (gate | up) or 4 (down);
    // a pair CTA takes 2 chunks
    CUtensorMap mXp, mWg, mWu, mH, mWd, mWdp;
    if ((!tn_f1 && !tc_map_2d(p, &mXp, a.Xp, M, s.d, 128)) || !tc_map_chunked_3d(p, &mWg, a.W_gate, s.E, s.d, s.f, 2) ||
        !tc_map_chunked_3d(p, &mWu, a.W_up, s.E, s.d, s.f, 2) || !tc_map_2d(p, &mH, a.H, M, s.f, 128) ||
        !tc_map_chunked_3d(p, &mWd, a.W_down, s.E, s.f, s.d, 4) ||
        !tc_map_chunked_3d(p, &mWdp, a.W_down, s.E, s.f, s.d, 2))
        return MOP_ERR_CUDA;
    if (gather) {
        if ((r = tn_up_swiglu_gather(p, a.x_gather, a, tiles + 2 * (tc_tile_table_bytes(s.T * s.k, s.E) / 4), status, st)) != MOP_OK) return r;
        ++*launches;
    } else if (tn_f1) {
        if ((r = tn_up_swiglu(p, a, tiles + 2 * (tc_tile_table_bytes(s.T * s.k, s.E) / 4), status, st)) != MOP_OK) return r;
        ++*launches;
    } else {   // F1: [G|U] = Xp [W_gate | W_up], SwiGLU epilogue
        TcArgs g = tc_base_args(p, a.offsets, tiles, status);
        g.tiles_n = ceil_div(s.f, 128); g.kblocks = ceil_div(s.d, TC_BK); g.N = s.f;
        g.ep.out0 = a.H; g.ep.out1 = a.G_save; g.ep.out2 = a.U_save; g.ep.ldo = s.f; g.ep.M_total = (int)M;
        if ((r = tc_rows_gemm<TC_F1>(p, "gemm_up_swiglu", "gemm_up_swiglu_2cta", mXp, mXp, mWg, mWu, mWg, mWu, g, tiles, st, launches)) != MOP_OK)
            return r;
    }
    if (!with_down) return MOP_OK;
    if (tn_f2) {
        if ((r = tn_down_gate(p, a, tiles + 2 * (tc_tile_table_bytes(s.T * s.k, s.E) / 4), status, st)) != MOP_OK) return r;
        ++*launches;
    } else {   // F2: Yp = gate * (H W_down)
        TcArgs g = tc_base_args(p, a.offsets, tiles, status);
        g.tiles_n = ceil_div(s.d, 256); g.kblocks = ceil_div(s.f, TC_BK); g.N = s.d;
        g.ep.out0 = a.Yp; g.ep.gate = a.gate; g.ep.row_src = a.row_src; g.ep.ldo = s.d; g.ep.M_total = (int)M;
        if ((r = tc_rows_gemm<TC_F2>(p, "gemm_down_gate", "gemm_down_gate_2cta", mH, mH, mWd, mWd, mWdp, mWdp, g, tiles, st, launches)) != MOP_OK)
            return r;
    }
    return MOP_OK;
}

inline mop_status tc_ffn_bwd(TcPlan* p, const TcBwdArgs& a, int32_t* tiles, int32_t* status, cudaStream_t st,
                             int* launches, int* ntile_part) {
    const mop_moe_shape& s = p->s;
    const uint64_t M = tc_rows(p);
    *ntile_part = ceil_div(s.f, 256);
    if (M == 0) {
        // no rows at all: gradients are zero unless accumulating
        if (!a.accumulate && !a.keep_empty) {
            const size_t n = (size_t)s.E * s.d * s.f * 4;
            if (cudaMemsetAsync(a.dW_gate, 0, n, st) != cudaSuccess || cudaMemsetAsync(a.dW_up, 0, n, st) != cudaSuccess ||
                cudaMemsetAsync(a.dW_down, 0, n, st) != cudaSuccess)
                return MOP_ERR_CUDA;
        }
        return MOP_OK;
    }
    mop_status r;
    if ((p->fwd_tn & 12) != 12) {   // row tiles of the tokens-on-M data gradients (the weight gradients need none)
        if ((r = tc_build_row_tiles(p, a.offsets, tiles, st)) != MOP_OK) return r;
        ++*launches;
    }
    CUtensorMap mWdKp, mWgKp, mWuKp;   // K-major weight maps boxed for a pair CTA (128 N rows)
    if (!tc_map_3d(p, &mWdKp, a.W_down, s.E, s.f, s.d, 128) || !tc_map_3d(p, &mWgKp, a.W_gate, s.E, s.d, s.f, 128) ||
        !tc_map_3d(p, &mWuKp, a.W_up, s.E, s.d, s.f, 128))
        return MOP_ERR_CUDA;
    CUtensorMap mdYpA, mWdK, mdG, mdU, mWgK, mWuK, mgH, mdYpB, mXpA, mdGB, mdUB, moWd, moWg, moWu;
    if (!tc_map_out_f32(p, &moWd, a.dW_down, s.E, s.f, s.d) || !tc_map_out_f32(p, &moWg, a.dW_gate, s.E, s.d, s.f) ||
        !tc_map_out_f32(p, &moWu, a.dW_up, s.E, s.d, s.f))
        return MOP_ERR_CUDA;
    if (!tc_map_2d(p, &mdYpA, a.dYp, M, s.d, 128) || !tc_map_3d(p, &mWdK, a.W_down, s.E, s.f, s.d, 256) ||
        !tc_map_2d(p, &mdG, a.dG, M, s.f, 128) || !tc_map_2d(p, &mdU, a.dU, M, s.f, 128) ||
        !tc_map_3d(p, &mWgK, a.W_gate, s.E, s.d, s.f, 256) || !tc_map_3d(p, &mWuK, a.W_up, s.E, s.d, s.f, 256) ||
        !tc_map_chunked_2d(p, &mgH, a.gH, M, s.f, 2) || !tc_map_chunked_2d(p, &mdYpB, a.dYp, M, s.d, 4) ||
        !tc_map_chunked_2d(p, &mXpA, a.Xp, M, s.d, 2) || !tc_map_chunked_2d(p, &mdGB, a.dG, M, s.f, 4) ||
        !tc_map_chunked_2d(p, &mdUB, a.dU, M, s.f, 4))
        return MOP_ERR_CUDA;
    int32_t* ttiles = tiles + 2 * (tc_tile_table_bytes(s.T * s.k, s.E) / 4);
    if (p->fwd_tn & 12) {
        if ((r = tn_build_tiles(p, a.offsets, ttiles, st)) != MOP_OK) return r;
        ++*launches;
    }
    if (p->fwd_tn & 8) {   // B2 on the tokens-on-N kernel: one dgate partial per 32 columns of f
        *ntile_part = ceil_div(s.f, 32);
        if ((r = tn_dgrad_down(p, a, ttiles, status, st)) != MOP_OK) return r;
        ++*launches;
    } else {   // B2: dHu = dYp W_down^T, SwiGLU backward epilogue
        TcArgs g = tc_base_args(p, a.offsets, tiles, status);
        g.tiles_n = ceil_div(s.f, 256); g.kblocks = ceil_div(s.d, TC_BK); g.N = s.f;
        g.ep.out0 = a.dG; g.ep.out1 = a.dU; g.ep.out2 = a.gH; g.ep.in0 = a.G_save; g.ep.in1 = a.U_save; g.ep.in2 = a.H;
        g.ep.gate = a.gate; g.ep.row_src = a.row_src; g.ep.part = a.part; g.ep.ldo = s.f; g.ep.M_total = (int)M;
        if ((r = tc_rows_gemm<TC_B2>(p, "gemm_dgrad_down_dswiglu", "gemm_dgrad_down_dswiglu_2cta", mdYpA, mdYpA, mWdK, mWdK, mWdKp, mWdKp, g, tiles, st,
                                     launches)) != MOP_OK)
            return r;
    }
    if (p->fwd_tn & 4) {   // B4 on the tokens-on-N kernel
        if ((r = tn_dgrad_gate_up(p, a, ttiles, status, st)) != MOP_OK) return r;
        ++*launches;
    } else {   // B4: dXp = dG W_gate^T + dU W_up^T
        TcArgs g = tc_base_args(p, a.offsets, tiles, status);
        g.tiles_n = ceil_div(s.d, 256); g.kblocks = ceil_div(s.f, TC_BK); g.N = s.d;
        g.ep.out0 = a.dXp; g.ep.ldo = s.d; g.ep.M_total = (int)M;
        if ((r = tc_rows_gemm<TC_B4>(p, "gemm_dgrad_gate_up", "gemm_dgrad_gate_up_2cta", mdG, mdU, mWgK, mWuK, mWgKp, mWuKp, g, tiles, st,
                                     launches)) != MOP_OK)
            return r;
    }
    {   // WD: dW_down[e] = (gate H)_e^T dYp_e
        TcArgs g = tc_base_args(p, a.offsets, tiles, status);
        g.tiles_n = ceil_div(s.d, 256); g.tiles_m_fixed = ceil_div(s.f, TC_BM); g.Mfix = s.f; g.N = s.d;
        g.ep.outf = a.dW_down; g.ep.accumulate = a.accumulate; g.keep_empty = a.keep_empty;
        if ((r = tc_launch<TC_WD>(p, "gemm_wgrad_down", mgH, mgH, mdYpB, mdYpB, moWd, moWd, g, st)) != MOP_OK) return r;
        ++*launches;
    }
    {   // WGU: dW_gate[e] = Xp_e^T dG_e and dW_up[e] = Xp_e^T dU_e: per m-block the n-tiles of dW_gate, then those of dW_up
        TcArgs g = tc_base_args(p, a.offsets, tiles, status);
        g.tiles_n = 2 * ceil_div(s.f, 256); g.tiles_m_fixed = ceil_div(s.d, TC_BM); g.Mfix = s.d; g.N = s.f;
        g.ep.outf = a.dW_gate; g.outf1 = a.dW_up; g.ep.accumulate = a.accumulate; g.keep_empty = a.keep_empty;
        if ((r = tc_launch<TC_WGU>(p, "gemm_wgrad_gate_up", mXpA, mXpA, mdGB, mdUB, moWg, moWu, g, st)) != MOP_OK) return r;
        ++*launches;
    }
    return MOP_OK;
}

}  // namespace mop
