// Tensor-core (tcgen05 / TMEM / TMA) grouped GEMMs -- interface.
#pragma once
#include "../../include/mop_moe.h"
#include "epilogue.cuh"

namespace mop {

struct TcPlan { int sm_count; mop_moe_shape s; };

struct TcFwdArgs {
    const bf16* Xp; const int32_t* offsets; const int32_t* row_src; const float* gate;
    const bf16 *W_gate, *W_up, *W_down;
    bf16 *G_save, *U_save, *H, *Yp;
};
struct TcBwdArgs {
    const bf16 *dYp, *Xp, *G_save, *U_save, *H;
    const int32_t* offsets; const int32_t* row_src; const float* gate;
    const bf16 *W_gate, *W_up, *W_down;
    bf16 *dG, *dU, *gH, *dXp; float* part;
    float *dW_gate, *dW_up, *dW_down; int accumulate;
};

inline bool tc_shape_supported(int d, int f) { (void)d; (void)f; return false; }
inline size_t tc_tile_table_bytes(int M, int E) { (void)M; (void)E; return 256; }
inline mop_status tc_plan_init(TcPlan*, const mop_moe_shape&, int) { return MOP_OK; }
inline mop_status tc_ffn_fwd(TcPlan*, const TcFwdArgs&, int32_t*, int32_t*, cudaStream_t, int*) { return MOP_ERR_UNSUPPORTED; }
inline mop_status tc_ffn_bwd(TcPlan*, const TcBwdArgs&, int32_t*, int32_t*, cudaStream_t, int*, int*) { return MOP_ERR_UNSUPPORTED; }

}  // namespace mop
