// C ABI of the routed-expert layer: argument checks, workspace, launches.  See include/mop_moe.h
// for the contract of every entry point.
#include "../../include/mop_moe.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <mutex>
#include <new>

#include "common.cuh"
#include "epilogue.cuh"
#include "gemm_scalar.cuh"
#include "gemm_host.cuh"
#include "gemm_rs.cuh"
#include "permute.cuh"
#include "route.cuh"

using namespace mop;

struct mop_ctx {
    mop_moe_shape s;
    int device;
    int sm_count;
    int64_t launches;
    bool tensor_ok;      // shape admits the tensor-core kernels
    // workspace (one allocation)
    char* ws;
    size_t ws_bytes;
    float* z;            // [T,E] logits
    int32_t* partial;    // [units,E] histogram partials -> unit bases
    int32_t* tiles;      // tile tables of the grouped GEMMs
    int32_t* status;     // device status word
    float* part;         // [ntile_max, M] partial dot products for dgate
    bf16 *dYp, *dG, *dU, *gH, *dXp;  // backward intermediates
    bf16 *rG, *rU, *rH;              // recompute-in-backward buffers (activation checkpointing)
    float *dz_sel, *dz_row, *wrT;    // router backward: dz per assignment / per permuted row; W_r^T [E,d]
    // tensor-core scoring path: bf16 pieces of W_r [3,d,E], W_r^T [E,d], column-norm partials, ||x_t||, scalars
    // (wmax, statistics), the {0, T} offsets and the 128-row tile table of the dense logit GEMM
    bool fast_route;
    cudaStream_t fr_stream;          // the row norms of x are taken beside the logit GEMM
    cudaEvent_t fr_fork, fr_join;
    bf16* fr_pieces;
    float *fr_wrT, *fr_colsq, *fr_xnorm, *fr_scal, *fr_wsq, *fr_z1;
    int32_t* fr_todo;
    int fr_rblocks;          // resident blocks of the resolving pass
    // host-buffer entry point scratch
    bf16 *hx, *hXp, *hH, *hYp, *hY, *hG, *hU, *hdY, *hdX;
    int32_t *hidx, *hcounts, *hoffsets, *hperm, *hsrc;
    float *hgate, *hdgate;
    cudaStream_t copy_stream;            // host-buffer entry points: copies that overlap the kernels
    cudaEvent_t ev_in, ev_mid, ev_out;
    // pipelined host entry points (host_io = 2): the second set of the buffers that copies touch,
    // a stream for device-to-host copies, and per-slot events
    bf16 *px[2], *pY[2], *pdY[2], *pdX[2];
    int32_t* pidx[2];
    float *pgate[2], *pdgate[2];
    cudaStream_t out_stream;
    cudaEvent_t ev_x[2], ev_dy[2], ev_fwd[2], ev_done[2], ev_drained[2];
    uint64_t host_steps;
    TcPlan plan;
    Profiler prof;
    unsigned long long guard_off[96];    // guard bands of the workspace (see make_layout)
    int n_guards;
};

namespace {

inline size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }

// Every region of the workspace is followed (and the first one preceded) by a guard band that no kernel
// may touch: mop_debug_guard_arm fills the bands with a pattern, mop_debug_guard_check counts the bytes
// that no longer hold it.  This is how writes past the end of a workspace buffer are caught in tests.
constexpr size_t GUARD_BYTES = 4096;
constexpr int MAX_GUARDS = 96;
constexpr uint32_t GUARD_PATTERN = 0xA5C3A5C3u;

struct Layout {
    size_t z, partial, tiles, status, part, dYp, dG, dU, gH, dXp, dz_sel, dz_row, wrT, rG, rU, rH;
    size_t fr_pieces, fr_wrT, fr_colsq, fr_xnorm, fr_scal, fr_wsq, fr_todo, fr_z1;
    size_t hx, hXp, hH, hYp, hY, hidx, hcounts, hoffsets, hperm, hsrc, hgate;
    size_t hG, hU, hdY, hdX, hdgate;
    size_t qx, qY, qidx, qgate, qdY, qdX, qdgate;   // second slot of the pipelined host entry points
    size_t total;
    size_t guard[MAX_GUARDS];                       // offsets of the guard bands
    int n_guards;
};

struct GuardList { unsigned long long off[MAX_GUARDS]; int n; };

__global__ void guard_fill_kernel(char* ws, GuardList g) {
    uint32_t* band = reinterpret_cast<uint32_t*>(ws + g.off[blockIdx.x]);
    for (int i = threadIdx.x; i < (int)(GUARD_BYTES / 4); i += blockDim.x) band[i] = GUARD_PATTERN;
}
__global__ void guard_check_kernel(const char* ws, GuardList g, unsigned long long* bad) {
    const uint32_t* band = reinterpret_cast<const uint32_t*>(ws + g.off[blockIdx.x]);
    int n = 0;
    for (int i = threadIdx.x; i < (int)(GUARD_BYTES / 4); i += blockDim.x) {
        const uint32_t x = band[i] ^ GUARD_PATTERN;     // count the bytes that differ
        n += ((x & 0xffu) != 0) + ((x & 0xff00u) != 0) + ((x & 0xff0000u) != 0) + ((x & 0xff000000u) != 0);
    }
    if (n) atomicAdd(bad, (unsigned long long)n);
}

int perm_units(const mop_moe_shape& s) { return ceil_div(s.T * s.k, PERM_SEG); }
// The tensor-core scoring path needs 64-wide K blocks of x and 64-wide column chunks of W_r.
bool route_fast_possible(const mop_moe_shape& s) {
    return s.route_path != MOP_ROUTE_EXACT && s.T > 0 && s.d % 64 == 0 && s.E % 64 == 0 && tc_shape_supported(s.d, s.f);
}
// Measured policy: the three-piece GEMM plus the selection with re-evaluation beats the fp32 chains once
// the scoring is large (configs 3-5: 45-60 GFLOP); small layers keep the chains.
bool route_fast_wanted(const mop_moe_shape& s) {
    if (s.route_path == MOP_ROUTE_TENSOR) return true;
    return 2.0 * s.T * s.d * s.E >= 2e10;
}
int part_tiles(const mop_moe_shape& s) { return ceil_div(s.f, 32); }

Layout make_layout(const mop_moe_shape& s) {
    Layout L{};
    size_t o = 0;
    auto band = [&]() { if (L.n_guards < MAX_GUARDS) L.guard[L.n_guards++] = o; o += GUARD_BYTES; };
    band();
    auto take = [&](size_t bytes) { size_t r = o; o += align_up(bytes); band(); return r; };
    const size_t T = s.T, d = s.d, E = s.E, k = s.k, f = s.f, M = T * k;
    L.z = take(T * E * 4);
    L.partial = take((size_t)perm_units(s) * E * 4 + 4);
    L.tiles = take(tc_tables_bytes(s.T * s.k, s.E));
    L.status = take(256);
    if (route_fast_possible(s)) {
        L.fr_pieces = take(3 * d * E * 2);
        L.fr_wrT = take(d * E * 4);
        L.fr_colsq = take((size_t)ceil_div(s.d, 32) * E * 4);
        L.fr_xnorm = take(T * 4 + 16);
        L.fr_scal = take(256);
        L.fr_wsq = take(E * 4);
        L.fr_todo = take(T * 4 + 16);
        L.fr_z1 = take(T * E * 4);
    }
    if (s.with_backward) {
        L.part = take((size_t)part_tiles(s) * M * 4);
        L.dYp = take(M * d * 2);
        L.dG = take(M * f * 2);
        L.dU = take(M * f * 2);
        L.gH = take(M * f * 2);
        L.dXp = take(M * d * 2);
        L.dz_sel = take(M * 4 + 16);
        L.dz_row = take(M * 4 + 16);
        L.wrT = take(d * E * 4);
        if (s.with_backward == 2) {
            L.rG = take(M * f * 2);
            L.rU = take(M * f * 2);
            L.rH = take(M * f * 2);
        }
    }
    if (s.host_io) {
        L.hx = take(T * d * 2);
        L.hXp = take(M * d * 2);
        L.hH = take(M * f * 2);
        L.hYp = take(M * d * 2);
        L.hY = take(T * d * 2);
        L.hidx = take(M * 4);
        L.hcounts = take(E * 4);
        L.hoffsets = take((E + 1) * 4);
        L.hperm = take(M * 4);
        L.hsrc = take(M * 4);
        L.hgate = take(M * 4);
        if (s.with_backward) {
            L.hG = take(M * f * 2);
            L.hU = take(M * f * 2);
            L.hdY = take(T * d * 2);
            L.hdX = take(T * d * 2);
            L.hdgate = take(M * 4);
        }
        if (s.host_io == 2) {
            L.qx = take(T * d * 2);
            L.qY = take(T * d * 2);
            L.qidx = take(M * 4);
            L.qgate = take(M * 4);
            if (s.with_backward) {
                L.qdY = take(T * d * 2);
                L.qdX = take(T * d * 2);
                L.qdgate = take(M * 4);
            }
        }
    }
    L.total = o;
    return L;
}

mop_status check_shape(const mop_moe_shape* s) {
    if (!s) return MOP_ERR_INVALID_ARG;
    if (s->T < 0 || s->d < 1 || s->E < 1 || s->k < 1 || s->f < 1) return MOP_ERR_INVALID_ARG;
    if (s->k > s->E) return MOP_ERR_INVALID_ARG;
    if (s->score_fn != MOP_SCORE_SOFTMAX && s->score_fn != MOP_SCORE_SIGMOID) return MOP_ERR_INVALID_ARG;
    if (s->bias_mode < MOP_BIAS_NONE || s->bias_mode > MOP_BIAS_PRE_LOGIT) return MOP_ERR_INVALID_ARG;
    if (s->bias_mode == MOP_BIAS_POST_SCORE && s->score_fn != MOP_SCORE_SIGMOID) return MOP_ERR_INVALID_ARG;
    if (s->gemm_path < MOP_GEMM_AUTO || s->gemm_path > MOP_GEMM_TENSOR_TN) return MOP_ERR_INVALID_ARG;
    if ((long long)s->T * s->k >= (1ll << 31) - 4096) return MOP_ERR_SHAPE;
    if (s->E > SEL_MAX_E || s->k > 32) return MOP_ERR_SHAPE;
    if ((long long)s->T * s->d >= (1ll << 40) || (long long)s->d * s->f >= (1ll << 31)) return MOP_ERR_SHAPE;
    if (s->d % 8 || s->f % 8) return MOP_ERR_ALIGN;
    if (s->host_io < 0 || s->host_io > 2) return MOP_ERR_INVALID_ARG;
    if (s->route_path < MOP_ROUTE_AUTO || s->route_path > MOP_ROUTE_TENSOR) return MOP_ERR_INVALID_ARG;
    return MOP_OK;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

#define REQ_PTR(p)                                      \
    do {                                                \
        if (!(p)) return MOP_ERR_INVALID_ARG;           \
        if (!aligned16(p)) return MOP_ERR_ALIGN;        \
    } while (0)

// token-sized tensors may be null when the layer has no tokens (an empty tensor has no storage)
#define REQ_PTR_T(p)                                    \
    do {                                                \
        if (c->s.T > 0) REQ_PTR(p);                     \
    } while (0)

#define CUDA_OK(expr)                                 \
    do {                                                \
        if ((expr) != cudaSuccess) return MOP_ERR_CUDA; \
    } while (0)

// Launch with optional event timing around it.
#define LAUNCH(c, name, st, ...)       \
    do {                               \
        (c)->prof.begin(name, st);     \
        __VA_ARGS__;                   \
        (c)->prof.end(st);             \
    } while (0)

inline mop_status after_launch(mop_ctx* c, int n = 1) {
    c->launches += n;
    return cudaGetLastError() == cudaSuccess ? MOP_OK : MOP_ERR_CUDA;
}

struct DeviceGuard {
    int prev = -1;
    bool ok;
    explicit DeviceGuard(int dev) {
        ok = cudaGetDevice(&prev) == cudaSuccess && (prev == dev || cudaSetDevice(dev) == cudaSuccess);
    }
    ~DeviceGuard() {
        int cur;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

bool use_tensor(const mop_ctx* c) { return c->tensor_ok && c->s.gemm_path != MOP_GEMM_SCALAR; }

// ---- scalar-path launches ---------------------------------------------------------------
mop_status launch_scalar(mop_ctx* c, const char* name, const ScalarGemmArgs& g, cudaStream_t st) {
    dim3 grid(ceil_div(g.N, SG_BN), c->s.E);
    LAUNCH(c, name, st, scalar_grouped_gemm_kernel<<<grid, 256, 0, st>>>(g));
    return after_launch(c);
}

}  // namespace

extern "C" {

const char* mop_status_string(mop_status s) {
    switch (s) {
        case MOP_OK: return "ok";
        case MOP_ERR_INVALID_ARG: return "invalid argument";
        case MOP_ERR_SHAPE: return "shape out of supported range";
        case MOP_ERR_ALIGN: return "misaligned pointer or row size";
        case MOP_ERR_WORKSPACE: return "workspace allocation failed";
        case MOP_ERR_CUDA: return "CUDA call failed";
        case MOP_ERR_UNSUPPORTED: return "unsupported request";
        case MOP_ERR_TIMEOUT: return "device-side wait ran out";
    }
    return "unknown status";
}

size_t mop_workspace_bytes(const mop_moe_shape* shape) {
    if (check_shape(shape) != MOP_OK) return 0;
    return make_layout(*shape).total;
}

mop_status mop_create(mop_ctx** out, const mop_moe_shape* shape, int device) {
    if (!out) return MOP_ERR_INVALID_ARG;
    *out = nullptr;
    mop_status st = check_shape(shape);
    if (st != MOP_OK) return st;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess) return MOP_ERR_CUDA;
    if (device < 0 || device >= ndev) return MOP_ERR_INVALID_ARG;
    DeviceGuard guard(device);
    if (!guard.ok) return MOP_ERR_CUDA;
    mop_ctx* c = new (std::nothrow) mop_ctx();
    if (!c) return MOP_ERR_WORKSPACE;
    c->s = *shape;
    c->device = device;
    c->launches = 0;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete c; return MOP_ERR_CUDA; }
    c->sm_count = prop.multiProcessorCount;
    c->tensor_ok = (prop.major == 10) && tc_shape_supported(shape->d, shape->f);
    if ((shape->gemm_path == MOP_GEMM_TENSOR || shape->gemm_path >= MOP_GEMM_TENSOR_1CTA) && !c->tensor_ok) {
        delete c;
        return MOP_ERR_UNSUPPORTED;
    }
    const Layout L = make_layout(*shape);
    c->ws_bytes = L.total;
    if (cudaMalloc(&c->ws, L.total) != cudaSuccess) { cudaGetLastError(); delete c; return MOP_ERR_WORKSPACE; }
    char* w = c->ws;
    c->z = reinterpret_cast<float*>(w + L.z);
    c->partial = reinterpret_cast<int32_t*>(w + L.partial);
    c->tiles = reinterpret_cast<int32_t*>(w + L.tiles);
    c->status = reinterpret_cast<int32_t*>(w + L.status);
    c->fast_route = false;
    if (route_fast_possible(*shape) && prop.major == 10) {
        c->fr_pieces = reinterpret_cast<bf16*>(w + L.fr_pieces);
        c->fr_wrT = reinterpret_cast<float*>(w + L.fr_wrT);
        c->fr_colsq = reinterpret_cast<float*>(w + L.fr_colsq);
        c->fr_xnorm = reinterpret_cast<float*>(w + L.fr_xnorm);
        c->fr_scal = reinterpret_cast<float*>(w + L.fr_scal);
        c->fr_wsq = reinterpret_cast<float*>(w + L.fr_wsq);
        c->fr_todo = reinterpret_cast<int32_t*>(w + L.fr_todo);
        c->fr_z1 = reinterpret_cast<float*>(w + L.fr_z1);
        c->fast_route = route_fast_wanted(*shape);
    } else if (shape->route_path == MOP_ROUTE_TENSOR) {
        cudaFree(c->ws); delete c;
        return MOP_ERR_UNSUPPORTED;
    }
    if (shape->with_backward) {
        c->part = reinterpret_cast<float*>(w + L.part);
        c->dYp = reinterpret_cast<bf16*>(w + L.dYp);
        c->dG = reinterpret_cast<bf16*>(w + L.dG);
        c->dU = reinterpret_cast<bf16*>(w + L.dU);
        c->gH = reinterpret_cast<bf16*>(w + L.gH);
        c->dXp = reinterpret_cast<bf16*>(w + L.dXp);
        c->dz_sel = reinterpret_cast<float*>(w + L.dz_sel);
        c->dz_row = reinterpret_cast<float*>(w + L.dz_row);
        c->wrT = reinterpret_cast<float*>(w + L.wrT);
        if (shape->with_backward == 2) {
            c->rG = reinterpret_cast<bf16*>(w + L.rG);
            c->rU = reinterpret_cast<bf16*>(w + L.rU);
            c->rH = reinterpret_cast<bf16*>(w + L.rH);
        }
    }
    if (shape->host_io) {
        c->hx = reinterpret_cast<bf16*>(w + L.hx);
        c->hXp = reinterpret_cast<bf16*>(w + L.hXp);
        c->hH = reinterpret_cast<bf16*>(w + L.hH);
        c->hYp = reinterpret_cast<bf16*>(w + L.hYp);
        c->hY = reinterpret_cast<bf16*>(w + L.hY);
        c->hidx = reinterpret_cast<int32_t*>(w + L.hidx);
        c->hcounts = reinterpret_cast<int32_t*>(w + L.hcounts);
        c->hoffsets = reinterpret_cast<int32_t*>(w + L.hoffsets);
        c->hperm = reinterpret_cast<int32_t*>(w + L.hperm);
        c->hsrc = reinterpret_cast<int32_t*>(w + L.hsrc);
        c->hgate = reinterpret_cast<float*>(w + L.hgate);
        if (shape->with_backward) {
            c->hG = reinterpret_cast<bf16*>(w + L.hG);
            c->hU = reinterpret_cast<bf16*>(w + L.hU);
            c->hdY = reinterpret_cast<bf16*>(w + L.hdY);
            c->hdX = reinterpret_cast<bf16*>(w + L.hdX);
            c->hdgate = reinterpret_cast<float*>(w + L.hdgate);
        }
    }
    if (shape->host_io) {
        c->px[0] = c->hx; c->pY[0] = c->hY; c->pidx[0] = c->hidx; c->pgate[0] = c->hgate;
        c->pdY[0] = c->hdY; c->pdX[0] = c->hdX; c->pdgate[0] = c->hdgate;
    }
    if (shape->host_io == 2) {
        c->px[1] = reinterpret_cast<bf16*>(w + L.qx);
        c->pY[1] = reinterpret_cast<bf16*>(w + L.qY);
        c->pidx[1] = reinterpret_cast<int32_t*>(w + L.qidx);
        c->pgate[1] = reinterpret_cast<float*>(w + L.qgate);
        if (shape->with_backward) {
            c->pdY[1] = reinterpret_cast<bf16*>(w + L.qdY);
            c->pdX[1] = reinterpret_cast<bf16*>(w + L.qdX);
            c->pdgate[1] = reinterpret_cast<float*>(w + L.qdgate);
        }
    }
    if (cudaMemset(c->status, 0, 256) != cudaSuccess) { cudaFree(c->ws); delete c; return MOP_ERR_CUDA; }
    c->n_guards = L.n_guards;
    for (int i = 0; i < L.n_guards; ++i) c->guard_off[i] = L.guard[i];
    if (shape->host_io == 2) {
        bool ok = cudaStreamCreateWithFlags(&c->out_stream, cudaStreamNonBlocking) == cudaSuccess;
        for (int i = 0; i < 2 && ok; ++i)
            ok = cudaEventCreateWithFlags(&c->ev_x[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&c->ev_dy[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&c->ev_fwd[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&c->ev_done[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&c->ev_drained[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) { cudaFree(c->ws); delete c; return MOP_ERR_CUDA; }
    }
    if (shape->host_io) {
        if (cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_in, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_mid, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_out, cudaEventDisableTiming) != cudaSuccess) {
            cudaFree(c->ws); delete c; return MOP_ERR_CUDA;
        }
    }
    if (c->tensor_ok) {
        st = tc_plan_init(&c->plan, *shape, c->sm_count, &c->prof);
        if (st == MOP_OK) st = tc2_init();
        if (st == MOP_OK) st = tn_init();
        if (st == MOP_OK) st = rs_init();
        if (st != MOP_OK) { cudaFree(c->ws); delete c; return st; }
        if (c->fast_route) {
            bool ok = cudaMemset(c->fr_scal, 0, 256) == cudaSuccess;
            c->fr_rblocks = route_resolve_resident(shape->E, c->sm_count);
            ok = ok && cudaStreamCreateWithFlags(&c->fr_stream, cudaStreamNonBlocking) == cudaSuccess &&
                 cudaEventCreateWithFlags(&c->fr_fork, cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&c->fr_join, cudaEventDisableTiming) == cudaSuccess;
            if (!ok) { cudaFree(c->ws); delete c; return MOP_ERR_CUDA; }
        }
        c->plan.pairs = shape->gemm_path == MOP_GEMM_TENSOR_2CTA ? 1 : shape->gemm_path == MOP_GEMM_TENSOR_MIXED ? 2 : 0;
        if (c->sm_count < 2) c->plan.pairs = 0;
        // Measured policy (B200): the tokens-on-N down-projection wins on every workload; the tokens-on-N
        // up-projection wins when the K loop is long enough to hide its heavier epilogue (d >= 4096).
        c->plan.fwd_tn = 0;
        if (c->sm_count >= 2) {
            // bits 2, 3: the data gradients of the up- and down-projection on the same kernel
            if (shape->gemm_path == MOP_GEMM_TENSOR_TN) c->plan.fwd_tn = 15;
            else if (shape->gemm_path == MOP_GEMM_AUTO || shape->gemm_path == MOP_GEMM_TENSOR)
                c->plan.fwd_tn = 8 | 4 | 2 | (shape->d >= 4096 ? 1 : 0);
        }
    }
    *out = c;
    return MOP_OK;
}

void mop_destroy(mop_ctx* c) {
    if (!c) return;
    DeviceGuard guard(c->device);
    if (c->prof.ev) {
        for (int i = 0; i < 2 * Profiler::MAX_REC; ++i) cudaEventDestroy(c->prof.ev[i]);
        delete[] c->prof.ev;
    }
    if (c->fast_route) {
        cudaStreamDestroy(c->fr_stream);
        cudaEventDestroy(c->fr_fork); cudaEventDestroy(c->fr_join);
    }
    if (c->s.host_io) {
        cudaStreamDestroy(c->copy_stream);
        cudaEventDestroy(c->ev_in); cudaEventDestroy(c->ev_mid); cudaEventDestroy(c->ev_out);
    }
    if (c->s.host_io == 2) {
        cudaStreamDestroy(c->out_stream);
        for (int i = 0; i < 2; ++i) {
            cudaEventDestroy(c->ev_x[i]); cudaEventDestroy(c->ev_dy[i]); cudaEventDestroy(c->ev_fwd[i]);
            cudaEventDestroy(c->ev_done[i]); cudaEventDestroy(c->ev_drained[i]);
        }
    }
    cudaFree(c->ws);
    delete c;
}

int64_t mop_launch_count(const mop_ctx* c) { return c ? c->launches : 0; }

mop_status mop_selftest_wait_timeout(mop_ctx* c, int64_t limit_cycles, void* stream) {
    if (!c || limit_cycles < 1 || limit_cycles > 4000000000ll) return MOP_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MOP_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t* gave_up = c->status + 8;                    // a spare word of the status block
    CUDA_OK(cudaMemsetAsync(gave_up, 0, 4, st));
    tc_wait_selftest_kernel<<<1, 32, 0, st>>>(c->status, limit_cycles, gave_up);
    if (after_launch(c) != MOP_OK) return MOP_ERR_CUDA;
    int32_t flag = 0;
    CUDA_OK(cudaMemcpyAsync(&flag, gave_up, 4, cudaMemcpyDeviceToHost, st));
    CUDA_OK(cudaStreamSynchronize(st));
    return flag == 1 ? MOP_OK : MOP_ERR_CUDA;            // the wait must have given up, not completed
}

mop_status mop_debug_guard_arm(mop_ctx* c, void* stream) {
    if (!c) return MOP_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MOP_ERR_CUDA;
    GuardList g;
    g.n = c->n_guards;
    for (int i = 0; i < g.n; ++i) g.off[i] = c->guard_off[i];
    guard_fill_kernel<<<g.n, 256, 0, static_cast<cudaStream_t>(stream)>>>(c->ws, g);
    return after_launch(c);
}

mop_status mop_debug_guard_poke(mop_ctx* c, int32_t band, int32_t byte, void* stream) {
    if (!c || band < 0 || band >= c->n_guards || byte < 0 || byte >= (int32_t)GUARD_BYTES) return MOP_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MOP_ERR_CUDA;
    CUDA_OK(cudaMemsetAsync(c->ws + c->guard_off[band] + byte, 0, 1, static_cast<cudaStream_t>(stream)));
    return MOP_OK;
}

mop_status mop_debug_guard_check(mop_ctx* c, int64_t* bad_bytes, void* stream) {
    if (!c || !bad_bytes) return MOP_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MOP_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    GuardList g;
    g.n = c->n_guards;
    for (int i = 0; i < g.n; ++i) g.off[i] = c->guard_off[i];
    unsigned long long* bad = reinterpret_cast<unsigned long long*>(c->status + 16);   // spare words of the status block
    CUDA_OK(cudaMemsetAsync(bad, 0, 8, st));
    guard_check_kernel<<<g.n, 256, 0, st>>>(c->ws, g, bad);
    if (after_launch(c) != MOP_OK) return MOP_ERR_CUDA;
    unsigned long long host = 0;
    CUDA_OK(cudaMemcpyAsync(&host, bad, 8, cudaMemcpyDeviceToHost, st));
    CUDA_OK(cudaStreamSynchronize(st));
    *bad_bytes = (int64_t)host;
    return MOP_OK;
}

mop_status mop_poll(mop_ctx* c, void* stream) {
    if (!c) return MOP_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MOP_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t word = 0;
    CUDA_OK(cudaMemcpyAsync(&word, c->status, 4, cudaMemcpyDeviceToHost, st));
    CUDA_OK(cudaStreamSynchronize(st));
    if (word != 0) {
        CUDA_OK(cudaMemsetAsync(c->status, 0, 4, st));
        CUDA_OK(cudaStreamSynchronize(st));
        return MOP_ERR_TIMEOUT;
    }
    return MOP_OK;
}

mop_status mop_moe_route(mop_ctx* c, const void* x, const float* W_r, const float* bias, int32_t* topk_idx,
                         float* topk_gate, float* logits_opt, void* stream) {
    if (!c) return MOP_ERR_INVALID_ARG;
    REQ_PTR_T(x); REQ_PTR(W_r); REQ_PTR_T(topk_idx); REQ_PTR_T(topk_gate);
    if ((c->s.bias_mode != MOP_BIAS_NONE) != (bias != nullptr)) return MOP_ERR_INVALID_ARG;
    if (logits_opt && !aligned16(logits_opt)) return MOP_ERR_ALIGN;
    const mop_moe_shape& s = c->s;
    if (s.T == 0) return MOP_OK;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MOP_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float* z = logits_opt ? logits_opt : c->z;
    if (c->fast_route) {
        // logits on the tensor cores from three bf16 pieces of W_r, then selection with the contract's chain
        // re-evaluated where the order is in doubt
        mop_status r;
        dim3 gp(ceil_div(s.E, 32), ceil_div(s.d, 32));
        LAUNCH(c, "route_prep", st,
               route_prep_kernel<<<gp, 256, 0, st>>>(W_r, c->fr_pieces, c->fr_wrT, c->fr_colsq, s.d, s.E));
        if ((r = after_launch(c)) != MOP_OK) return r;
        // only the selection needs the norms of x's rows and of W_r's columns: they run on a side stream beside
        // the logit GEMM (which leaves room on every SM for such blocks, and DRAM idle)
        CUDA_OK(cudaEventRecord(c->fr_fork, st));
        CUDA_OK(cudaStreamWaitEvent(c->fr_stream, c->fr_fork, 0));
        route_wnorm_kernel<<<ceil_div(s.E, 8), 256, 0, c->fr_stream>>>(c->fr_colsq, c->fr_wsq, ceil_div(s.d, 32), s.E);
        route_xnorm_kernel<<<ceil_div(s.T, 8), 256, 0, c->fr_stream>>>(static_cast<const bf16*>(x), c->fr_xnorm, s.T, s.d);
        CUDA_OK(cudaEventRecord(c->fr_join, c->fr_stream));
        c->launches += 2;
        int splits = 1;
        if ((r = rs_launch(&c->plan, "route_score_tc", x, c->fr_pieces, z, c->fr_z1, s.T, s.d, s.E, c->status, &splits, st)) != MOP_OK)
            return r;
        const float* z1 = splits == 2 ? c->fr_z1 : nullptr;
        c->launches += 1;
        CUDA_OK(cudaStreamWaitEvent(st, c->fr_join, 0));
        int32_t* stats = reinterpret_cast<int32_t*>(c->fr_scal) + 8;
        int32_t* n_todo = reinterpret_cast<int32_t*>(c->fr_scal) + 16;
        CUDA_OK(cudaMemsetAsync(n_todo, 0, 4, st));
        const int rblocks = min(ceil_div(s.T, SELF_WARPS), c->fr_rblocks);
        LAUNCH(c, "route_select_screen", st,
               route_select_fast(z, z1, bias, static_cast<const bf16*>(x), c->fr_wrT, c->fr_xnorm, c->fr_wsq, topk_idx,
                                 topk_gate, c->fr_todo, n_todo, stats, s.T, s.d, s.E, s.k, s.score_fn, s.bias_mode, 0,
                                 rblocks, st));
        if ((r = after_launch(c)) != MOP_OK) return r;
        LAUNCH(c, "route_select_resolve", st,
               route_select_fast(z, nullptr, bias, static_cast<const bf16*>(x), c->fr_wrT, c->fr_xnorm, c->fr_wsq, topk_idx,
                                 topk_gate, c->fr_todo, n_todo, stats, s.T, s.d, s.E, s.k, s.score_fn, s.bias_mode, 1,
                                 rblocks, st));
        return after_launch(c);
    }
    LAUNCH(c, "route_score", st, route_score(static_cast<const bf16*>(x), W_r, z, s.T, s.d, s.E, c->sm_count, st));
    mop_status r = after_launch(c);
    if (r != MOP_OK) return r;
    const size_t smem = (size_t)SEL_WARPS * 2 * s.E * sizeof(float);
    LAUNCH(c, "route_select", st,
           route_select_kernel<<<ceil_div(s.T, SEL_WARPS), SEL_WARPS * 32, smem, st>>>(
               z, bias, topk_idx, topk_gate, s.T, s.E, s.k, s.score_fn, s.bias_mode));
    return after_launch(c);
}

mop_status mop_route_stats(mop_ctx* c, int64_t* tokens_reevaluated, int64_t* chains, int64_t* beyond_half_bound,
                           void* stream) {
    if (!c || !tokens_reevaluated || !chains || !beyond_half_bound) return MOP_ERR_INVALID_ARG;
    *tokens_reevaluated = *chains = *beyond_half_bound = 0;
    if (!c->fast_route) return MOP_OK;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MOP_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t host[3] = {0, 0, 0};
    int32_t* dev = reinterpret_cast<int32_t*>(c->fr_scal) + 8;
    CUDA_OK(cudaMemcpyAsync(host, dev, 12, cudaMemcpyDeviceToHost, st));
    CUDA_OK(cudaMemsetAsync(dev, 0, 12, st));
    CUDA_OK(cudaStreamSynchronize(st));
    *tokens_reevaluated = host[0];
    *chains = host[1];
    *beyond_half_bound = host[2];
    return MOP_OK;
}

mop_status mop_moe_permute(mop_ctx* c, const void* x, const int32_t* topk_idx, int32_t* counts, int32_t* offsets,
                           int32_t* perm_row, int32_t* row_src, void* Xp, void* stream) {
    if (!c) return MOP_ERR_INVALID_ARG;
    REQ_PTR_T(topk_idx); REQ_PTR(counts); REQ_PTR(offsets); REQ_PTR_T(perm_row); REQ_PTR_T(row_src);
    if (Xp) { REQ_PTR_T(x); REQ_PTR_T(Xp); }   // Xp == NULL: tables only, for the gathering forward
    const mop_moe_shape& s = c->s;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MOP_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int M = s.T * s.k;
    const int units = perm_units(s);
    const size_t smem = (size_t)PERM_WARPS * s.E * sizeof(int32_t);
    mop_status r;
    if (perm_small_fits(units, s.E)) {   // a few units: one block does histogram, scan and rank
        LAUNCH(c, "perm_small", st,
               perm_small_kernel<<<1, 1024, ((size_t)units * s.E + s.E + 1) * sizeof(int32_t), st>>>(
                   topk_idx, counts, offsets, perm_row, row_src, M, s.E, units));
        if ((r = after_launch(c)) != MOP_OK) return r;
    } else {
    if (units > 0) {
        LAUNCH(c, "perm_hist", st,
               perm_hist_kernel<<<ceil_div(units, PERM_WARPS), PERM_WARPS * 32, smem, st>>>(topk_idx, c->partial, M,
                                                                                            s.E));
        if ((r = after_launch(c)) != MOP_OK) return r;
    }
    if (units == 0) {   // nothing to permute: counts and offsets are all zero
        LAUNCH(c, "perm_scan", st,
               perm_scan_kernel<<<1, 1024, (s.E + 1) * sizeof(int32_t), st>>>(c->partial, counts, offsets, units, s.E));
        return after_launch(c);
    }
    LAUNCH(c, "perm_scan", st,
           perm_scan_cols_kernel<<<ceil_div(s.E, 32), PSCAN_WARPS * 32, 0, st>>>(c->partial, counts, units, s.E));
    if ((r = after_launch(c)) != MOP_OK) return r;
    LAUNCH(c, "perm_rank", st,
           perm_rank_kernel<<<ceil_div(units, PERM_WARPS), PERM_WARPS * 32, smem + (s.E + 1) * sizeof(int32_t), st>>>(
               topk_idx, c->partial, counts, offsets, perm_row, row_src, M, s.E));
    if ((r = after_launch(c)) != MOP_OK) return r;
    }
    if (!Xp) return MOP_OK;
    LAUNCH(c, "permute_scatter_rows", st,
           launch_scatter_rows(static_cast<const uint4*>(x), static_cast<uint4*>(Xp), perm_row, s.T, s.k, s.d / 8,
                               c->sm_count, st));
    return after_launch(c);
}

mop_status mop_moe_combine(mop_ctx* c, const void* Yp, const int32_t* perm_row, void* Y, void* stream) {
    if (!c) return MOP_ERR_INVALID_ARG;
    REQ_PTR_T(Yp); REQ_PTR_T(perm_row); REQ_PTR_T(Y);
    const mop_moe_shape& s = c->s;
    if (s.T == 0) return MOP_OK;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MOP_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    LAUNCH(c, "combine_rows", st,
           launch_combine_rows(static_cast<const uint4*>(Yp), perm_row, static_cast<uint4*>(Y), s.T, s.k, s.d / 8,
                               c->sm_count, st));
    return after_launch(c);
}

namespace {
// G, U, H = SwiGLU up-projection of the permuted rows (the first half of the forward; also the
// recomputation step of the backward).  Tensor-core or scalar path as the context was created.
mop_status up_projection(mop_ctx* c, const void* Xp, const int32_t* offsets, const void* W_gate, const void* W_up,
                         void* G_save, void* U_save, void* H, cudaStream_t st) {
    const mop_moe_shape& s = c->s;
    const int M = s.T * s.k;
    if (use_tensor(c)) {
        TcFwdArgs a{};
        a.Xp = static_cast<const bf16*>(Xp); a.offsets = offsets;
        a.W_gate = static_cast<const bf16*>(W_gate); a.W_up = static_cast<const bf16*>(W_up);
        a.G_save = static_cast<bf16*>(G_save); a.U_save = static_cast<bf16*>(U_save); a.H = static_cast<bf16*>(H);
        int n = 0;
        mop_status r = tc_up_only(&c->plan, a, c->tiles, c->status, st, &n);
        c->launches += n;
        return r;
    }
    ScalarGemmArgs g{};
    g.A[0] = g.A[1] = static_cast<const bf16*>(Xp);
    g.B[0] = static_cast<const bf16*>(W_gate); g.B[1] = static_cast<const bf16*>(W_up);
    g.sAm = s.d; g.sAk = 1; g.sBk = s.f; g.sBn = 1; g.sBe = (long)s.d * s.f;
    g.offsets = offsets; g.ragged_k = 0; g.N = s.f; g.Kfix = s.d; g.npairs = 2; g.dual_acc = 1; g.epi = EPI_SWIGLU;
    g.ep.out0 = static_cast<bf16*>(H); g.ep.out1 = static_cast<bf16*>(G_save); g.ep.out2 = static_cast<bf16*>(U_save);
    g.ep.ldo = s.f; g.ep.M_total = M;
    return launch_scalar(c, "scalar_up_swiglu", g, st);
}
}  // namespace

mop_status mop_moe_expert_ffn_fwd(mop_ctx* c, const void* Xp, const int32_t* offsets, const int32_t* row_src,
                                  const float* topk_gate, const void* W_gate, const void* W_up, const void* W_down,
                                  void* G_save, void* U_save, void* H, void* Yp, void* stream) {
    if (!c) return MOP_ERR_INVALID_ARG;
    REQ_PTR_T(Xp); REQ_PTR(offsets); REQ_PTR_T(row_src); REQ_PTR_T(topk_gate); REQ_PTR(W_gate); REQ_PTR(W_up);
    REQ_PTR(W_down); REQ_PTR_T(H); REQ_PTR_T(Yp);
    if ((G_save == nullptr) != (U_save == nullptr)) return MOP_ERR_INVALID_ARG;
    if (G_save && (!aligned16(G_save) || !aligned16(U_save))) return MOP_ERR_ALIGN;
    const mop_moe_shape& s = c->s;
    if (s.T == 0) return MOP_OK;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MOP_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int M = s.T * s.k;
    if (use_tensor(c)) {
        TcFwdArgs a{};
        a.Xp = static_cast<const bf16*>(Xp); a.offsets = offsets; a.row_src = row_src; a.gate = topk_gate;
        a.W_gate = static_cast<const bf16*>(W_gate); a.W_up = static_cast<const bf16*>(W_up);
        a.W_down = static_cast<const bf16*>(W_down);
        a.G_save = static_cast<bf16*>(G_save); a.U_save = static_cast<bf16*>(U_save);
        a.H = static_cast<bf16*>(H); a.Yp = static_cast<bf16*>(Yp);
        int n = 0;
        mop_status r = tc_ffn_fwd(&c->plan, a, c->tiles, c->status, st, &n);
        c->launches += n;
        return r;
    }
    ScalarGemmArgs g{};
    g.A[0] = g.A[1] = static_cast<const bf16*>(Xp);
    g.B[0] = static_cast<const bf16*>(W_gate); g.B[1] = static_cast<const bf16*>(W_up);
    g.sAm = s.d; g.sAk = 1; g.sBk = s.f; g.sBn = 1; g.sBe = (long)s.d * s.f;
    g.offsets = offsets; g.ragged_k = 0; g.N = s.f; g.Kfix = s.d; g.npairs = 2; g.dual_acc = 1; g.epi = EPI_SWIGLU;
    g.ep.out0 = static_cast<bf16*>(H); g.ep.out1 = static_cast<bf16*>(G_save); g.ep.out2 = static_cast<bf16*>(U_save);
    g.ep.ldo = s.f; g.ep.M_total = M;
    mop_status r = launch_scalar(c, "scalar_up_swiglu", g, st);
    if (r != MOP_OK) return r;
    ScalarGemmArgs h{};
    h.A[0] = static_cast<const bf16*>(H); h.B[0] = static_cast<const bf16*>(W_down);
    h.sAm = s.f; h.sAk = 1; h.sBk = s.d; h.sBn = 1; h.sBe = (long)s.d * s.f;
    h.offsets = offsets; h.ragged_k = 0; h.N = s.d; h.Kfix = s.f; h.npairs = 1; h.epi = EPI_GATE;
    h.ep.out0 = static_cast<bf16*>(Yp); h.ep.gate = topk_gate; h.ep.row_src = row_src; h.ep.ldo = s.d; h.ep.M_total = M;
    return launch_scalar(c, "scalar_down_gate", h, st);
}

mop_status mop_moe_expert_ffn_fwd_gather(mop_ctx* c, const void* x, const int32_t* offsets, const int32_t* row_src,
                                         const float* topk_gate, const void* W_gate, const void* W_up,
                                         const void* W_down, void* H, void* Yp, void* stream) {
    if (!c) return MOP_ERR_INVALID_ARG;
    REQ_PTR_T(x); REQ_PTR(offsets); REQ_PTR_T(row_src); REQ_PTR_T(topk_gate); REQ_PTR(W_gate); REQ_PTR(W_up);
    REQ_PTR(W_down); REQ_PTR_T(H); REQ_PTR_T(Yp);
    if (!use_tensor(c)) return MOP_ERR_UNSUPPORTED;   // the gather is a TMA feature of the tensor-core path
    const mop_moe_shape& s = c->s;
    if (s.T == 0) return MOP_OK;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MOP_ERR_CUDA;
    TcFwdArgs a{};
    a.x_gather = static_cast<const bf16*>(x); a.offsets = offsets; a.row_src = row_src; a.gate = topk_gate;
    a.W_gate = static_cast<const bf16*>(W_gate); a.W_up = static_cast<const bf16*>(W_up);
    a.W_down = static_cast<const bf16*>(W_down);
    a.H = static_cast<bf16*>(H); a.Yp = static_cast<bf16*>(Yp);
    int n = 0;
    mop_status r = tc_ffn_fwd(&c->plan, a, c->tiles, c->status, static_cast<cudaStream_t>(stream), &n);
    c->launches += n;
    return r;
}

mop_status mop_moe_expert_ffn_bwd(mop_ctx* c, const void* dY, const void* Xp, const void* G_save,
                                  const void* U_save, const void* H, const int32_t* offsets, const int32_t* perm_row,
                                  const int32_t* row_src, const float* topk_gate, const void* W_gate,
                                  const void* W_up, const void* W_down, void* dX, float* dW_gate, float* dW_up,
                                  float* dW_down, float* dgate, void* stream) {
    if (!c) return MOP_ERR_INVALID_ARG;
    if (!c->s.with_backward) return MOP_ERR_UNSUPPORTED;
    // Recompute mode (activation checkpointing): with G_save, U_save and H all NULL the up-projection is
    // run again from Xp into the context's own buffers (the same kernel as the forward: same bits).
    const bool recompute = c->s.T > 0 && !G_save && !U_save && !H;
    if (recompute && c->s.with_backward != 2) return MOP_ERR_UNSUPPORTED;
    REQ_PTR_T(dY); REQ_PTR_T(Xp); REQ_PTR(offsets);
    if (!recompute) { REQ_PTR_T(G_save); REQ_PTR_T(U_save); REQ_PTR_T(H); }
    REQ_PTR_T(perm_row); REQ_PTR_T(row_src); REQ_PTR_T(topk_gate); REQ_PTR(W_gate); REQ_PTR(W_up); REQ_PTR(W_down);
    REQ_PTR_T(dX); REQ_PTR(dW_gate); REQ_PTR(dW_up); REQ_PTR(dW_down); REQ_PTR_T(dgate);
    const mop_moe_shape& s = c->s;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MOP_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int M = s.T * s.k;
    mop_status r;
    if (recompute && s.T > 0) {
        if ((r = up_projection(c, Xp, offsets, W_gate, W_up, c->rG, c->rU, c->rH, st)) != MOP_OK) return r;
        G_save = c->rG; U_save = c->rU; H = c->rH;
    }
    if (s.T > 0) {
        // dYp[p,:] = dY[t,:]  (unscaled; the gate enters through dH and gate*H)
        LAUNCH(c, "dy_scatter_rows", st,
               launch_scatter_rows(static_cast<const uint4*>(dY), reinterpret_cast<uint4*>(c->dYp), perm_row, s.T, s.k,
                                   s.d / 8, c->sm_count, st));
        if ((r = after_launch(c)) != MOP_OK) return r;
    }
    int ntile_part = 0;
    if (use_tensor(c)) {
        TcBwdArgs a{};
        a.dYp = c->dYp; a.Xp = static_cast<const bf16*>(Xp); a.G_save = static_cast<const bf16*>(G_save);
        a.U_save = static_cast<const bf16*>(U_save); a.H = static_cast<const bf16*>(H);
        a.offsets = offsets; a.row_src = row_src; a.gate = topk_gate;
        a.W_gate = static_cast<const bf16*>(W_gate); a.W_up = static_cast<const bf16*>(W_up);
        a.W_down = static_cast<const bf16*>(W_down);
        a.dG = c->dG; a.dU = c->dU; a.gH = c->gH; a.dXp = c->dXp; a.part = c->part;
        a.dW_gate = dW_gate; a.dW_up = dW_up; a.dW_down = dW_down; a.accumulate = s.dw_accumulate;
        int n = 0;
        r = tc_ffn_bwd(&c->plan, a, c->tiles, c->status, st, &n, &ntile_part);
        c->launches += n;
        if (r != MOP_OK) return r;
    } else {
        if (s.T > 0) {
            ScalarGemmArgs g{};  // dHu = dYp W_down^T, SwiGLU backward in the epilogue
            g.A[0] = c->dYp; g.B[0] = static_cast<const bf16*>(W_down);
            g.sAm = s.d; g.sAk = 1; g.sBk = 1; g.sBn = s.d; g.sBe = (long)s.d * s.f;
            g.offsets = offsets; g.N = s.f; g.Kfix = s.d; g.npairs = 1; g.epi = EPI_DH;
            g.ep.out0 = c->dG; g.ep.out1 = c->dU; g.ep.out2 = c->gH;
            g.ep.in0 = static_cast<const bf16*>(G_save); g.ep.in1 = static_cast<const bf16*>(U_save);
            g.ep.in2 = static_cast<const bf16*>(H);
            g.ep.gate = topk_gate; g.ep.row_src = row_src; g.ep.part = c->part; g.ep.ldo = s.f; g.ep.M_total = M;
            if ((r = launch_scalar(c, "scalar_dgrad_down", g, st)) != MOP_OK) return r;
            ntile_part = ceil_div(s.f, SG_BN);
            ScalarGemmArgs h{};  // dXp = dG W_gate^T + dU W_up^T
            h.A[0] = c->dG; h.A[1] = c->dU;
            h.B[0] = static_cast<const bf16*>(W_gate); h.B[1] = static_cast<const bf16*>(W_up);
            h.sAm = s.f; h.sAk = 1; h.sBk = 1; h.sBn = s.f; h.sBe = (long)s.d * s.f;
            h.offsets = offsets; h.N = s.d; h.Kfix = s.f; h.npairs = 2; h.dual_acc = 0; h.epi = EPI_BF16;
            h.ep.out0 = c->dXp; h.ep.ldo = s.d; h.ep.M_total = M;
            if ((r = launch_scalar(c, "scalar_dgrad_gate_up", h, st)) != MOP_OK) return r;
        }
        // weight gradients (ragged K = the expert's rows); run even for T = 0 so that dW is defined
        ScalarGemmArgs w{};
        w.offsets = offsets; w.ragged_k = 1; w.npairs = 1; w.epi = EPI_F32; w.ep.accumulate = s.dw_accumulate;
        w.A[0] = c->gH; w.sAm = 1; w.sAk = s.f; w.B[0] = c->dYp; w.sBk = s.d; w.sBn = 1;
        w.Mfix = s.f; w.N = s.d; w.ep.outf = dW_down;
        if ((r = launch_scalar(c, "scalar_wgrad", w, st)) != MOP_OK) return r;
        w.A[0] = static_cast<const bf16*>(Xp); w.sAm = 1; w.sAk = s.d; w.B[0] = c->dG; w.sBk = s.f; w.sBn = 1;
        w.Mfix = s.d; w.N = s.f; w.ep.outf = dW_gate;
        if ((r = launch_scalar(c, "scalar_wgrad", w, st)) != MOP_OK) return r;
        w.B[0] = c->dU; w.ep.outf = dW_up;
        if ((r = launch_scalar(c, "scalar_wgrad", w, st)) != MOP_OK) return r;
    }
    if (s.T == 0) return MOP_OK;
    LAUNCH(c, "dgate_reduce", st,
           dgate_reduce_kernel<<<ceil_div(M, 256), 256, 0, st>>>(c->part, perm_row, dgate, M, ntile_part));
    if ((r = after_launch(c)) != MOP_OK) return r;
    return mop_moe_combine(c, c->dXp, perm_row, dX, stream);
}

// ---------------------------------------------------------------------------------------------
// Expert-chunked layer: the expert-contiguous buffers (Xp, H, Yp and the backward's intermediates) exist
// for one chunk of experts at a time, in a workspace the caller provides.
// ---------------------------------------------------------------------------------------------
namespace {
struct ChunkLayout {
    size_t off_c, row_src_c, perm_c, bounds, Xp, H, Yp, acc, G, U, dYp, dG, dU, gH, dXp, part, total;
    long long cap;   // rows of a chunk's buffers
};
ChunkLayout chunk_layout(const mop_moe_shape& s, int C, int bwd) {
    ChunkLayout L{};
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t r = o; o += align_up(bytes); return r; };
    const size_t T = s.T, d = s.d, E = s.E, k = s.k, f = s.f, M = T * k;
    // a chunk ends at an expert boundary at or past its share of the rows: at most one expert more than M / C
    size_t cap = (M + C - 1) / C + T;
    if (cap > M) cap = M;
    cap = (cap + 15) / 16 * 16;
    L.cap = (long long)cap;
    L.off_c = take((E + 1) * 4);
    L.row_src_c = take(cap * 4 + 16);
    L.perm_c = take(M * 4 + 16);
    L.bounds = take(16);
    L.Xp = take(cap * d * 2);
    L.H = take(cap * f * 2);
    L.Yp = take(cap * d * 2);
    L.acc = take(T * d * 4);
    if (bwd) {
        L.G = take(cap * f * 2);
        L.U = take(cap * f * 2);
        L.dYp = take(cap * d * 2);
        L.dG = take(cap * f * 2);
        L.dU = take(cap * f * 2);
        L.gH = take(cap * f * 2);
        L.dXp = take(cap * d * 2);
        L.part = take((size_t)part_tiles(s) * cap * 4);
    }
    L.total = o;
    return L;
}
mop_status chunk_check(mop_ctx* c, int32_t n_chunks, const void* workspace) {
    if (!c) return MOP_ERR_INVALID_ARG;
    if (n_chunks < 1 || n_chunks > 64) return MOP_ERR_INVALID_ARG;
    if (!workspace) return MOP_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return MOP_ERR_ALIGN;
    if (!use_tensor(c)) return MOP_ERR_UNSUPPORTED;    // the chunked layer runs on the tensor-core kernels only
    return MOP_OK;
}
// tables, gathered inputs of chunk i
mop_status chunk_begin(mop_ctx* c, const ChunkLayout& L, char* w, int i, int C, const void* src, size_t dst_off,
                       const int32_t* offsets, const int32_t* perm_row, const int32_t* row_src, bool tables,
                       cudaStream_t st) {
    const mop_moe_shape& s = c->s;
    const int M = s.T * s.k;
    int32_t* off_c = reinterpret_cast<int32_t*>(w + L.off_c);
    int32_t* row_src_c = reinterpret_cast<int32_t*>(w + L.row_src_c);
    int32_t* perm_c = reinterpret_cast<int32_t*>(w + L.perm_c);
    int32_t* bounds = reinterpret_cast<int32_t*>(w + L.bounds);
    mop_status r;
    if (tables) {
        LAUNCH(c, "chunk_tables", st,
               chunk_tables_kernel<<<min(ceil_div(M, 256), c->sm_count * 4), 256, 0, st>>>(
                   offsets, row_src, perm_row, off_c, row_src_c, perm_c, bounds, s.E, M, i, C));
        if ((r = after_launch(c)) != MOP_OK) return r;
    }
    LAUNCH(c, "chunk_gather_rows", st,
           gather_rows_kernel<<<c->sm_count * 8, 256, 0, st>>>(static_cast<const uint4*>(src),
                                                               reinterpret_cast<uint4*>(w + dst_off), row_src_c, bounds,
                                                               s.k, s.d / 8));
    return after_launch(c);
}
}  // namespace

size_t mop_moe_chunked_workspace_bytes(const mop_moe_shape* shape, int32_t n_chunks, int32_t with_backward) {
    if (check_shape(shape) != MOP_OK || n_chunks < 1 || n_chunks > 64) return 0;
    return chunk_layout(*shape, n_chunks, with_backward).total;
}

mop_status mop_moe_layer_fwd_chunked(mop_ctx* c, int32_t n_chunks, const void* x, const float* W_r, const float* bias,
                                     const void* W_gate, const void* W_up, const void* W_down, int32_t* topk_idx,
                                     float* topk_gate, int32_t* counts, int32_t* offsets, int32_t* perm_row,
                                     int32_t* row_src, void* Y, void* workspace, void* stream) {
    mop_status r = chunk_check(c, n_chunks, workspace);
    if (r != MOP_OK) return r;
    REQ_PTR_T(x); REQ_PTR(W_r); REQ_PTR(W_gate); REQ_PTR(W_up); REQ_PTR(W_down); REQ_PTR_T(topk_idx); REQ_PTR_T(topk_gate);
    REQ_PTR(counts); REQ_PTR(offsets); REQ_PTR_T(perm_row); REQ_PTR_T(row_src); REQ_PTR_T(Y);
    const mop_moe_shape& s = c->s;
    if ((r = mop_moe_route(c, x, W_r, bias, topk_idx, topk_gate, nullptr, stream)) != MOP_OK) return r;
    if ((r = mop_moe_permute(c, nullptr, topk_idx, counts, offsets, perm_row, row_src, nullptr, stream)) != MOP_OK) return r;
    if (s.T == 0) return MOP_OK;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MOP_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const ChunkLayout L = chunk_layout(s, n_chunks, 0);
    char* w = static_cast<char*>(workspace);
    const int blocks = min(ceil_div(s.T, 8), c->sm_count * 8);
    c->plan.rows_override = L.cap;
    for (int i = 0; i < n_chunks && r == MOP_OK; ++i) {
        if ((r = chunk_begin(c, L, w, i, n_chunks, x, L.Xp, offsets, perm_row, row_src, true, st)) != MOP_OK) break;
        TcFwdArgs a{};
        a.Xp = reinterpret_cast<const bf16*>(w + L.Xp); a.offsets = reinterpret_cast<const int32_t*>(w + L.off_c);
        a.row_src = reinterpret_cast<const int32_t*>(w + L.row_src_c); a.gate = topk_gate;
        a.W_gate = static_cast<const bf16*>(W_gate); a.W_up = static_cast<const bf16*>(W_up);
        a.W_down = static_cast<const bf16*>(W_down);
        a.H = reinterpret_cast<bf16*>(w + L.H); a.Yp = reinterpret_cast<bf16*>(w + L.Yp);
        int n = 0;
        r = tc_ffn_fwd(&c->plan, a, c->tiles, c->status, st, &n);
        c->launches += n;
        if (r != MOP_OK) break;
        LAUNCH(c, "chunk_combine_acc", st,
               combine_acc_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<const uint4*>(w + L.Yp),
                                                         reinterpret_cast<const int32_t*>(w + L.perm_c),
                                                         reinterpret_cast<float4*>(w + L.acc), static_cast<uint4*>(Y), s.T,
                                                         s.k, s.d / 8, i == 0, i == n_chunks - 1));
        r = after_launch(c);
    }
    c->plan.rows_override = 0;
    return r;
}

mop_status mop_moe_layer_bwd_chunked(mop_ctx* c, int32_t n_chunks, const void* x, const void* dY,
                                     const float* topk_gate, const int32_t* offsets, const int32_t* perm_row,
                                     const int32_t* row_src, const void* W_gate, const void* W_up, const void* W_down,
                                     void* dX, float* dW_gate, float* dW_up, float* dW_down, float* dgate,
                                     void* workspace, void* stream) {
    mop_status r = chunk_check(c, n_chunks, workspace);
    if (r != MOP_OK) return r;
    REQ_PTR_T(x); REQ_PTR_T(dY); REQ_PTR_T(topk_gate); REQ_PTR(offsets); REQ_PTR_T(perm_row); REQ_PTR_T(row_src);
    REQ_PTR(W_gate); REQ_PTR(W_up); REQ_PTR(W_down); REQ_PTR_T(dX); REQ_PTR(dW_gate); REQ_PTR(dW_up); REQ_PTR(dW_down);
    REQ_PTR_T(dgate);
    const mop_moe_shape& s = c->s;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MOP_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t wvec = (size_t)s.d * s.f / 4;
    if (s.T == 0) {
        if (!s.dw_accumulate) {
            const size_t n = (size_t)s.E * s.d * s.f * 4;
            CUDA_OK(cudaMemsetAsync(dW_gate, 0, n, st)); CUDA_OK(cudaMemsetAsync(dW_up, 0, n, st));
            CUDA_OK(cudaMemsetAsync(dW_down, 0, n, st));
        }
        return MOP_OK;
    }
    const ChunkLayout L = chunk_layout(s, n_chunks, 1);
    char* w = static_cast<char*>(workspace);
    const int M = s.T * s.k;
    const int blocks = min(ceil_div(s.T, 8), c->sm_count * 8);
    c->plan.rows_override = L.cap;
    for (int i = 0; i < n_chunks && r == MOP_OK; ++i) {
        // the chunk's inputs again, and its up-projection recomputed (nothing of the forward was kept)
        if ((r = chunk_begin(c, L, w, i, n_chunks, x, L.Xp, offsets, perm_row, row_src, true, st)) != MOP_OK) break;
        if ((r = chunk_begin(c, L, w, i, n_chunks, dY, L.dYp, offsets, perm_row, row_src, false, st)) != MOP_OK) break;
        const int32_t* off_c = reinterpret_cast<const int32_t*>(w + L.off_c);
        const int32_t* row_src_c = reinterpret_cast<const int32_t*>(w + L.row_src_c);
        TcFwdArgs fa{};
        fa.Xp = reinterpret_cast<const bf16*>(w + L.Xp); fa.offsets = off_c;
        fa.W_gate = static_cast<const bf16*>(W_gate); fa.W_up = static_cast<const bf16*>(W_up);
        fa.G_save = reinterpret_cast<bf16*>(w + L.G); fa.U_save = reinterpret_cast<bf16*>(w + L.U);
        fa.H = reinterpret_cast<bf16*>(w + L.H);
        int n = 0;
        r = tc_up_only(&c->plan, fa, c->tiles, c->status, st, &n);
        c->launches += n;
        if (r != MOP_OK) break;
        TcBwdArgs a{};
        a.dYp = reinterpret_cast<const bf16*>(w + L.dYp); a.Xp = fa.Xp; a.G_save = fa.G_save; a.U_save = fa.U_save; a.H = fa.H;
        a.offsets = off_c; a.row_src = row_src_c; a.gate = topk_gate;
        a.W_gate = fa.W_gate; a.W_up = fa.W_up; a.W_down = static_cast<const bf16*>(W_down);
        a.dG = reinterpret_cast<bf16*>(w + L.dG); a.dU = reinterpret_cast<bf16*>(w + L.dU);
        a.gH = reinterpret_cast<bf16*>(w + L.gH); a.dXp = reinterpret_cast<bf16*>(w + L.dXp);
        a.part = reinterpret_cast<float*>(w + L.part);
        a.dW_gate = dW_gate; a.dW_up = dW_up; a.dW_down = dW_down; a.accumulate = s.dw_accumulate; a.keep_empty = 1;
        int ntile_part = 0;
        n = 0;
        r = tc_ffn_bwd(&c->plan, a, c->tiles, c->status, st, &n, &ntile_part);
        c->launches += n;
        if (r != MOP_OK) break;
        LAUNCH(c, "chunk_dgate_reduce", st,
               dgate_reduce_chunk_kernel<<<ceil_div(M, 256), 256, 0, st>>>(a.part, reinterpret_cast<const int32_t*>(w + L.perm_c),
                                                                           dgate, M, (int)L.cap, ntile_part));
        if ((r = after_launch(c)) != MOP_OK) break;
        LAUNCH(c, "chunk_combine_acc", st,
               combine_acc_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<const uint4*>(w + L.dXp),
                                                         reinterpret_cast<const int32_t*>(w + L.perm_c),
                                                         reinterpret_cast<float4*>(w + L.acc), static_cast<uint4*>(dX), s.T,
                                                         s.k, s.d / 8, i == 0, i == n_chunks - 1));
        r = after_launch(c);
    }
    c->plan.rows_override = 0;
    if (r != MOP_OK) return r;
    if (!s.dw_accumulate) {   // experts that received no row: zero gradients
        dim3 gz((unsigned)min((size_t)64, (wvec + 255) / 256), s.E);
        LAUNCH(c, "chunk_zero_empty_experts", st,
               zero_empty_experts_kernel<<<gz, 256, 0, st>>>(offsets, reinterpret_cast<float4*>(dW_gate),
                                                             reinterpret_cast<float4*>(dW_up),
                                                             reinterpret_cast<float4*>(dW_down), wvec));
        r = after_launch(c);
    }
    return r;
}

mop_status mop_moe_route_bwd(mop_ctx* c, const float* logits, const float* bias, const int32_t* topk_idx,
                             const float* topk_gate, const float* dgate, const void* Xp, const int32_t* offsets,
                             const int32_t* perm_row, const float* W_r, float* dW_r, float* dbias_opt, void* dX,
                             void* stream) {
    if (!c) return MOP_ERR_INVALID_ARG;
    if (!c->s.with_backward) return MOP_ERR_UNSUPPORTED;
    REQ_PTR_T(logits); REQ_PTR_T(topk_idx); REQ_PTR_T(topk_gate); REQ_PTR_T(dgate); REQ_PTR_T(Xp); REQ_PTR(offsets);
    REQ_PTR_T(perm_row); REQ_PTR(W_r); REQ_PTR(dW_r); REQ_PTR_T(dX);
    if ((c->s.bias_mode != MOP_BIAS_NONE) != (bias != nullptr)) return MOP_ERR_INVALID_ARG;
    if (dbias_opt && !aligned16(dbias_opt)) return MOP_ERR_ALIGN;
    const mop_moe_shape& s = c->s;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MOP_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    mop_status r;
    if (s.T > 0) {
        LAUNCH(c, "route_bwd_dz", st,
               route_bwd_dz_kernel<<<ceil_div(s.T, 8), 256, 0, st>>>(logits, bias, topk_idx, topk_gate, dgate, perm_row,
                                                                     c->dz_sel, c->dz_row, s.T, s.E, s.k, s.score_fn,
                                                                     s.bias_mode));
        if ((r = after_launch(c)) != MOP_OK) return r;
    }
    dim3 gw(ceil_div(s.d, 1024), s.E);
    float* db = (dbias_opt && s.bias_mode == MOP_BIAS_PRE_LOGIT) ? dbias_opt : nullptr;
    if (dbias_opt && !db) CUDA_OK(cudaMemsetAsync(dbias_opt, 0, (size_t)s.E * 4, st));
    LAUNCH(c, "route_bwd_dwr", st,
           route_bwd_dwr_kernel<<<gw, 128, 0, st>>>(static_cast<const bf16*>(Xp), c->dz_row, offsets, dW_r, db, s.d, s.E));
    if ((r = after_launch(c)) != MOP_OK) return r;
    if (s.T == 0) return MOP_OK;
    dim3 gt(ceil_div(s.E, 32), ceil_div(s.d, 32));
    LAUNCH(c, "route_bwd_wrT", st, transpose_f32_kernel<<<gt, 256, 0, st>>>(W_r, c->wrT, s.d, s.E));
    if ((r = after_launch(c)) != MOP_OK) return r;
    LAUNCH(c, "route_bwd_dx", st,
           route_bwd_dx_kernel<<<s.T, 256, 0, st>>>(c->wrT, topk_idx, c->dz_sel, static_cast<bf16*>(dX), s.T, s.d, s.E,
                                                    s.k));
    return after_launch(c);
}

namespace {
mop_status step_host(mop_ctx* c, const void* x_host, const void* dY_host, const float* W_r, const float* bias,
                     const void* W_gate, const void* W_up, const void* W_down, void* Y_host, int32_t* idx_host,
                     float* gate_host, void* dX_host, float* dgate_host, float* dW_gate, float* dW_up, float* dW_down,
                     void* stream) {
    const mop_moe_shape& s = c->s;
    const bool bwd = dY_host != nullptr;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MOP_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t M = (size_t)s.T * s.k, xb = (size_t)s.T * s.d * 2;
    // Copies that the kernels do not wait for run on the context's copy stream: dY comes in while the
    // forward runs, Y (and the routing) goes out while the backward runs.
    cudaStream_t cs = c->copy_stream;
    if (s.T > 0) {
        CUDA_OK(cudaMemcpyAsync(c->hx, x_host, xb, cudaMemcpyHostToDevice, st));
        if (bwd) {
            CUDA_OK(cudaEventRecord(c->ev_in, st));            // orders the copy stream after earlier work on st
            CUDA_OK(cudaStreamWaitEvent(cs, c->ev_in, 0));
            CUDA_OK(cudaMemcpyAsync(c->hdY, dY_host, xb, cudaMemcpyHostToDevice, cs));
            CUDA_OK(cudaEventRecord(c->ev_in, cs));
        }
    }
    mop_status r;
    if ((r = mop_moe_route(c, c->hx, W_r, bias, c->hidx, c->hgate, nullptr, stream)) != MOP_OK) return r;
    if ((r = mop_moe_permute(c, c->hx, c->hidx, c->hcounts, c->hoffsets, c->hperm, c->hsrc, c->hXp, stream)) != MOP_OK)
        return r;
    if ((r = mop_moe_expert_ffn_fwd(c, c->hXp, c->hoffsets, c->hsrc, c->hgate, W_gate, W_up, W_down,
                                    bwd ? c->hG : nullptr, bwd ? c->hU : nullptr, c->hH, c->hYp, stream)) != MOP_OK)
        return r;
    if ((r = mop_moe_combine(c, c->hYp, c->hperm, c->hY, stream)) != MOP_OK) return r;
    if (s.T > 0) {
        cudaStream_t os = bwd ? cs : st;                       // forward only: nothing to overlap with
        if (bwd) {
            CUDA_OK(cudaEventRecord(c->ev_mid, st));
            CUDA_OK(cudaStreamWaitEvent(cs, c->ev_mid, 0));
        }
        CUDA_OK(cudaMemcpyAsync(Y_host, c->hY, xb, cudaMemcpyDeviceToHost, os));
        if (idx_host) CUDA_OK(cudaMemcpyAsync(idx_host, c->hidx, M * 4, cudaMemcpyDeviceToHost, os));
        if (gate_host) CUDA_OK(cudaMemcpyAsync(gate_host, c->hgate, M * 4, cudaMemcpyDeviceToHost, os));
        if (bwd) CUDA_OK(cudaEventRecord(c->ev_out, cs));
    }
    if (bwd) {
        if (s.T > 0) CUDA_OK(cudaStreamWaitEvent(st, c->ev_in, 0));   // dY has arrived
        if ((r = mop_moe_expert_ffn_bwd(c, c->hdY, c->hXp, c->hG, c->hU, c->hH, c->hoffsets, c->hperm, c->hsrc,
                                        c->hgate, W_gate, W_up, W_down, c->hdX, dW_gate, dW_up, dW_down, c->hdgate,
                                        stream)) != MOP_OK)
            return r;
        if (s.T > 0) {
            CUDA_OK(cudaMemcpyAsync(dX_host, c->hdX, xb, cudaMemcpyDeviceToHost, st));
            if (dgate_host) CUDA_OK(cudaMemcpyAsync(dgate_host, c->hdgate, M * 4, cudaMemcpyDeviceToHost, st));
            CUDA_OK(cudaStreamWaitEvent(st, c->ev_out, 0));     // st completes only after the Y copy
        }
    }
    CUDA_OK(cudaStreamSynchronize(st));
    return MOP_OK;
}
}  // namespace

namespace {
// One step on host buffers WITHOUT waiting for it: step i's inputs come in on the copy stream while
// step i-1 computes, its results leave on the output stream while step i+1 computes.  Two slots of
// every buffer a copy touches; per-slot events order the three streams:
//   copy stream   : [slot free: step i-2 computed] -> x, dY in          -> ev_x, ev_dy
//   caller stream : [ev_x] [slot's results of step i-2 copied out] forward -> ev_fwd, [ev_dy] backward -> ev_done
//   output stream : [ev_fwd] Y, idx, gate out; [ev_done] dX, dgate out  -> ev_drained
mop_status step_host_pipelined(mop_ctx* c, const void* x_host, const void* dY_host, const float* W_r,
                               const float* bias, const void* W_gate, const void* W_up, const void* W_down,
                               void* Y_host, int32_t* idx_host, float* gate_host, void* dX_host, float* dgate_host,
                               float* dW_gate, float* dW_up, float* dW_down, void* stream) {
    const mop_moe_shape& s = c->s;
    const bool bwd = dY_host != nullptr;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MOP_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream), in = c->copy_stream, out = c->out_stream;
    const size_t M = (size_t)s.T * s.k, xb = (size_t)s.T * s.d * 2;
    const int q = (int)(c->host_steps++ & 1);
    if (s.T > 0) {
        CUDA_OK(cudaStreamWaitEvent(in, c->ev_done[q], 0));       // step i-2 no longer reads this slot's inputs
        CUDA_OK(cudaMemcpyAsync(c->px[q], x_host, xb, cudaMemcpyHostToDevice, in));
        CUDA_OK(cudaEventRecord(c->ev_x[q], in));
        if (bwd) {
            CUDA_OK(cudaMemcpyAsync(c->pdY[q], dY_host, xb, cudaMemcpyHostToDevice, in));
            CUDA_OK(cudaEventRecord(c->ev_dy[q], in));
        }
        CUDA_OK(cudaStreamWaitEvent(st, c->ev_x[q], 0));
        CUDA_OK(cudaStreamWaitEvent(st, c->ev_drained[q], 0));    // step i-2's results have left this slot
    }
    mop_status r;
    if ((r = mop_moe_route(c, c->px[q], W_r, bias, c->pidx[q], c->pgate[q], nullptr, stream)) != MOP_OK) return r;
    if ((r = mop_moe_permute(c, c->px[q], c->pidx[q], c->hcounts, c->hoffsets, c->hperm, c->hsrc, c->hXp, stream)) !=
        MOP_OK)
        return r;
    if ((r = mop_moe_expert_ffn_fwd(c, c->hXp, c->hoffsets, c->hsrc, c->pgate[q], W_gate, W_up, W_down,
                                    bwd ? c->hG : nullptr, bwd ? c->hU : nullptr, c->hH, c->hYp, stream)) != MOP_OK)
        return r;
    if ((r = mop_moe_combine(c, c->hYp, c->hperm, c->pY[q], stream)) != MOP_OK) return r;
    if (s.T > 0) {
        CUDA_OK(cudaEventRecord(c->ev_fwd[q], st));
        CUDA_OK(cudaStreamWaitEvent(out, c->ev_fwd[q], 0));
        CUDA_OK(cudaMemcpyAsync(Y_host, c->pY[q], xb, cudaMemcpyDeviceToHost, out));
        if (idx_host) CUDA_OK(cudaMemcpyAsync(idx_host, c->pidx[q], M * 4, cudaMemcpyDeviceToHost, out));
        if (gate_host) CUDA_OK(cudaMemcpyAsync(gate_host, c->pgate[q], M * 4, cudaMemcpyDeviceToHost, out));
    }
    if (bwd) {
        if (s.T > 0) CUDA_OK(cudaStreamWaitEvent(st, c->ev_dy[q], 0));
        if ((r = mop_moe_expert_ffn_bwd(c, c->pdY[q], c->hXp, c->hG, c->hU, c->hH, c->hoffsets, c->hperm, c->hsrc,
                                        c->pgate[q], W_gate, W_up, W_down, c->pdX[q], dW_gate, dW_up, dW_down,
                                        c->pdgate[q], stream)) != MOP_OK)
            return r;
    }
    if (s.T > 0) {
        CUDA_OK(cudaEventRecord(c->ev_done[q], st));
        if (bwd) {
            CUDA_OK(cudaStreamWaitEvent(out, c->ev_done[q], 0));
            CUDA_OK(cudaMemcpyAsync(dX_host, c->pdX[q], xb, cudaMemcpyDeviceToHost, out));
            if (dgate_host) CUDA_OK(cudaMemcpyAsync(dgate_host, c->pdgate[q], M * 4, cudaMemcpyDeviceToHost, out));
        }
        CUDA_OK(cudaEventRecord(c->ev_drained[q], out));
    }
    return MOP_OK;
}
}  // namespace

mop_status mop_moe_forward_host_async(mop_ctx* c, const void* x_host, const float* W_r, const float* bias,
                                      const void* W_gate, const void* W_up, const void* W_down, void* Y_host,
                                      int32_t* idx_host, float* gate_host, void* stream) {
    if (!c) return MOP_ERR_INVALID_ARG;
    if (c->s.T > 0 && (!x_host || !Y_host)) return MOP_ERR_INVALID_ARG;
    if (c->s.host_io != 2) return MOP_ERR_UNSUPPORTED;
    return step_host_pipelined(c, x_host, nullptr, W_r, bias, W_gate, W_up, W_down, Y_host, idx_host, gate_host,
                               nullptr, nullptr, nullptr, nullptr, nullptr, stream);
}

mop_status mop_moe_train_step_host_async(mop_ctx* c, const void* x_host, const void* dY_host, const float* W_r,
                                         const float* bias, const void* W_gate, const void* W_up, const void* W_down,
                                         void* Y_host, void* dX_host, float* dgate_host, float* dW_gate,
                                         float* dW_up, float* dW_down, void* stream) {
    if (!c) return MOP_ERR_INVALID_ARG;
    if (c->s.T > 0 && (!x_host || !dY_host || !Y_host || !dX_host)) return MOP_ERR_INVALID_ARG;
    if (c->s.host_io != 2 || !c->s.with_backward) return MOP_ERR_UNSUPPORTED;
    if (c->s.T == 0 && !dY_host) dY_host = c;  // any non-null token: selects the backward branch
    return step_host_pipelined(c, x_host, dY_host, W_r, bias, W_gate, W_up, W_down, Y_host, nullptr, nullptr,
                               dX_host, dgate_host, dW_gate, dW_up, dW_down, stream);
}

mop_status mop_host_drain(mop_ctx* c, void* stream) {
    if (!c) return MOP_ERR_INVALID_ARG;
    if (c->s.host_io != 2) return MOP_ERR_UNSUPPORTED;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MOP_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    for (int q = 0; q < 2; ++q) CUDA_OK(cudaStreamWaitEvent(st, c->ev_drained[q], 0));
    CUDA_OK(cudaStreamSynchronize(st));
    return MOP_OK;
}

mop_status mop_moe_forward_host(mop_ctx* c, const void* x_host, const float* W_r, const float* bias,
                                const void* W_gate, const void* W_up, const void* W_down, void* Y_host,
                                int32_t* idx_host, float* gate_host, void* stream) {
    if (!c) return MOP_ERR_INVALID_ARG;
    if (c->s.T > 0 && (!x_host || !Y_host)) return MOP_ERR_INVALID_ARG;
    if (!c->s.host_io) return MOP_ERR_UNSUPPORTED;
    return step_host(c, x_host, nullptr, W_r, bias, W_gate, W_up, W_down, Y_host, idx_host, gate_host, nullptr,
                     nullptr, nullptr, nullptr, nullptr, stream);
}

mop_status mop_moe_train_step_host(mop_ctx* c, const void* x_host, const void* dY_host, const float* W_r,
                                   const float* bias, const void* W_gate, const void* W_up, const void* W_down,
                                   void* Y_host, void* dX_host, float* dgate_host, float* dW_gate, float* dW_up,
                                   float* dW_down, void* stream) {
    if (!c) return MOP_ERR_INVALID_ARG;
    if (c->s.T > 0 && (!x_host || !dY_host || !Y_host || !dX_host)) return MOP_ERR_INVALID_ARG;
    if (!c->s.host_io || !c->s.with_backward) return MOP_ERR_UNSUPPORTED;
    if (c->s.T == 0 && !dY_host) dY_host = c;  // any non-null token: selects the backward branch
    return step_host(c, x_host, dY_host, W_r, bias, W_gate, W_up, W_down, Y_host, nullptr, nullptr, dX_host,
                     dgate_host, dW_gate, dW_up, dW_down, stream);
}

mop_status mop_profile_enable(mop_ctx* c, int on) {
    if (!c) return MOP_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return MOP_ERR_CUDA;
    if (on && !c->prof.ev) {
        c->prof.ev = new (std::nothrow) cudaEvent_t[2 * Profiler::MAX_REC];
        if (!c->prof.ev) return MOP_ERR_WORKSPACE;
        for (int i = 0; i < 2 * Profiler::MAX_REC; ++i)
            if (cudaEventCreate(&c->prof.ev[i]) != cudaSuccess) return MOP_ERR_CUDA;
    }
    c->prof.on = on != 0;
    c->prof.n = 0;
    return MOP_OK;
}

int32_t mop_profile_read(mop_ctx* c, void* stream, int32_t max_names, const char** names, float* total_ms,
                         int32_t* calls) {
    if (!c || !names || !total_ms || !calls || max_names < 1) return -1;
    DeviceGuard guard(c->device);
    if (!guard.ok) return -1;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return -1;
    int32_t n = 0;
    for (int i = 0; i < c->prof.n; ++i) {
        float ms = 0.0f;
        if (cudaEventElapsedTime(&ms, c->prof.ev[2 * i], c->prof.ev[2 * i + 1]) != cudaSuccess) return -1;
        int32_t j = 0;
        while (j < n && names[j] != c->prof.names[i]) ++j;   // names are string literals: compare pointers
        if (j == n) {
            if (n == max_names) continue;
            names[n] = c->prof.names[i]; total_ms[n] = 0.0f; calls[n] = 0; ++n;
        }
        total_ms[j] += ms;
        calls[j] += 1;
    }
    c->prof.n = 0;
    return n;
}

// ---------------------------------------------------------------------------------------------
// Permutation without any allocation.  Some callers may not call cudaMalloc at all: a serving
// or training process that handed the whole HBM to its own arena at start-up (a second
// allocator would fail or fragment it), or a latency-critical loop that cannot afford the
// device-wide synchronisation an allocation implies.  mop_create allocates, so those callers
// cannot hold a context.  For them the unit histogram of the permutation lives in the
// file-scope device array below, which every GPU that loads this library holds until exit.
// ---------------------------------------------------------------------------------------------
#define MOP_STATIC_SCRATCH_INTS 262144   /* 1 MiB: ceil(T*k/512) * E entries must fit */
static __device__ __align__(256) int32_t g_static_scratch[MOP_STATIC_SCRATCH_INTS];

namespace {
constexpr int kMaxDevices = 64;
struct StaticSetup { bool done; int32_t* scratch; int sm_count; };
StaticSetup g_static_setup[kMaxDevices];   // zero-initialised
std::mutex g_static_mutex;

// Device address of g_static_scratch on `device` (which must be current).  In host code the
// array's name is only a handle; the kernels need the address that cudaGetSymbolAddress returns
// for the current device.
mop_status static_setup(int device, StaticSetup* out) {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticSetup& s = g_static_setup[device];
    if (!s.done) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return MOP_ERR_CUDA;
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return MOP_ERR_CUDA;
        s.scratch = static_cast<int32_t*>(ptr);
        s.sm_count = sms;
        s.done = true;
    }
    *out = s;
    return MOP_OK;
}
}  // namespace

mop_status mop_moe_permute_static(int device, int32_t T, int32_t d, int32_t E, int32_t k, const void* x,
                                  const int32_t* topk_idx, int32_t* counts, int32_t* offsets, int32_t* perm_row,
                                  int32_t* row_src, void* Xp, void* stream) {
    if (T < 0 || d < 1 || E < 1 || k < 1 || k > E) return MOP_ERR_INVALID_ARG;
    if (d % 8) return MOP_ERR_ALIGN;
    if (E > SEL_MAX_E || k > 32 || (long long)T * k >= (1ll << 31) - 4096) return MOP_ERR_SHAPE;
    const int M = T * k;
    const int units = ceil_div(M, PERM_SEG);
    if ((long long)units * E > MOP_STATIC_SCRATCH_INTS) return MOP_ERR_SHAPE;   // beyond the static scratch
    if (!counts || !offsets) return MOP_ERR_INVALID_ARG;
    if (!aligned16(counts) || !aligned16(offsets)) return MOP_ERR_ALIGN;
    if (T > 0) {
        if (!topk_idx || !perm_row || !row_src) return MOP_ERR_INVALID_ARG;
        if (!aligned16(topk_idx) || !aligned16(perm_row) || !aligned16(row_src)) return MOP_ERR_ALIGN;
        if (Xp) {                                   // Xp == NULL: tables only, as in mop_moe_permute
            if (!x) return MOP_ERR_INVALID_ARG;
            if (!aligned16(x) || !aligned16(Xp)) return MOP_ERR_ALIGN;
        }
    }
    if (device < 0 || device >= kMaxDevices) return MOP_ERR_INVALID_ARG;
    DeviceGuard guard(device);
    if (!guard.ok) return MOP_ERR_CUDA;
    StaticSetup su;
    mop_status r = static_setup(device, &su);
    if (r != MOP_OK) return r;
    cudaGetLastError();                             // an error left by an earlier call is not this call's
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t smem = (size_t)PERM_WARPS * E * sizeof(int32_t);
    // Nothing in the scratch has to start at zero: the histogram kernel writes every entry
    // [unit][expert] that the scan and rank kernels read, so a previous call's contents are dead.
    if (units > 0) {
        perm_hist_kernel<<<ceil_div(units, PERM_WARPS), PERM_WARPS * 32, smem, st>>>(topk_idx, su.scratch, M, E);
        if (cudaGetLastError() != cudaSuccess) return MOP_ERR_CUDA;
    }
    if (units == 0) {
        perm_scan_kernel<<<1, 1024, (E + 1) * sizeof(int32_t), st>>>(su.scratch, counts, offsets, units, E);
        return cudaGetLastError() == cudaSuccess ? MOP_OK : MOP_ERR_CUDA;
    }
    perm_scan_cols_kernel<<<ceil_div(E, 32), PSCAN_WARPS * 32, 0, st>>>(su.scratch, counts, units, E);
    if (cudaGetLastError() != cudaSuccess) return MOP_ERR_CUDA;
    perm_rank_kernel<<<ceil_div(units, PERM_WARPS), PERM_WARPS * 32, smem + (E + 1) * sizeof(int32_t), st>>>(
        topk_idx, su.scratch, counts, offsets, perm_row, row_src, M, E);
    if (cudaGetLastError() != cudaSuccess) return MOP_ERR_CUDA;
    if (!Xp) return MOP_OK;
    launch_scatter_rows(static_cast<const uint4*>(x), static_cast<uint4*>(Xp), perm_row, T, k, d / 8, su.sm_count, st);
    return cudaGetLastError() == cudaSuccess ? MOP_OK : MOP_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// Vocabulary projection + online log-likelihood (no context: the caller owns the workspace)
// ---------------------------------------------------------------------------------------------
namespace {
struct VocabLayout { size_t off, tiles, status, ylab, part, total; };
VocabLayout vocab_layout(int N, int V) {
    VocabLayout L{};
    size_t o = 0;
    auto take = [&](size_t b) { size_t r = o; o += align_up(b); return r; };
    L.status = take(256);                 // first: mop_vocab_poll reads it without knowing the shape
    L.off = take(16);
    L.tiles = take(tc_tile_table_bytes(N, 1));
    L.ylab = take((size_t)N * 4);
    L.part = take((size_t)ceil_div(V, 256) * N * 8);
    L.total = o;
    return L;
}
std::mutex g_vocab_mutex;
TcPlan g_vocab_plan[kMaxDevices];
Profiler g_vocab_prof;           // never enabled: the plan needs one
bool g_vocab_ready[kMaxDevices];
mop_status vocab_plan(int device, TcPlan** out) {
    TcPlan* p = &g_vocab_plan[device];
    std::lock_guard<std::mutex> lock(g_vocab_mutex);
    if (!g_vocab_ready[device]) {
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return MOP_ERR_CUDA;
        if (prop.major != 10) return MOP_ERR_UNSUPPORTED;
        mop_moe_shape dummy{};
        mop_status r = tc_plan_init(p, dummy, prop.multiProcessorCount, &g_vocab_prof);
        if (r == MOP_OK) r = tc2_init();
        if (r != MOP_OK) return r;
        g_vocab_ready[device] = true;
    }
    *out = p;
    return MOP_OK;
}
}  // namespace

size_t mop_vocab_workspace_bytes(int32_t N, int32_t H, int32_t V) {
    if (N < 0 || H < 64 || V < 64 || H % 64 || V % 64) return 0;
    return vocab_layout(N, V).total;
}

mop_status mop_vocab_loss_fwd(int device, int32_t N, int32_t H, int32_t V, const void* X, const void* W_voc,
                              const int32_t* targets, float* loss, float* lse_opt, void* workspace, void* stream) {
    if (N < 0 || H < 1 || V < 1) return MOP_ERR_INVALID_ARG;
    if (H % 64 || V % 64) return MOP_ERR_UNSUPPORTED;
    if ((long long)N * 2 >= (1ll << 31) || (long long)H * V >= (1ll << 40)) return MOP_ERR_SHAPE;
    if (N == 0) return MOP_OK;
    if (!X || !W_voc || !targets || !loss || !workspace) return MOP_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(W_voc) || !aligned16(targets) || !aligned16(loss) ||
        (reinterpret_cast<uintptr_t>(workspace) & 255u) || (lse_opt && !aligned16(lse_opt)))
        return MOP_ERR_ALIGN;
    if (device < 0 || device >= kMaxDevices) return MOP_ERR_INVALID_ARG;
    DeviceGuard guard(device);
    if (!guard.ok) return MOP_ERR_CUDA;
    TcPlan* p = nullptr;
    {
        mop_status pr = vocab_plan(device, &p);
        if (pr != MOP_OK) return pr;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const VocabLayout L = vocab_layout(N, V);
    char* w = static_cast<char*>(workspace);
    int32_t* off = reinterpret_cast<int32_t*>(w + L.off);
    int32_t* tiles = reinterpret_cast<int32_t*>(w + L.tiles);
    int32_t* status = reinterpret_cast<int32_t*>(w + L.status);
    float* ylab = reinterpret_cast<float*>(w + L.ylab);
    float* part = reinterpret_cast<float*>(w + L.part);
    const int32_t host_off[2] = {0, N};
    CUDA_OK(cudaMemcpyAsync(off, host_off, sizeof(host_off), cudaMemcpyHostToDevice, st));
    CUDA_OK(cudaMemsetAsync(status, 0, 4, st));
    const bool pair = false;                // measured: the one-CTA kernel is as fast here (online log-sum-exp epilogue)
    if (pair) tc_build_pairtiles_kernel<<<1, 1024, 0, st>>>(off, 1, reinterpret_cast<int4*>(tiles + 64), tiles);
    else tc_build_mtiles_kernel<<<1, 1024, 0, st>>>(off, 1, reinterpret_cast<int4*>(tiles + 64), tiles);
    CUtensorMap mX, mW;
    if (!tc_map_2d(p, &mX, X, N, H, 128) || !tc_map_chunked_3d(p, &mW, W_voc, 1, H, V, pair ? 2 : 4)) return MOP_ERR_CUDA;
    TcArgs g{};
    g.offsets = off; g.n_mtiles = tiles; g.mtiles = reinterpret_cast<const int4*>(tiles + 64);
    g.E = 1; g.status = status;
    g.tiles_n = ceil_div(V, 256); g.kblocks = ceil_div(H, TC_BK); g.N = V; g.m_fastest = 1;
    g.targets = targets; g.ylab = ylab; g.ep.part = part; g.ep.M_total = N;
    mop_status r = pair ? tc2_launch<TC_VL>(p, "vocab_logits_lse", mX, mX, mW, mW, g, st)
                        : tc_launch<TC_VL>(p, "vocab_logits_lse", mX, mX, mW, mW, mX, mX, g, st);
    if (r != MOP_OK) return r;
    vocab_lse_merge_kernel<<<ceil_div(N, 256), 256, 0, st>>>(reinterpret_cast<const float2*>(part), ylab, loss,
                                                            lse_opt, N, g.tiles_n);
    return cudaGetLastError() == cudaSuccess ? MOP_OK : MOP_ERR_CUDA;
}

namespace {
constexpr int kVocabBlock = 8192;   // vocabulary columns whose logit gradients are live at a time
struct VocabBwdLayout { size_t off, tiles, status, dy, dx32, total; int vc; };
VocabBwdLayout vocab_bwd_layout(int N, int H, int V) {
    VocabBwdLayout L{};
    size_t o = 0;
    auto take = [&](size_t b) { size_t r = o; o += align_up(b); return r; };
    L.vc = V < kVocabBlock ? V : kVocabBlock;
    L.status = take(256);                 // first, as in the forward's workspace
    L.off = take(16);
    L.tiles = take(tc_tile_table_bytes(N, 1));
    L.dy = take((size_t)N * L.vc * 2);
    L.dx32 = take((size_t)N * H * 4);
    L.total = o;
    return L;
}
}  // namespace

mop_status mop_vocab_poll(int device, void* workspace, void* stream) {
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return MOP_ERR_INVALID_ARG;
    if (device < 0 || device >= kMaxDevices) return MOP_ERR_INVALID_ARG;
    DeviceGuard guard(device);
    if (!guard.ok) return MOP_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t word = 0;   // both vocabulary workspaces start with their status block
    CUDA_OK(cudaMemcpyAsync(&word, workspace, 4, cudaMemcpyDeviceToHost, st));
    CUDA_OK(cudaStreamSynchronize(st));
    if (word != 0) {
        CUDA_OK(cudaMemsetAsync(workspace, 0, 4, st));
        CUDA_OK(cudaStreamSynchronize(st));
        return MOP_ERR_TIMEOUT;
    }
    return MOP_OK;
}

mop_status mop_vocab_selftest_wait_timeout(int device, void* workspace, int64_t limit_cycles, void* stream) {
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return MOP_ERR_INVALID_ARG;
    if (limit_cycles < 1 || limit_cycles > 4000000000ll || device < 0 || device >= kMaxDevices) return MOP_ERR_INVALID_ARG;
    DeviceGuard guard(device);
    if (!guard.ok) return MOP_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t* status = static_cast<int32_t*>(workspace);
    int32_t* gave_up = status + 8;                       // a spare word of the status block
    CUDA_OK(cudaMemsetAsync(gave_up, 0, 4, st));
    tc_wait_selftest_kernel<<<1, 32, 0, st>>>(status, limit_cycles, gave_up);
    if (cudaGetLastError() != cudaSuccess) return MOP_ERR_CUDA;
    int32_t flag = 0;
    CUDA_OK(cudaMemcpyAsync(&flag, gave_up, 4, cudaMemcpyDeviceToHost, st));
    CUDA_OK(cudaStreamSynchronize(st));
    return flag == 1 ? MOP_OK : MOP_ERR_CUDA;
}

size_t mop_vocab_bwd_workspace_bytes(int32_t N, int32_t H, int32_t V) {
    if (N < 0 || H < 64 || V < 64 || H % 64 || V % 64) return 0;
    return vocab_bwd_layout(N, H, V).total;
}

mop_status mop_vocab_loss_bwd(int device, int32_t N, int32_t H, int32_t V, const void* X, const void* W_voc,
                              const int32_t* targets, const float* lse, const float* dloss, void* dX, float* dW_voc,
                              void* workspace, void* stream) {
    if (N < 0 || H < 1 || V < 1) return MOP_ERR_INVALID_ARG;
    if (H % 64 || V % 64) return MOP_ERR_UNSUPPORTED;
    if ((long long)N * 2 >= (1ll << 31) || (long long)H * V >= (1ll << 40)) return MOP_ERR_SHAPE;
    if (!W_voc || !dW_voc || !workspace) return MOP_ERR_INVALID_ARG;
    if (N > 0 && (!X || !targets || !lse || !dloss || !dX)) return MOP_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(W_voc) || !aligned16(targets) || !aligned16(lse) || !aligned16(dloss) ||
        !aligned16(dX) || !aligned16(dW_voc) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return MOP_ERR_ALIGN;
    if (device < 0 || device >= kMaxDevices) return MOP_ERR_INVALID_ARG;
    DeviceGuard guard(device);
    if (!guard.ok) return MOP_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (N == 0) {   // no tokens: the weight gradient is zero
        CUDA_OK(cudaMemsetAsync(dW_voc, 0, (size_t)H * V * 4, st));
        return MOP_OK;
    }
    TcPlan* p = nullptr;
    mop_status r = vocab_plan(device, &p);
    if (r != MOP_OK) return r;
    const VocabBwdLayout L = vocab_bwd_layout(N, H, V);
    char* w = static_cast<char*>(workspace);
    int32_t* off = reinterpret_cast<int32_t*>(w + L.off);
    int32_t* tiles = reinterpret_cast<int32_t*>(w + L.tiles);
    int32_t* status = reinterpret_cast<int32_t*>(w + L.status);
    bf16* dY = reinterpret_cast<bf16*>(w + L.dy);
    float* dx32 = reinterpret_cast<float*>(w + L.dx32);
    const int32_t host_off[2] = {0, N};
    CUDA_OK(cudaMemcpyAsync(off, host_off, sizeof(host_off), cudaMemcpyHostToDevice, st));
    CUDA_OK(cudaMemsetAsync(status, 0, 4, st));
    const bool pair = p->sm_count >= 2;     // dY and dX products on the two-CTA kernel (256-row pair tiles)
    if (pair) tc_build_pairtiles_kernel<<<1, 1024, 0, st>>>(off, 1, reinterpret_cast<int4*>(tiles + 64), tiles);
    else tc_build_mtiles_kernel<<<1, 1024, 0, st>>>(off, 1, reinterpret_cast<int4*>(tiles + 64), tiles);
    CUtensorMap mX, mXT, mWn, mWk;
    if (!tc_map_2d(p, &mX, X, N, H, 128) || !tc_map_chunked_2d(p, &mXT, X, N, H, 2) ||
        !tc_map_chunked_3d(p, &mWn, W_voc, 1, H, V, pair ? 2 : 4) || !tc_map_3d(p, &mWk, W_voc, 1, H, V, pair ? 128 : 256))
        return MOP_ERR_CUDA;
    for (int c0 = 0; c0 < V; c0 += L.vc) {
        const int cw = V - c0 < L.vc ? V - c0 : L.vc;
        CUtensorMap mdYk, mdYn, mOut;
        if (!tc_map_2d_pitch(p, &mdYk, dY, N, cw, L.vc, 128) || !tc_map_chunked_2d_pitch(p, &mdYn, dY, N, cw, L.vc, 4) ||
            !tc_map_out_f32_pitch(p, &mOut, dW_voc + c0, H, cw, V))
            return MOP_ERR_CUDA;
        TcArgs base{};
        base.offsets = off; base.n_mtiles = tiles; base.mtiles = reinterpret_cast<const int4*>(tiles + 64);
        base.E = 1; base.status = status; base.ep.M_total = N;
        {   // dY block = g ([v = t] - exp(X W - lse)), logits recomputed on the tensor cores
            TcArgs g = base;
            g.tiles_n = ceil_div(cw, 256); g.kblocks = ceil_div(H, TC_BK); g.N = V; g.m_fastest = 1; g.n_base = c0;
            g.targets = targets; g.row_lse = lse; g.row_g = dloss; g.ep.out0 = dY; g.ep.ldo = L.vc;
            r = pair ? tc2_launch<TC_VP>(p, "vocab_dlogits", mX, mX, mWn, mWn, g, st)
                     : tc_launch<TC_VP>(p, "vocab_dlogits", mX, mX, mWn, mWn, mX, mX, g, st);
            if (r != MOP_OK) return r;
        }
        {   // dW[:, block] = X^T dY (K = the N tokens), written once
            TcArgs g = base;
            g.tiles_n = ceil_div(cw, 256); g.tiles_m_fixed = ceil_div(H, TC_BM); g.Mfix = H; g.N = cw;
            g.ep.outf = dW_voc + c0; g.ep.accumulate = 0;
            if ((r = tc_launch<TC_WD>(p, "vocab_wgrad", mXT, mXT, mdYn, mdYn, mOut, mOut, g, st)) != MOP_OK) return r;
        }
        {   // dX += dY W[:, block]^T in fp32 across the blocks
            TcArgs g = base;
            g.tiles_n = ceil_div(H, 256); g.kblocks = ceil_div(cw, TC_BK); g.N = H; g.kb_base = c0;
            g.ep.outf = dx32; g.ep.accumulate = c0 > 0 ? 1 : 0;
            r = pair ? tc2_launch<TC_VX>(p, "vocab_dgrad", mdYk, mdYk, mWk, mWk, g, st)
                     : tc_launch<TC_VX>(p, "vocab_dgrad", mdYk, mdYk, mWk, mWk, mX, mX, g, st);
            if (r != MOP_OK) return r;
        }
    }
    const size_t n8 = (size_t)N * H / 8;
    const size_t cap = (size_t)p->sm_count * 16;
    f32_to_bf16_kernel<<<(unsigned)((n8 + 255) / 256 < cap ? (n8 + 255) / 256 : cap), 256, 0, st>>>(
        reinterpret_cast<const float4*>(dx32), static_cast<uint4*>(dX), n8);
    return cudaGetLastError() == cudaSuccess ? MOP_OK : MOP_ERR_CUDA;
}

}  // extern "C"
