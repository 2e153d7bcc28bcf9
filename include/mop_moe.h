/* mop_moe.h -- C ABI of the B200 (sm_100a) routed-expert feed-forward layer.
 *
 * The layer is the MoE block of Section 2.1 of the paper ("Mixture-of-Experts" paragraph):
 * E parallel expert networks and a router that sends each token to its top-k experts.
 * Symbols follow Section 3.1: T tokens resident on the device (the paper's N), model width d
 * (H), expert intermediate width f (I), E experts, routing degree k.  The buffers named Xp and
 * H below are the O(N k H) and O(N_r I) terms of the activation peak in Eq. 4.
 *
 * Conventions for every call
 *   - All tensor pointers are DEVICE pointers owned by the caller, 16-byte aligned, dense and
 *     row-major with the shape given in the comment.  "bf16" means bfloat16 bit patterns.
 *     The library allocates no tensor and keeps no pointer after the call's stream work ends.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls
 *     enqueue work and return; they do not synchronise.
 *   - Argument errors are detected on the host before any launch and reported by the return
 *     code; nothing is thrown, nothing aborts.  Kernels never trap: a wait that runs out of
 *     its poll budget records a code in the context's status word, which mop_poll() reads.
 *   - d and f must be multiples of 8 (16-byte rows); the tensor-core kernels further need
 *     d and f to be multiples of 64 and otherwise the call uses the scalar kernels.
 *   - No output is produced with atomics: results are bitwise reproducible run to run.
 *   - A context is bound to one device and one shape; calls on one context must not overlap
 *     on the GPU (they share its workspace).
 */
#ifndef MOP_MOE_H_
#define MOP_MOE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mop_ctx mop_ctx; /* opaque: shape, workspace, status word */

typedef enum {
    MOP_OK = 0,
    MOP_ERR_INVALID_ARG = 1, /* null pointer, bad enum, k > E, ... */
    MOP_ERR_SHAPE = 2,       /* sizes out of the supported range (T*k >= 2^31, E > 1024, k > 32, ...) */
    MOP_ERR_ALIGN = 3,       /* pointer not 16-byte aligned, or d / f not a multiple of 8 */
    MOP_ERR_WORKSPACE = 4,   /* device allocation of the context's workspace failed */
    MOP_ERR_CUDA = 5,        /* a CUDA runtime or driver call failed */
    MOP_ERR_UNSUPPORTED = 6, /* valid request that this build does not implement */
    MOP_ERR_TIMEOUT = 7      /* a bounded device-side wait ran out (see mop_poll) */
} mop_status;

typedef enum { MOP_SCORE_SOFTMAX = 0, MOP_SCORE_SIGMOID = 1 } mop_score_fn;

/* Where the per-expert router bias enters.  POST_SCORE: key = sigmoid(z) + b (selection
 * only); PRE_LOGIT: key = z + b and the score is taken of z + b.  The bias never enters the
 * gate numerator in POST_SCORE mode. */
typedef enum { MOP_BIAS_NONE = 0, MOP_BIAS_POST_SCORE = 1, MOP_BIAS_PRE_LOGIT = 2 } mop_bias_mode;

/* AUTO: tensor cores when the shape allows, else scalar.  TENSOR: tensor cores or fail.  Both pick
 * per GEMM the schedule measured fastest: the forward down-projection, both data gradients (and the
 * up-projection when d >= 4096) on the two-CTA tokens-on-N kernel, the weight gradients (and the
 * up-projection otherwise) on the one-CTA kernel (128 x 256 tiles).
 * The remaining values force one schedule for testing and measurement: TENSOR_1CTA = one-CTA kernel
 * for all token-row GEMMs; TENSOR_2CTA = two-CTA kernel on 256-row pair tiles; TENSOR_MIXED = full
 * pairs on the two-CTA kernel, remaining rows on the one-CTA kernel; TENSOR_TN = all four token-row
 * GEMMs on the tokens-on-N kernel. */
typedef enum { MOP_GEMM_AUTO = 0, MOP_GEMM_TENSOR = 1, MOP_GEMM_SCALAR = 2, MOP_GEMM_TENSOR_1CTA = 3,
               MOP_GEMM_TENSOR_2CTA = 4, MOP_GEMM_TENSOR_MIXED = 5, MOP_GEMM_TENSOR_TN = 6 } mop_gemm_path;

/* How mop_moe_route computes the logits.  EXACT: one fp32 fused multiply-add chain per (token, expert) on
 * the CUDA cores.  TENSOR: logits on the tensor cores from three bf16 pieces of W_r, then the chain is
 * evaluated only for the experts of a token whose order the approximate keys leave in doubt (needs d and E
 * multiples of 64, else MOP_ERR_UNSUPPORTED).  Both give the same indices in the same order; AUTO takes
 * TENSOR when the scoring is large (2 T d E >= 2e10 flop) and the shape allows it. */
typedef enum { MOP_ROUTE_AUTO = 0, MOP_ROUTE_EXACT = 1, MOP_ROUTE_TENSOR = 2 } mop_route_path;

typedef struct {
    int32_t T, d, E, k, f;
    int32_t score_fn;      /* mop_score_fn */
    int32_t bias_mode;     /* mop_bias_mode; POST_SCORE requires MOP_SCORE_SIGMOID */
    int32_t with_backward; /* 1: the context also holds the backward's intermediates; 2: and buffers to
                              recompute G, U, H in the backward (activation checkpointing) */
    int32_t dw_accumulate; /* 0: dW is overwritten (empty experts get zeros); 1: dW += */
    int32_t gemm_path;     /* mop_gemm_path; AUTO = tensor cores when the shape allows */
    int32_t host_io;       /* 1: the context also holds the activations of the host-buffer entry points;
                              2: and a second slot of every buffer a copy touches, for the *_async forms */
    int32_t route_path;    /* mop_route_path */
} mop_moe_shape;

/* Create / destroy a context on `device` (a CUDA ordinal).  mop_create allocates the
 * workspace (mop_workspace_bytes) with cudaMalloc; every other call allocates nothing. */
mop_status mop_create(mop_ctx** ctx, const mop_moe_shape* shape, int device);
void mop_destroy(mop_ctx* ctx);
size_t mop_workspace_bytes(const mop_moe_shape* shape);
const char* mop_status_string(mop_status s);

/* Synchronises `stream` and returns MOP_ERR_TIMEOUT if any kernel of this context recorded an
 * exhausted wait since the last poll (then clears the word), MOP_ERR_CUDA on a CUDA error. */
mop_status mop_poll(mop_ctx* ctx, void* stream);

/* Self-test of the failure path: launches one thread that waits on a barrier nothing completes, with
 * a limit of `limit_cycles` SM cycles (<= 4e9), synchronises, and returns MOP_OK if the wait gave up
 * and the kernel ended normally.  The kernel records its code in the status word, so the next
 * mop_poll on this context returns MOP_ERR_TIMEOUT (and clears it).  Nothing faults or traps. */
mop_status mop_selftest_wait_timeout(mop_ctx* ctx, int64_t limit_cycles, void* stream);

/* Guard bands of the context's workspace (a check that stands in for a memory checker; the paper has no
 * counterpart).  Every buffer inside the workspace is followed, and the first one preceded, by a
 * 4 KiB band that no kernel may write.  mop_debug_guard_arm fills the bands with a pattern (enqueued on
 * `stream`); mop_debug_guard_check synchronises `stream` and returns in *bad_bytes how many band bytes
 * no longer hold it (0 = no kernel wrote outside its buffers since the bands were armed).
 * mop_debug_guard_poke overwrites one byte of band number `band` from the host side, so that a test can
 * see the check respond without any kernel misbehaving. */
mop_status mop_debug_guard_arm(mop_ctx* ctx, void* stream);
mop_status mop_debug_guard_check(mop_ctx* ctx, int64_t* bad_bytes, void* stream);
mop_status mop_debug_guard_poke(mop_ctx* ctx, int32_t band, int32_t byte, void* stream);

/* Number of kernels launched through this context since it was created. */
int64_t mop_launch_count(const mop_ctx* ctx);

/* The device entry points below (route, permute, expert_ffn_fwd / _gather, combine, expert_ffn_bwd,
 * route_bwd) only enqueue work on `stream`: no allocation, no synchronisation, no host read of device
 * data.  A sequence of them may therefore be captured into a CUDA graph and replayed. */

/* Router of the MoE block (Section 2.1): scores every token against the E experts and keeps its k best.
 *   z[t,e]   = sum_i x[t,i] * W_r[i,e]: one fp32 fused multiply-add per i, i ascending.
 *   key      = z | sigmoid(z) + bias | z + bias       (score_fn, bias_mode)
 *   topk_idx = the k experts with the largest key, descending; equal keys -> lower id.
 *   gate     = score of the selected expert / sum of the k selected scores.
 * x [T,d] bf16; W_r [d,E] f32; bias [E] f32 (NULL iff MOP_BIAS_NONE);
 * topk_idx [T,k] i32 out; topk_gate [T,k] f32 out; logits_opt [T,E] f32 out or NULL.
 * On the tensor-core path (mop_route_path) the returned logits are the chain's value for the experts that
 * were re-evaluated and within 24 * 2^-24 ||x_t|| max_e ||W_r[:,e]|| of it elsewhere, the indices and
 * their order are those of the chain, and the gates agree to 1e-6 + 1e-5 |g|. */
mop_status mop_moe_route(mop_ctx* ctx, const void* x, const float* W_r, const float* bias, int32_t* topk_idx,
                         float* topk_gate, float* logits_opt, void* stream);

/* Statistics of the tensor-core scoring path since the last call: tokens whose approximate keys left the
 * order in doubt, the chains evaluated for them, and how many of those exact logits lay further than half
 * the assumed error bound from their approximation (expected 0: the bound is a model of the rounding
 * errors, and this is its running check).  Zeros on the exact path.  Synchronises `stream`. */
mop_status mop_route_stats(mop_ctx* ctx, int64_t* tokens_reevaluated, int64_t* chains, int64_t* beyond_half_bound,
                           void* stream);

/* Count and prefix-sum permutation of assignments a = t*k + j into expert-contiguous rows
 * (the buffer of N k rows of width H in Eq. 4).
 *   counts[e]   = number of assignments to expert e;   offsets = exclusive scan, offsets[E] = T*k
 *   perm_row[a] = offsets[idx[a]] + (number of a' < a with the same expert)     (stable)
 *   row_src     = inverse of perm_row;   Xp[p,:] = x[row_src[p] / k, :]
 * x [T,d] bf16; topk_idx [T,k]; counts [E]; offsets [E+1]; perm_row, row_src [T*k] i32 out;
 * Xp [T*k,d] bf16 out, or NULL: only the tables are built (x is then not read), for
 * mop_moe_expert_ffn_fwd_gather.  Indices outside [0,E) are a caller error (rows are dropped). */
mop_status mop_moe_permute(mop_ctx* ctx, const void* x, const int32_t* topk_idx, int32_t* counts, int32_t* offsets,
                           int32_t* perm_row, int32_t* row_src, void* Xp, void* stream);

/* Grouped SwiGLU expert feed-forward over the permuted rows (Section 2.1 "expert networks";
 * H is the N_r I term of Eq. 4).  For the rows p of expert e (offsets[e] <= p < offsets[e+1]):
 *   G = Xp W_gate[e], U = Xp W_up[e] (fp32 accumulation);  H = bf16(silu(G) * U)
 *   Yp[p,:] = bf16( gate(p) * (H[p,:] W_down[e]) ),  gate(p) = topk_gate[row_src[p]]
 * Xp [T*k,d] bf16; offsets [E+1]; row_src [T*k]; topk_gate [T,k] f32;
 * W_gate, W_up [E,d,f] bf16; W_down [E,f,d] bf16;
 * G_save, U_save [T*k,f] bf16 out, both NULL (forward only) or both set (kept for backward);
 * H [T*k,f] bf16 out (required); Yp [T*k,d] bf16 out. */
mop_status mop_moe_expert_ffn_fwd(mop_ctx* ctx, const void* Xp, const int32_t* offsets, const int32_t* row_src,
                                  const float* topk_gate, const void* W_gate, const void* W_up, const void* W_down,
                                  void* G_save, void* U_save, void* H, void* Yp, void* stream);

/* The same forward without the expert-contiguous copy of the inputs: the up-projection fetches
 * row p of expert e straight from x[row_src[p] / k, :] while it stages its operand tiles, so Xp
 * is never written or read (the N k H term of Eq. 4 drops out of the activation peak; the
 * single-GPU counterpart of keeping only a fraction of the routed inputs resident, Section 3.3).
 * Results are bit-identical to mop_moe_permute + mop_moe_expert_ffn_fwd.  No stash is written:
 * this is the inference form.  Needs the tensor-core path (MOP_ERR_UNSUPPORTED otherwise).
 * It trades time for memory: 4-row gather copies keep the TMA unit busier than 128-row boxes, and
 * the up-projection takes about 2.4 times as long as in the permuting form.
 * x [T,d] bf16; the other arguments as above. */
mop_status mop_moe_expert_ffn_fwd_gather(mop_ctx* ctx, const void* x, const int32_t* offsets,
                                         const int32_t* row_src, const float* topk_gate, const void* W_gate,
                                         const void* W_up, const void* W_down, void* H, void* Yp, void* stream);

/* Unpermute-combine, the last step of the MoE block of Section 2.1 (a token's output is the gate-weighted
 * sum of its k experts' outputs): Y[t,:] = bf16( sum_j Yp[perm_row[t*k+j], :] ), fp32 sum, j ascending.
 * (The gate was applied by mop_moe_expert_ffn_fwd.)  Also used for dX from dXp.
 * Yp [T*k,d] bf16; perm_row [T*k]; Y [T,d] bf16 out. */
mop_status mop_moe_combine(mop_ctx* ctx, const void* Yp, const int32_t* perm_row, void* Y, void* stream);

/* Backward of expert_ffn_fwd followed by combine (the paper counts forward and backward compute of every
 * block, Section 1, and its expert path supports backward gradient propagation, Section 3.3; the formulas
 * below are the derivative of the forward above), with topk_idx and topk_gate as inputs of the
 * function (the router's own backward is mop_moe_route_bwd).  With p <-> (t,j,e):
 *   dgate[t,j] = < dY[t,:] W_down[e]^T , H[p,:] >
 *   dH = gate * dY[t,:] W_down[e]^T;  dG = dH * U * s(G) (1 + G (1 - s(G)));  dU = dH * silu(G)
 *   dX[t,:]    = sum_j ( dG[p_j,:] W_gate[e_j]^T + dU[p_j,:] W_up[e_j]^T )
 *   dW_gate[e] = Xp_e^T dG_e;  dW_up[e] = Xp_e^T dU_e;  dW_down[e] = (gate * H_e)^T dY_e
 * dY [T,d] bf16; Xp, G_save, U_save, H, offsets, perm_row, row_src, topk_gate, W_* as above;
 * dX [T,d] bf16 out; dW_gate, dW_up [E,d,f] f32 out; dW_down [E,f,d] f32 out;
 * dgate [T,k] f32 out.  Needs a context created with with_backward >= 1.  Inputs must be finite.
 * Activation checkpointing (Section 3.1 lists it among the ways to cut transient activation memory):
 * with G_save, U_save and H all NULL (context created with with_backward = 2) the forward may have
 * run without the stash and the up-projection is recomputed here from Xp, bit for bit. */
mop_status mop_moe_expert_ffn_bwd(mop_ctx* ctx, const void* dY, const void* Xp, const void* G_save,
                                  const void* U_save, const void* H, const int32_t* offsets, const int32_t* perm_row,
                                  const int32_t* row_src, const float* topk_gate, const void* W_gate,
                                  const void* W_up, const void* W_down, void* dX, float* dW_gate, float* dW_up,
                                  float* dW_down, float* dgate, void* stream);

/* Expert-chunked layer: the memory-lean form of Section 3.3, where only a fraction of the routed buffers is
 * resident at any instant (the O(N k H + N_r I) activation term of Eq. 4 shrinks to one chunk of it).  The
 * experts are cut into n_chunks groups of about T k / n_chunks rows each (a group ends at an expert boundary, so
 * it holds at most one expert's rows more than its share); per group the rows are gathered from x, run through
 * the expert feed-forward, and added to an fp32 accumulator of Y in group order (fixed order, no atomics:
 * reproducible), which is rounded to bf16 once.  Xp, H and Yp therefore exist for one group at a time, in the
 * caller's `workspace` of mop_moe_chunked_workspace_bytes(shape, n_chunks, with_backward) bytes (256-byte
 * aligned).  The weights are read once, as in the unchunked layer.  The sum over a token's experts runs in
 * expert order here and in score order in mop_moe_combine: Y agrees to fp32 summation order, not bit for bit.
 * The backward keeps nothing of the forward: per group it gathers x and dY again, recomputes the up-projection,
 * runs the data and weight gradients of the group (each expert's dW is written once), and accumulates dX the
 * same way; experts without rows get zero gradients (or keep theirs when dw_accumulate is set).
 * Needs the tensor-core path (MOP_ERR_UNSUPPORTED otherwise); 1 <= n_chunks <= 64.
 * fwd: x, W_r, bias, W_* in; topk_idx, topk_gate, counts, offsets, perm_row, row_src, Y out (as in mop_moe_route,
 * mop_moe_permute, mop_moe_combine).  bwd: x, dY, topk_gate, offsets, perm_row, row_src, W_* in; dX, dW_*, dgate out
 * (as in mop_moe_expert_ffn_bwd); every intermediate lives in `workspace`, so any context of the shape will do. */
size_t mop_moe_chunked_workspace_bytes(const mop_moe_shape* shape, int32_t n_chunks, int32_t with_backward);
mop_status mop_moe_layer_fwd_chunked(mop_ctx* ctx, int32_t n_chunks, const void* x, const float* W_r, const float* bias,
                                     const void* W_gate, const void* W_up, const void* W_down, int32_t* topk_idx,
                                     float* topk_gate, int32_t* counts, int32_t* offsets, int32_t* perm_row,
                                     int32_t* row_src, void* Y, void* workspace, void* stream);
mop_status mop_moe_layer_bwd_chunked(mop_ctx* ctx, int32_t n_chunks, const void* x, const void* dY,
                                     const float* topk_gate, const int32_t* offsets, const int32_t* perm_row,
                                     const int32_t* row_src, const void* W_gate, const void* W_up, const void* W_down,
                                     void* dX, float* dW_gate, float* dW_up, float* dW_down, float* dgate,
                                     void* workspace, void* stream);

/* Router backward with the selection held fixed (Section 2.1's router, differentiated through the
 * gate renormalisation and the score function; the step on either side of the expert path).
 *   softmax:  dz_j = g_j (dgate_j - sum_l g_l dgate_l)
 *   sigmoid:  dz_j = (dgate_j - sum_l g_l dgate_l) / S * s_j (1 - s_j),  s = sigmoid(logit), S = sum_l s_l
 * over a token's k selected experts (dz = 0 elsewhere), then
 *   dW_r = x^T dz,   dX += dz W_r^T   (added to the expert-path gradient already in dX),
 *   dbias = column sums of dz for MOP_BIAS_PRE_LOGIT (a post-score bias only steers the selection).
 * logits [T,E] f32 as returned by mop_moe_route (logits_opt); topk_idx, topk_gate [T,k];
 * dgate [T,k] f32 (from mop_moe_expert_ffn_bwd); Xp [T*k,d] bf16, offsets [E+1], perm_row [T*k]
 * from mop_moe_permute; W_r [d,E] f32; bias as in mop_moe_route;
 * dW_r [d,E] f32 out; dbias_opt [E] f32 out or NULL; dX [T,d] bf16 in/out.
 * Needs a context created with with_backward = 1. */
mop_status mop_moe_route_bwd(mop_ctx* ctx, const float* logits, const float* bias, const int32_t* topk_idx,
                             const float* topk_gate, const float* dgate, const void* Xp, const int32_t* offsets,
                             const int32_t* perm_row, const float* W_r, float* dW_r, float* dbias_opt, void* dX,
                             void* stream);

/* Whole forward with HOST buffers (pageable or pinned): copies x in, runs route, permute,
 * expert_ffn_fwd and combine on `stream`, copies Y, topk_idx and topk_gate back, and
 * synchronises.  Weights stay on the device (they are parameters, not step inputs).
 * Scratch activations come from the context (created with this shape).
 * x_host [T,d] bf16; Y_host [T,d] bf16 out; idx_host [T,k] i32 out or NULL;
 * gate_host [T,k] f32 out or NULL. */
mop_status mop_moe_forward_host(mop_ctx* ctx, const void* x_host, const float* W_r, const float* bias,
                                const void* W_gate, const void* W_up, const void* W_down, void* Y_host,
                                int32_t* idx_host, float* gate_host, void* stream);

/* Pipelined forms of the two host-buffer entry points (the paper has no counterpart: it never
 * leaves the device).  A call enqueues one step and returns without waiting: its inputs are copied
 * on a copy stream while the previous step computes on `stream`, and its results are copied out on
 * an output stream while the next step computes.  The context double-buffers what the copies
 * touch (host_io = 2).  Host buffers must be pinned for the copies to overlap, must stay valid and
 * untouched until mop_host_drain returns, and output buffers of the last TWO calls must be
 * distinct only if the caller reads them before draining.  mop_host_drain makes `stream` wait for
 * every outstanding copy and synchronises it (call it before mop_destroy too); errors of the kernels
 * surface through mop_poll.
 * Arguments as in the synchronous forms; results are bit-identical to them. */
mop_status mop_moe_forward_host_async(mop_ctx* ctx, const void* x_host, const float* W_r, const float* bias,
                                      const void* W_gate, const void* W_up, const void* W_down, void* Y_host,
                                      int32_t* idx_host, float* gate_host, void* stream);
mop_status mop_moe_train_step_host_async(mop_ctx* ctx, const void* x_host, const void* dY_host, const float* W_r,
                                         const float* bias, const void* W_gate, const void* W_up,
                                         const void* W_down, void* Y_host, void* dX_host, float* dgate_host,
                                         float* dW_gate, float* dW_up, float* dW_down, void* stream);
mop_status mop_host_drain(mop_ctx* ctx, void* stream);

/* Whole training step of the layer with HOST activations: copies x and dY in, runs route,
 * permute, expert_ffn_fwd (keeping G, U), combine and expert_ffn_bwd on `stream`, copies Y, dX
 * and dgate back, and synchronises.  Weights and weight gradients stay on the device (they are
 * parameters and optimiser inputs, not step inputs).  Needs with_backward = 1 and host_io = 1.
 * x_host, dY_host [T,d] bf16; Y_host, dX_host [T,d] bf16 out; dgate_host [T,k] f32 out or NULL;
 * dW_gate, dW_up [E,d,f], dW_down [E,f,d] f32 DEVICE out. */
mop_status mop_moe_train_step_host(mop_ctx* ctx, const void* x_host, const void* dY_host, const float* W_r,
                                   const float* bias, const void* W_gate, const void* W_up, const void* W_down,
                                   void* Y_host, void* dX_host, float* dgate_host, float* dW_gate, float* dW_up,
                                   float* dW_down, void* stream);

/* Per-kernel timing.  mop_profile_enable(ctx, 1) creates a pool of CUDA events on first use and
 * from then on brackets every kernel launch of this context with an event pair on the launching
 * stream (up to 8192 launches between reads; later ones are not recorded).  mop_profile_read
 * synchronises `stream`, sums the recorded durations by kernel name into names / total_ms / calls
 * (arrays of max_names entries; names point to static strings), clears the records and returns
 * the number of distinct kernels, or -1 on error. */
mop_status mop_profile_enable(mop_ctx* ctx, int on);
int32_t mop_profile_read(mop_ctx* ctx, void* stream, int32_t max_names, const char** names, float* total_ms,
                         int32_t* calls);

/* Vocabulary projection with an online loss (Eq. 5 of the paper): with X [N,H] and W_voc [H,V],
 *   Y = X W_voc,   loss[n] = Y[n, t_n] - log sum_v exp(Y[n, v])      (the token's log-likelihood)
 * computed tile by tile on the tensor cores (bf16 operands, fp32 accumulation) with a running
 * maximum and sum per row, so that the N x V logits are never stored: the only intermediate is one
 * (max, sum) pair per row and 256-column block.  One-GPU counterpart of Section 3.4's projection.  H and V must be multiples of 64.
 * X [N,H] bf16; W_voc [H,V] bf16; targets [N] i32 in [0,V); loss [N] f32 out; lse_opt [N] f32 out or
 * NULL; workspace: device memory of mop_vocab_workspace_bytes(N, H, V) bytes, 256-byte aligned,
 * owned by the caller (nothing is allocated here).  `device` is the CUDA ordinal. */
size_t mop_vocab_workspace_bytes(int32_t N, int32_t H, int32_t V);
mop_status mop_vocab_loss_fwd(int device, int32_t N, int32_t H, int32_t V, const void* X, const void* W_voc,
                              const int32_t* targets, float* loss, float* lse_opt, void* workspace, void* stream);

/* Gradients of those log-likelihoods, again without the N x V matrix.  With p[n,v] =
 * exp(Y[n,v] - lse[n]) and an upstream weight dloss[n] per token (for a mean negative
 * log-likelihood: -1/N),
 *   dY[n,v] = dloss[n] ([v == t_n] - p[n,v]),   dX = dY W_voc^T,   dW_voc = X^T dY.
 * The vocabulary is walked in blocks of 8192 columns: the block's logits are recomputed on the
 * tensor cores, turned into dY in the epilogue (bf16, N x 8192, the only piece of the N x V matrix
 * that ever exists), multiplied into dW_voc[:, block] (written once) and accumulated into dX in
 * fp32 across the blocks (rounded to bf16 at the end).  Eq. 5 defines the loss; its derivative is
 * written out here.  lse is the output of mop_vocab_loss_fwd.
 * X [N,H] bf16; W_voc [H,V] bf16; targets [N] i32; lse, dloss [N] f32; dX [N,H] bf16 out;
 * dW_voc [H,V] f32 out (overwritten); workspace: mop_vocab_bwd_workspace_bytes(N, H, V) bytes of
 * device memory, 256-byte aligned, owned by the caller. */
size_t mop_vocab_bwd_workspace_bytes(int32_t N, int32_t H, int32_t V);

/* The two vocabulary calls have no context, so their kernels record an exhausted device-side wait in the
 * first word of the caller's workspace.  mop_vocab_poll synchronises `stream`, returns MOP_ERR_TIMEOUT if
 * the last call that used `workspace` recorded one (its outputs are then not valid) and clears the word.
 * Check it after a call whose results matter, as mop_poll is checked for a context. */
mop_status mop_vocab_poll(int device, void* workspace, void* stream);
/* Self-test of that path, as mop_selftest_wait_timeout: one thread waits `limit_cycles` on a barrier that
 * nothing completes and records the code in `workspace` (at least 256 bytes); nothing faults or traps. */
mop_status mop_vocab_selftest_wait_timeout(int device, void* workspace, int64_t limit_cycles, void* stream);
mop_status mop_vocab_loss_bwd(int device, int32_t N, int32_t H, int32_t V, const void* X, const void* W_voc,
                              const int32_t* targets, const float* lse, const float* dloss, void* dX,
                              float* dW_voc, void* workspace, void* stream);

/* The same permutation as mop_moe_permute for callers that may not allocate device memory (the
 * paper has no counterpart; this is a property of the library, not of the method).  A process
 * that gave all of HBM to its own arena, or a loop that cannot take the device-wide
 * synchronisation of an allocation, cannot create a context (mop_create calls cudaMalloc).  This
 * entry point needs none: its only scratch, the per-segment expert histogram, is a 1 MiB array
 * compiled into the library, resident on every GPU that loads it until the process exits.
 *   - Limit: ceil(T*k / 512) * E <= 262144, otherwise MOP_ERR_SHAPE and nothing is launched
 *     (for example T*k = 131072 with E up to 1024).  Also E <= 1024, k <= 32, d % 8 == 0.
 *   - It calls no cudaMalloc, cudaFree or other allocating routine.  The first call on a device
 *     looks up the array's device address (cudaGetSymbolAddress) and the SM count; make that
 *     first call outside any stream capture.
 *   - Every call on a device uses the same array and leaves its last contents there.  Nothing has
 *     to be cleared between calls (each call overwrites every entry it reads), but two calls
 *     that overlap on the GPU, on different streams or from different threads, race on it:
 *     serialise them.
 * Arguments as in mop_moe_permute, with the shape passed directly and `device` the CUDA ordinal. */
mop_status mop_moe_permute_static(int device, int32_t T, int32_t d, int32_t E, int32_t k, const void* x,
                                  const int32_t* topk_idx, int32_t* counts, int32_t* offsets, int32_t* perm_row,
                                  int32_t* row_src, void* Xp, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MOP_MOE_H_ */
