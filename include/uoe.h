/*
 * uoe.h -- C ABI of the Union-of-Experts routed hot path for NVIDIA B200 (sm_100a).
 *
 * The library evaluates one Union-of-Experts block the way the paper states the problem
 * (Section III): a transformer MLP (or the attention projections) is split column-wise /
 * row-wise into n equivalent experts (Eq. 1-7, Eq. 8-11); every sample goes to its top-k of n
 * experts (Eq. 21-23), every chosen expert takes at most c of the sample's m patches (Eq. 12-17),
 * and the expert outputs are added back at the selected positions (Eq. 20, 26, 36, 40).
 *
 * Conventions for every entry point
 *   - Pointers marked "device" are CUDA device pointers on the current device; `prob` is a host
 *     pointer.  All arrays are dense, row-major, and 16-byte aligned.
 *   - The caller owns every buffer, including the workspace `ws` (size from
 *     uoe_workspace_bytes).  The library never allocates or frees device memory and never
 *     synchronises, except uoe_read_device_status.  All work is enqueued on `cuda_stream`
 *     (a cudaStream_t passed as void*; NULL = the legacy default stream).
 *   - Outputs are overwritten, not accumulated into.
 *   - Errors are return codes.  Arguments are validated on the host before anything is launched.
 *     A device-side anomaly (a bounded wait that ran out, an index out of range) is recorded in
 *     the first word of the workspace and reported by uoe_read_device_status; kernels never trap.
 *     That word is sticky: it keeps the first anomaly recorded since it was last cleared, and no
 *     call clears it on its own (a clear on the stream would sit between the kernels of
 *     consecutive calls and stop them from overlapping).  A new workspace is prepared once with
 *     uoe_workspace_init; uoe_read_device_status clears the word after reporting an anomaly.
 *   - Devices and threads.  A process may use the library on several devices; kernel attributes and cached
 *     device properties are set up per device by the first call that needs them there.  That first call per
 *     device (of each entry point, uoe_route_static included) is not thread-safe; afterwards calls from several
 *     threads are safe as long as they use distinct workspaces.  uoe_profile_* is never thread-safe.
 *   - Element type: `dtype` selects float32 or bfloat16 storage for x, weights and y.  Products are
 *     accumulated in float32.  Routing probabilities and gates are always float32.
 *
 * Routed buffers.  Rows routed to expert i form one contiguous region that starts at row
 * expert_offsets[i]; inside it the samples that chose i appear in ascending order, each with
 * exactly l_a = c*l_p rows (its selected patches in ascending order; an unused slot, patch index
 * -1, is l_p zero rows).  Every region is padded to a multiple of UOE_ROW_ALIGN rows, so
 * expert_offsets[n] <= uoe_max_routed_rows(prob).
 */
#ifndef UOE_H_
#define UOE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define UOE_ROW_ALIGN 128

typedef enum {
    UOE_OK = 0,
    UOE_ERR_INVALID_ARG = 1,   /* null pointer, bad shape, misaligned buffer */
    UOE_ERR_UNSUPPORTED = 2,   /* valid problem outside what the kernels cover */
    UOE_ERR_WORKSPACE = 3,     /* ws_bytes smaller than uoe_workspace_bytes */
    UOE_ERR_CUDA = 4,          /* a CUDA runtime / driver call failed */
    UOE_ERR_TIMEOUT = 5,       /* device status: a bounded wait inside a kernel ran out */
    UOE_ERR_DEVICE_INDEX = 6,  /* device status: a routing index was out of range */
    UOE_ERR_STATIC_SCRATCH = 7 /* uoe_route_static: the problem needs more scratch than the built-in array holds */
} uoe_status;

typedef enum { UOE_F32 = 0, UOE_BF16 = 1 } uoe_dtype;

typedef enum {
    UOE_ACT_GELU_ERF = 0,
    UOE_ACT_GELU_TANH = 1,
    UOE_ACT_SILU = 2,          /* the paper's choice for UoME (below Eq. 39) */
    UOE_ACT_IDENTITY = 3
} uoe_act;

enum {
    UOE_FLAG_RESIDUAL = 1,     /* y = x + sum(...) (the selective residual of Eq. 20); else y = sum(...) */
    UOE_FLAG_GATE = 2,         /* combine weight = P_samp[b,i] * P_patch[b,i,j]; else 1 (Eq. 20 literal) */
    UOE_FLAG_CAUSAL = 4,       /* SMHA: shared lower-triangular mask over the gathered tokens (Fig. 4) */
    UOE_FLAG_DYNAMIC_C = 8,    /* uoe_route: two-stage routing (Eq. 15-16): every chosen expert of a sample takes
                                  min(c, c_b) patches, c_b = the largest number of patches any expert receives when
                                  each patch goes to its k best experts; the remaining slots are unused (-1) */
    UOE_FLAG_GENERAL_PATH = 16 /* take the general routed path even for the two single-mode cases below (same results;
                                  for verification and for measuring what the special cases save) */
};

/*
 * The two selection modes the paper uses on their own (end of Section III-B) are recognised from the problem and
 * take shorter paths with the same results:
 *   k == n  pure data selection (Eq. 12-20): every sample uses all n experts.  No expert ranking; every expert's
 *           region holds exactly B pairs, so expert_offsets and each pair's rows follow from (b, i) alone and no
 *           step of the router waits for the other samples.
 *   c >= number of patches that hold a real token, without UOE_FLAG_DYNAMIC_C  pure expert selection (Eq. 21-26): a
 *           chosen expert takes the whole sample.  No patch ranking; slot u of a pair is patch u, so neither the
 *           router nor the consumers inside uoe_block_forward build or read a patch plan or an inverse map: the
 *           combine finds the at most k rows of a token from the pair's first row and the token's position.
 */

typedef enum { UOE_OP_ROUTE = 0, UOE_OP_MLP_FWD = 1, UOE_OP_MLP_BWD = 2, UOE_OP_SMHA_FWD = 3, UOE_OP_SMHA_BWD = 4,
               UOE_OP_BALANCE_BWD = 5 } uoe_op;

/* One Union-of-Experts block.  L must equal m * l_p; rows t >= L_valid of every sample are padding
 * (they take no part in routing means, are masked as attention keys (Eq. 41), and y = x there).
 * Padding rows of x and dy must hold finite values (zeros by convention): whole patches travel through the
 * tensor-core kernels, where a padding row is neutralised by a zero weight or a zero probability, and
 * 0 * Inf or 0 * NaN would spread into the real rows of the same expert (weight gradients, attention outputs).
 * A buffer padded from uninitialised memory must be zero-filled first. */
typedef struct {
    int32_t B;        /* samples */
    int32_t L;        /* tokens per sample, padded: L = m * l_p */
    int32_t L_valid;  /* real tokens per sample, 1 <= L_valid <= L */
    int32_t d;        /* model width */
    int32_t n;        /* experts */
    int32_t k;        /* experts per sample, 1 <= k <= n */
    int32_t m;        /* patches per sample */
    int32_t c;        /* patches per expert, 1 <= c <= m */
    int32_t d_e;      /* UoME: hidden width of one expert (d_ff / n); 0 if unused */
    int32_t H;        /* SMHA: attention heads, H % n == 0; 0 if unused */
    int32_t d_h;      /* SMHA: width of one head */
    int32_t dtype;    /* uoe_dtype */
    int32_t act;      /* uoe_act */
    uint32_t flags;   /* UOE_FLAG_* */
    int32_t d_rope;   /* SMHA: rotary channels per head (Eq. 32), even, 0 <= d_rope <= d_h; 0 = no RoPE.  The last
                         d_rope channels of every head of q and k are rotated in pairs (2i, 2i+1) by the angle
                         t * 10000^(-2i/d_rope), t = the token's position in its sample */
} uoe_problem;

/* Upper bound on expert_offsets[n]: B*k*c*l_p rows plus per-expert padding.  Buffers indexed by routed
 * row (saved_h, lse) must hold this many rows.  Returns 0 on an invalid problem. */
int64_t uoe_max_routed_rows(const uoe_problem* prob);

/* Bytes of device workspace that `op` (a uoe_op) needs for this problem (0 on an invalid problem). */
size_t uoe_workspace_bytes(const uoe_problem* prob, int op);

/*
 * Router scoring and fused selection (Eq. 12-17 and 21-23, combined as in Fig. 3).
 *   patch score   g'[b,i,j] = mean over the real tokens t of patch j of  x[b,t,:] . W_r[:,i]   (Eq. 13)
 *   p_patch[b,:,j] = softmax over the n experts of g'[b,:,j]                                     (Eq. 14)
 *   p_samp[b,:]    = softmax over experts of (mean over real tokens of x[b]) . W_r               (Eq. 21)
 *   expert_idx[b,:] = the k experts with the largest p_samp, ascending (ties: lower index)       (Eq. 22)
 *   patch_idx[b,s,:] = for the s-th chosen expert i, the min(c, #patches with a real token) patches
 *                      with the largest p_patch[b,i,:], ascending; unused slots are -1            (Eq. 17)
 *                      (with UOE_FLAG_DYNAMIC_C also at most the sample's own capacity, Eq. 15-16)
 *   gate[b,s,u]     = p_samp[b,i] * p_patch[b,i,patch] with UOE_FLAG_GATE, else 1; 0 in unused slots
 *   expert_offsets  = row offsets of the per-expert regions (see "Routed buffers")               (Eq. 23)
 * All arguments except prob are device pointers.  x [B,L,d] and W_r [d,n] have prob->dtype;
 * the outputs are int32 / float32 with the shapes given.  Scores accumulate in float32.
 */
uoe_status uoe_route(const uoe_problem* prob, const void* x, const void* W_r,
                     int32_t* expert_idx /* [B,k] */, int32_t* patch_idx /* [B,k,c] */,
                     float* gate /* [B,k,c] */, float* p_samp /* [B,n] */, float* p_patch /* [B,n,m] */,
                     int32_t* expert_offsets /* [n+1] */, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Load statistics of the patch gate (device pointers; p_patch [B,n,m] as written by uoe_route):
 *   expert_count[b,i] = number of real patches of sample b that have expert i among their k best experts
 *                       (Eq. 15; ties: lower index)                                       int32 [B,n], or NULL
 *   c_dyn[b]          = max_i expert_count[b,i], the dynamic capacity of Eq. 16            int32 [B], or NULL
 *   lb_loss[b]        = alpha * sum_i f_i P_i, the sequence-wise load-balancing loss of Eq. 42-44 taken over the
 *                       sample's real patches: f_i = n/(k l) expert_count[b,i], P_i = mean gate of expert i
 *                                                                                           float32 [B], or NULL
 * Needs no workspace.
 */
uoe_status uoe_route_balance(const uoe_problem* prob, const float* p_patch, float alpha, float* lb_loss,
                             int32_t* expert_count, int32_t* c_dyn, void* cuda_stream);

/*
 * Gradient of sum_b dloss[b] * lb_loss[b] (the loss of uoe_route_balance, Eq. 42-44) with respect to x and W_r.
 * f_i counts top-k memberships and is piecewise constant, so the gradient flows through P_i only: through the patch
 * softmax (Eq. 14) and the mean-pooled linear router (Eq. 13).  The paper gives no backward text.
 *   dx [B,L,d] in prob->dtype and dW_r [d,n] float32 are overwritten (add them to the layer's own gradients);
 *   dloss [B] float32; p_patch [B,n,m] as written by uoe_route for the same x and W_r.  bfloat16 only.
 * Workspace: uoe_workspace_bytes(prob, UOE_OP_BALANCE_BWD).  All pointers except prob are device pointers.
 */
uoe_status uoe_route_balance_backward(const uoe_problem* prob, const void* x, const void* W_r, const float* p_patch,
                                      float alpha, const float* dloss, void* dx, float* dW_r,
                                      void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * UoME forward (Eq. 37-40 with the index-select of Eq. 18 and the index-add of Eq. 20):
 *   y[b,t,:] = x[b,t,:] + sum over (expert i, patch j) that selected token t of
 *              gate[b,i,j] * ( phi( x[b,t,:] W1[i] + b1[i] ) W2[i] + b2[i] )
 * W1 [n,d,d_e] holds the column slices of the first layer, W2 [n,d_e,d] the row slices of the
 * second (Eq. 1-7); no activation follows the second layer.  b1 [n,d_e], b2 [n,d] (in prob->dtype) may be NULL;
 * they are the in-place bias of the batched product (Section III-D.2): b1[i] enters before phi, b2[i] is added to
 * expert i's output before the combine weight (the backward entry point does not return their gradients).  The routing arrays are the outputs of uoe_route or any
 * arrays of the same form supplied by the caller (sorted, in range, offsets consistent with
 * expert_idx).  With UOE_FLAG_GATE the combine weight is gate[b,s,u], otherwise 1.  saved_h, if
 * not NULL, receives the pre-activation x W1[i] of every routed row,
 * [uoe_max_routed_rows, d_e] in prob->dtype, for uoe_mlp_backward.  All pointers except prob are
 * device pointers.
 */
uoe_status uoe_mlp_forward(const uoe_problem* prob, const void* x, const void* W1, const void* W2,
                           const void* b1, const void* b2,
                           const int32_t* expert_idx, const int32_t* patch_idx, const float* gate,
                           const int32_t* expert_offsets, void* y /* [B,L,d] */, void* saved_h,
                           void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * UoME backward: gradients of sum(y * dy) with the selection (expert_idx, patch_idx) held constant.
 * The paper gives no backward text; this is the derivative of Eq. 38-40 and, with UOE_FLAG_GATE, of
 * the gate through both softmaxes (Eq. 14, 21) into W_r and x.
 *   dx [B,L,d] in prob->dtype; dW1 [n,d,d_e], dW2 [n,d_e,d], dW_r [d,n] in float32, overwritten.
 * saved_h is the array written by uoe_mlp_forward for the same inputs.  Biases are not supported
 * here.  All pointers except prob are device pointers.
 */
uoe_status uoe_mlp_backward(const uoe_problem* prob, const void* x, const void* W1, const void* W2,
                            const void* W_r, const int32_t* expert_idx, const int32_t* patch_idx,
                            const float* gate, const int32_t* expert_offsets,
                            const float* p_samp, const float* p_patch, const void* saved_h,
                            const void* dy /* [B,L,d] */, void* dx /* [B,L,d] */,
                            float* dW1, float* dW2, float* dW_r,
                            void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * SMHA forward (Eq. 27-30, 32-36; masks Eq. 41 and Fig. 4; RoPE of Eq. 32 when prob->d_rope > 0).
 * Attention expert i owns the column slices Wq/Wk/Wv[i] [d, d_g] and the row slice Wo[i] [d_g, d]
 * with d_g = (H/n)*d_h (Eq. 8-11).  For each sample b and chosen expert i the l_a gathered tokens
 * attend to each other per head: softmax(q k^T / sqrt(d_h) + mask) v, where pad tokens are masked as
 * keys and, with UOE_FLAG_CAUSAL, key position > query position in gathered order is masked.  The
 * projected result is added back as in uoe_mlp_forward:  y = x + sum gate * (o Wo[i]).
 * lse, if not NULL, receives the log-sum-exp of every (routed row, head of the expert):
 * [uoe_max_routed_rows, H/n] float32.  All pointers except prob are device pointers.
 */
uoe_status uoe_smha_forward(const uoe_problem* prob, const void* x, const void* Wq, const void* Wk,
                            const void* Wv, const void* Wo,
                            const int32_t* expert_idx, const int32_t* patch_idx, const float* gate,
                            const int32_t* expert_offsets, void* y /* [B,L,d] */, float* lse,
                            void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * SMHA backward: gradients of sum(y * dy) for y = uoe_smha_forward(x, ...) with the selection (expert_idx,
 * patch_idx) held constant.  The paper gives no backward text; this is the derivative of Eq. 28-30 and 33-36
 * (masked softmax attention per chosen expert and head, projections, weighted index-add) and, with
 * UOE_FLAG_GATE, of the gate through both softmaxes (Eq. 14, 21) into W_r and x.  Nothing saved by the
 * forward is needed: q, k, v, the attention output and its log-sum-exp are recomputed inside.
 *   dx [B,L,d] in prob->dtype; dWq, dWk, dWv [n,d,d_g], dWo [n,d_g,d], dW_r [d,n] in float32, overwritten.
 * bfloat16 with 64-wide heads and d % 128 == 0 only (UOE_ERR_UNSUPPORTED otherwise).  All pointers except
 * prob are device pointers.
 */
uoe_status uoe_smha_backward(const uoe_problem* prob, const void* x, const void* Wq, const void* Wk,
                             const void* Wv, const void* Wo, const void* W_r,
                             const int32_t* expert_idx, const int32_t* patch_idx, const float* gate,
                             const int32_t* expert_offsets, const float* p_samp, const float* p_patch,
                             const void* dy /* [B,L,d] */, void* dx /* [B,L,d] */,
                             float* dWq, float* dWk, float* dWv, float* dWo, float* dW_r,
                             void* ws, size_t ws_bytes, void* cuda_stream);

/* Device arrays written by a router (shapes as for uoe_route).  A set is complete or absent as a whole. */
typedef struct {
    int32_t* expert_idx;      /* [B,k] */
    int32_t* patch_idx;       /* [B,k,c] */
    float* gate;              /* [B,k,c] */
    float* p_samp;            /* [B,n] */
    float* p_patch;           /* [B,n,m] */
    int32_t* expert_offsets;  /* [n+1] */
} uoe_routing;

/*
 * One UoE transformer block in one call (Section III-C, Fig. 2): selective attention over attention experts
 * followed by the MLP experts, each half with its own router,
 *     u = uoe_smha_forward(att, x, ...) with the routing of uoe_route(att, x, Wr_att),
 *     y = uoe_mlp_forward (mlp, u, ...) with the routing of uoe_route(mlp, u, Wr_mlp),
 * and the same results as that sequence of calls (Eq. 27-36, then Eq. 37-40; routing Eq. 12-17, 21-23).  Either
 * half may be left out by passing NULL for its problem (then its weights are ignored and y is the other half's
 * output; with only the MLP half, x is its input).  One workspace of uoe_block_workspace_bytes(att, mlp) bytes,
 * prepared once with uoe_workspace_init, serves the whole call: the routers share their scratch, write their
 * routing plans themselves, and the routed buffers of the two halves share memory, so a block costs fewer
 * launches and less memory than the four separate calls.
 *   att, mlp   host pointers; both describe the same B, L, L_valid, d and dtype (n, k, m, c may differ).
 *   x [B,L,d]; Wr_att, Wr_mlp [d,n]; Wq, Wk, Wv [n,d,d_g]; Wo [n,d_g,d]; W1 [n,d,d_e]; W2 [n,d_e,d]   device, inputs.
 *   r_att, r_mlp   host pointers to sets of device arrays that receive each router's outputs (for a later
 *              backward call), or NULL to keep them inside the workspace.
 *   u [B,L,d]  device, output of the attention half; required when both halves are present; distinct from x and y.
 *   y [B,L,d]  device, output of the block.
 *   saved_h    as for uoe_mlp_forward, or NULL.     lse   as for uoe_smha_forward, or NULL.
 * Biases are not supported here.  Errors as for the separate calls; nothing is launched when an argument is rejected.
 */
size_t uoe_block_workspace_bytes(const uoe_problem* att, const uoe_problem* mlp);
uoe_status uoe_block_forward(const uoe_problem* att, const uoe_problem* mlp, const void* x,
                             const void* Wr_att, const void* Wq, const void* Wk, const void* Wv, const void* Wo,
                             const void* Wr_mlp, const void* W1, const void* W2,
                             const uoe_routing* r_att, const uoe_routing* r_mlp, void* u, void* y,
                             void* saved_h, float* lse, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * uoe_route without a workspace argument and without any allocation.  (The paper has no counterpart;
 * this exists for callers that cannot hand the library device memory of their own.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a region that must not
 * synchronise the device or touch the allocator (a latency-critical serving loop, a plugin hosted by
 * a framework that owns all device memory and offers no way to request scratch, start-up code that
 * runs before the host application's memory pool exists).  Such a caller can pass its inputs and
 * outputs but has nowhere to get the extra buffer that uoe_route needs for its partial scores and tickets.
 *
 * Here that buffer is a fixed array of UOE_ROUTE_STATIC_SCRATCH_BYTES compiled into the library's
 * device image, so every GPU on which the library is loaded holds that many bytes until the process
 * exits.  Results are identical to uoe_route.  Arguments are as for uoe_route, minus ws / ws_bytes.
 *
 *   - Limit: the problem must satisfy uoe_workspace_bytes(prob, UOE_OP_ROUTE) <=
 *     UOE_ROUTE_STATIC_SCRATCH_BYTES; otherwise nothing is launched and UOE_ERR_STATIC_SCRATCH is returned.
 *   - The first call on each device looks up the array's device address (a one-time set-up step, done
 *     with that device current).  Make that first call before starting any stream capture.
 *   - The function calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - All calls on a device share the one array.  It starts zeroed, and the kernels leave the counters that must
 *     start at zero (completion tickets, expert loads) at zero again when a call finishes, whatever shapes the
 *     calls have; the rest still holds what the previous call left and is overwritten before it is read.  Two calls
 *     whose kernels may overlap on the GPU (different streams, no ordering between them) race on the array and
 *     give wrong routing: order them, or use uoe_route with separate workspaces.
 *   - No device status word is kept for this variant (uoe_read_device_status does not apply).
 */
#define UOE_ROUTE_STATIC_SCRATCH_BYTES (2 << 20)
uoe_status uoe_route_static(const uoe_problem* prob, const void* x, const void* W_r,
                            int32_t* expert_idx /* [B,k] */, int32_t* patch_idx /* [B,k,c] */,
                            float* gate /* [B,k,c] */, float* p_samp /* [B,n] */, float* p_patch /* [B,n,m] */,
                            int32_t* expert_offsets /* [n+1] */, void* cuda_stream);

/* Text for a status code (static storage). */
const char* uoe_status_string(int status);

/* Prepares a new workspace (device pointer, at least 1024 bytes): enqueues on `cuda_stream` the zeroing of its
 * control block (the first 1 MiB, or all of a smaller workspace: the status word and the counters that the
 * kernels leave at zero again after every call).  Call it once per workspace, before the first call that
 * uses it. */
uoe_status uoe_workspace_init(void* ws, size_t ws_bytes, void* cuda_stream);

/* Synchronises `cuda_stream`, reads the status word of workspace `ws` and returns it: UOE_OK, or the first
 * anomaly a kernel recorded there since the word was last cleared.  A reported anomaly is cleared. */
uoe_status uoe_read_device_status(void* ws, void* cuda_stream);

/* Number of this library's kernel launches enqueued by this process so far (for benchmarks). */
int64_t uoe_launch_count(void);

/* Number of TMA tensor maps this process has encoded so far.  Encoded maps are kept in a table keyed by buffer
 * address and shape, so repeated calls on the same buffers encode nothing new (for benchmarks and tests). */
int64_t uoe_tensor_map_encodings(void);

/*
 * Per-kernel timing for benchmarks (instrumentation; the paper times whole passes with a profiler,
 * Section IV).  uoe_profile_enable(1) clears the record list and starts recording: from then on every
 * kernel the library launches is bracketed by two CUDA events on its stream.  uoe_profile_enable(0)
 * stops recording.  uoe_profile_get waits for record i to finish and returns its label (static
 * storage) and duration in milliseconds.  Not thread-safe; leave it off outside measurements.
 */
void uoe_profile_enable(int on);
int uoe_profile_count(void);
uoe_status uoe_profile_get(int i, const char** name, float* ms);

#ifdef __cplusplus
}
#endif
#endif /* UOE_H_ */
