/*
 * arl2.h -- C ABI of the ARL^2 hybrid attention layer for NVIDIA B200 (sm_100a).
 *
 * The layer is the attention core that an autoregressive video-diffusion model runs at
 * every denoising step of every block (paper Sec. 3.2-3.3, Algorithm 1):
 *
 *   O_intra = Softmax(RoPE(Q), RoPE(K), V)          over the block's L tokens   (Eq. 2)
 *   Q'      = L2Norm(RoPE(phi_q(Q)))                                            (Eq. 3)
 *   O_inter = Q' S                                   same pre-update S for all   (Eq. 5, 8)
 *   O       = O_intra + sigmoid(g) (.) O_inter       headwise gate               (Eq. 6-7)
 *   S      <- sigmoid(a) S + K'^T V'                 once per block, clean pass  (Eq. 4, Sec. 3.3)
 *
 * Conventions shared by every call
 *   - All `d_*` pointers are DEVICE pointers owned by the caller; the library never
 *     allocates or frees device memory and keeps only the pointers it is given
 *     (state, workspace, parameters) until arl2_destroy.
 *   - Tensors are contiguous.  Q, K, V, O: [B, L, H, D] (token-major).  State S:
 *     [B, H, D, D] fp32, row = key dimension, column = value dimension.  Combine-gate
 *     logits g: [B, L, H] fp32.  Decay logits a: [B, H] fp32.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls are
 *     asynchronous on it; ordering between calls is stream order.
 *   - Every function returns an arl2_status (0 = ok, negative = error).  Argument errors
 *     are found on the host before any launch and leave S untouched.  Nothing aborts,
 *     traps or throws.  arl2_last_error() gives a thread-local message for the last error.
 *   - A context is not thread-safe; distinct contexts are independent.
 */
#ifndef ARL2_H
#define ARL2_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct arl2_ctx arl2_ctx; /* opaque, host memory owned by the library */

typedef enum {
    ARL2_OK = 0,
    ARL2_ERR_INVALID_ARG = -1, /* NULL pointer, bad size, bad struct_size ...              */
    ARL2_ERR_UNSUPPORTED = -2, /* shape / dtype combination with no kernel                  */
    ARL2_ERR_CUDA = -3,        /* a CUDA runtime or driver call failed                      */
    ARL2_ERR_TIMEOUT = -4,     /* a bounded wait inside a kernel expired (device status)    */
    ARL2_ERR_WORKSPACE = -5    /* workspace too small or misaligned                         */
} arl2_status;

typedef enum {
    ARL2_BF16 = 0, /* bf16 inputs/outputs, tensor-core contractions, fp32 accumulation      */
    ARL2_FP32 = 1  /* fp32 inputs/outputs, fp32 FMA arithmetic end to end (the 1e-4 mode)   */
} arl2_dtype;

/* arl2_config.flags */
#define ARL2_FLAG_FORCE_SIMT 1u /* bf16 I/O through the plain-FMA kernels (debug / A-B checks) */
/* Granularity of the combine gate of arl2_denoise_step (Eq. 6-7 take one gate per token and head;
   the other two are the variants of the paper's gate ablation, offered for comparison):          */
#define ARL2_FLAG_GATE_SCALAR 4u      /* d_gate_logits is [B, L]: one gate per token, all heads     */
#define ARL2_FLAG_GATE_ELEMENTWISE 8u /* d_gate_logits is [B, L, H, D]: one gate per output channel */
#define ARL2_FLAG_TOKEN_GATES 2u /* reserve workspace for arl2_commit_tokens (3 fp32 copies of a
                                    [B, H, ceil(L/64)*64, D] tensor)                             */
/* arl2_commit_tokens: each token's prediction is made against the state after its own forget gate,
   S <- alpha_l S + beta_l K'_l^T (V'_l - K'_l (alpha_l S)) -- the Gated DeltaNet's form -- instead of Eq. 4
   as printed (prediction against the undecayed state).                                                   */
#define ARL2_FLAG_DELTA_DECAYED_PREDICTION 32u
/* Test hook for the time-out path: every bounded wait inside the tensor-core kernels gives up
   after `polls` polls of its barrier (0 .. 65534) instead of 2^24.  With 0 the first wait of a
   launch expires at once: the kernel records ARL2_ERR_TIMEOUT and the wait's site in the status
   block, every role leaves through the common exit (copies in flight are still awaited with the
   full bound, tensor memory is freed), the output is undefined, S is untouched by a denoise
   pass, and arl2_sync_status reports it.  Never set in production.                              */
#define ARL2_FLAG_DEBUG_WAIT_LIMIT_SHIFT 16
#define ARL2_FLAG_DEBUG_WAIT_LIMIT(polls) (((uint32_t)(polls) + 1u) << ARL2_FLAG_DEBUG_WAIT_LIMIT_SHIFT)

typedef struct {
    uint32_t struct_size; /* sizeof(arl2_config), for versioning                            */
    int32_t B;            /* independent streams (videos), >= 1                             */
    int32_t H;            /* heads, >= 1                                                    */
    int32_t L;            /* tokens per autoregressive block, >= 1, any value               */
    int32_t D;            /* head dimension: 64 or 128                                      */
    int32_t io_dtype;     /* arl2_dtype of Q, K, V, O and of the feature-map weights        */
    float softmax_scale;  /* 0 -> 1/sqrt(D) (Eq. 1)                                         */
    float l2_eps;         /* epsilon inside the root of L2Norm; 0 -> 1e-6                   */
    int32_t commit_rule;  /* 0 = gated linear S <- alpha S + K'^T V'; others reserved       */
    uint32_t flags;       /* ARL2_FLAG_*                                                    */
} arl2_config;

/*
 * Bytes of device scratch a context of this shape needs (256-byte aligned base).  It
 * holds a status word, the rotated copy of K made once per step, two tensor-core operand
 * copies of S (a commit writes the one that is not current) and one of each feature map, the
 * packed rotation table, the partial sums of the commit reduction (two sets: the delta rule
 * has two accumulators), the per-token decay weights, with bf16 I/O and D = 128 the partial rows
 * of attention work items cut into key ranges (about 39 MB: when the last wave of a step launch
 * would leave more than half of the SMs idle, its items are computed as 2 to 4 parts and a second
 * small launch merges them) and, with ARL2_FLAG_TOKEN_GATES, the chunk factors of
 * arl2_commit_tokens.  Returns 0 for an invalid configuration.
 */
size_t arl2_workspace_bytes(const arl2_config* cfg);

/*
 * Create a context (Algorithm 1: the state lives for one video per stream).
 *   d_state      [B, H, D, D] fp32, caller-owned; NOT cleared by this call -- call
 *                arl2_reset, or arl2_set_state to resume from a checkpoint.
 *   d_workspace  >= arl2_workspace_bytes(cfg) bytes, 256-byte aligned, caller-owned,
 *                private to this context until arl2_destroy.
 * Launches one small kernel on `stream` that clears the workspace header.
 */
int arl2_create(const arl2_config* cfg, void* d_state, void* d_workspace,
                size_t workspace_bytes, void* stream, arl2_ctx** out);

/*
 * Feature maps phi_q, phi_k, phi_v (Eq. 3: per-head grouped 1x1 maps, read here as
 * bias-free linear maps applied as row-vector times matrix) and the rotary tables.
 *   d_wphi_*   [H, D, D] indexed [head][in][out], io_dtype; NULL = identity map.
 *   d_rope_cos, d_rope_sin  [L, D/2] fp32: cos / sin of the angle of pair (2m, 2m+1) at
 *              token l; both NULL = no rotation.  The same tables serve Q and K and both
 *              branches.
 * The pointers are kept; the buffers must stay valid and unchanged until replaced or
 * the context is destroyed.  On the tensor-core path this call also launches a kernel
 * that writes operand copies of the maps into the workspace.
 */
int arl2_set_params(arl2_ctx* ctx, const void* d_wphi_q, const void* d_wphi_k,
                    const void* d_wphi_v, const float* d_rope_cos, const float* d_rope_sin,
                    void* stream);

/*
 * One denoising pass of the layer (Algorithm 1, inner loop; Eq. 2, 3, 5-8):
 *   d_out[b,i,h,:] = softmax_j(<RoPE(q_i), RoPE(k_j)> scale) v_j
 *                    + sigmoid(g[b,i,h]) * L2Norm(RoPE(q_i Wphi_q[h])) S[b,h]
 * READS the state, never writes it (clean-pass-only update, Sec. 3.3): S is bitwise
 * unchanged after any number of calls.  d_q, d_k, d_v, d_out: [B, L, H, D] io_dtype;
 * d_gate_logits: [B, L, H] fp32 (the projection x W_g of Eq. 6), or [B, L] / [B, L, H, D] when
 * the context was created with ARL2_FLAG_GATE_SCALAR / ARL2_FLAG_GATE_ELEMENTWISE.  d_out must
 * not alias an input.
 */
int arl2_denoise_step(arl2_ctx* ctx, const void* d_q, const void* d_k, const void* d_v,
                      const float* d_gate_logits, void* d_out, void* stream);

/*
 * Token-level state access, the comparison mode of the paper's "State access granularity" ablation
 * (Sec. 4.3; the layer itself uses frame-level access, Eq. 8).  Token i reads the state advanced by the
 * tokens of the block before it -- each token sees its own sequentially accumulated state -- the
 * gated-linear update being applied token by token on a private copy:
 *   S^(0) = S,  S^(i+1) = alpha_i S^(i) + K'_i^T V'_i,
 *   d_out[b,i,h,:] = softmax_j(<RoPE(q_i), RoPE(k_j)> scale) v_j + sigmoid(g[b,i,h]) Q'_i S^(i),
 * with K' = L2Norm(RoPE(k Wphi_k)), V' = v Wphi_v of the pass's own k, v and alpha_i =
 * sigmoid(d_alpha_logits[b,i,h]) (NULL: 1).  Token 0 reads S itself; a one-token block equals
 * arl2_denoise_step.  READS the state, never writes it.  Computed chunkwise (128 tokens per chunk: a
 * causal score matrix inside the chunk, the chunk-entry state in tensor memory across chunks) after the
 * ordinary attention kernel has written the softmax branch.  Forget gates that stay below about 0.5
 * for a whole chunk leave the fp32 range of the chunk factors.  Contexts with bf16 I/O, D = 128 and the
 * headwise gate only (ARL2_ERR_UNSUPPORTED otherwise).  Other arguments as arl2_denoise_step.
 */
int arl2_denoise_step_token_level(arl2_ctx* ctx, const void* d_q, const void* d_k, const void* d_v,
                                  const float* d_gate_logits, const float* d_alpha_logits, void* d_out,
                                  void* stream);

/*
 * The teacher's layer for comparison (Eq. 1): plain softmax attention of the current block's L
 * queries over a key/value cache of `cache_tokens` tokens (the blocks generated so far plus the
 * current one), all visible to every query:
 *   d_out[b,i,h,:] = softmax_j(<q_i, k_j> scale) v_j,   j = 0 .. cache_tokens-1.
 * d_q, d_out: [B, L, H, D]; d_k_cache, d_v_cache: [B, cache_tokens, H, D], io_dtype.  No rotation
 * is applied (a cache holds rotated keys; pass rotated queries), the feature maps, the gate and
 * the recurrent state play no part.  Its cost grows with cache_tokens where arl2_denoise_step's
 * does not: this entry point exists to measure that on the same kernels.  Contexts with bf16 I/O
 * and D = 128 only (ARL2_ERR_UNSUPPORTED otherwise).  Honours arl2_set_profile_events.
 */
int arl2_teacher_step(arl2_ctx* ctx, const void* d_q, const void* d_k_cache, const void* d_v_cache,
                      int32_t cache_tokens, void* d_out, void* stream);

/*
 * State commit, once per block, from the clean pass's K and V (Algorithm 1, clean-pass
 * branch; Eq. 4 in its gated-linear form):
 *   S[b,h] <- sigmoid(a[b,h]) S[b,h] + sum_l K'_l^T V'_l,
 *   K' = L2Norm(RoPE(k Wphi_k[h])),  V' = v Wphi_v[h].
 * The ONLY call that changes S besides reset / set_state.  The reduction over tokens
 * is split across thread blocks and summed in a fixed order: results are bitwise
 * reproducible.  d_k_clean, d_v_clean: [B, L, H, D] io_dtype; d_decay_logits: [B, H] fp32.
 */
int arl2_commit(arl2_ctx* ctx, const void* d_k_clean, const void* d_v_clean,
                const float* d_decay_logits, void* stream);

/*
 * The clean pass of a block in one call (Algorithm 1, clean-pass branch; Sec. 3.3 "Clean-pass
 * update"): the layer's output for the clean latent, read against the state as it stood BEFORE the
 * call (Eq. 8), and then the gated-linear commit of that same block,
 *   d_out  = arl2_denoise_step(q, k_clean, v_clean, gate_logits)  with the pre-update S,
 *   S     <- sigmoid(a) S + sum_l K'_l^T V'_l                       from the same k_clean, v_clean.
 * Equal to arl2_denoise_step followed by arl2_commit on the same tensors, but K_c is read and
 * rotated once: the kernel that forms the partial sums of the state update also writes RoPE(K_c)
 * for the softmax branch, the attention kernel runs next, and the kernel that adds the partial
 * sums into S runs last.  Arguments, layouts and error behaviour as in those two calls.
 */
int arl2_clean_pass(arl2_ctx* ctx, const void* d_q, const void* d_k_clean, const void* d_v_clean,
                    const float* d_gate_logits, const float* d_decay_logits, void* d_out, void* stream);

/*
 * State commit with the delta rule of Eq. 4 as printed, applied once per block to the clean
 * pass's tokens (all of them against the state as it stood before the call):
 *   S[b,h] <- sigmoid(a[b,h]) S[b,h] + sum_l beta_l K'_l^T (V'_l - K'_l S_old[b,h]),
 *   beta_l = sigmoid(d_beta_logits[b,l,h]),  K', V' as in arl2_commit.
 * The result does not depend on the order of the tokens.  d_beta_logits: [B, L, H] fp32, or
 * NULL for beta = 1.  Other arguments, reproducibility and error behaviour as arl2_commit.  With
 * bf16 I/O and D = 128 the prediction K' S_old is a tensor-core contraction against the bf16
 * operand copy of S_old.  Any context may mix calls of arl2_commit and arl2_commit_delta.
 */
int arl2_commit_delta(arl2_ctx* ctx, const void* d_k_clean, const void* d_v_clean,
                      const float* d_decay_logits, const float* d_beta_logits, void* stream);

/*
 * The gated-linear commit with one forget gate per token (the gate granularity the paper states;
 * Eq. 4 without its correction term, token by token): for l = 0..L-1
 *   S[b,h] <- alpha_l S[b,h] + K'_l^T V'_l,   alpha_l = sigmoid(d_alpha_logits[b,l,h]),
 * computed in closed form as (prod_l alpha_l) S + sum_l (prod_{i>l} alpha_i) K'_l^T V'_l: a small
 * kernel forms the suffix products, then arl2_commit's kernels run with weighted value rows.
 * d_alpha_logits: [B, L, H] fp32.  Other arguments, reproducibility and errors as arl2_commit.
 */
int arl2_commit_decay_tokens(arl2_ctx* ctx, const void* d_k_clean, const void* d_v_clean,
                             const float* d_alpha_logits, void* stream);

/*
 * State commit with Eq. 4 applied token by token, in order, with per-token gates (the sentence
 * after Eq. 4): for l = 0..L-1
 *   S[b,h] <- alpha_l S[b,h] + beta_l K'_l^T (V'_l - K'_l S[b,h]),
 *   alpha_l = sigmoid(d_alpha_logits[b,l,h]), beta_l = sigmoid(d_beta_logits[b,l,h]),
 * both uses of S on the right being the state before token l (Eq. 4 as printed).  Computed in
 * chunkwise form (64 tokens per chunk: a triangular solve per chunk in parallel, then one ordered
 * pass over the chunks); bitwise reproducible.  With fp32 I/O, or D = 64, the arithmetic is fp32
 * throughout; with bf16 I/O and D = 128 the chunk factors are bf16 tensor-core operands with fp32
 * accumulation, the state itself staying fp32.
 * d_alpha_logits, d_beta_logits: [B, L, H] fp32, each may be NULL (gate = 1).  The context must
 * have been created with ARL2_FLAG_TOKEN_GATES (else ARL2_ERR_WORKSPACE).  K', V' as in
 * arl2_commit; calls of the three commit entry points may be mixed on one context.
 */
int arl2_commit_tokens(arl2_ctx* ctx, const void* d_k_clean, const void* d_v_clean,
                       const float* d_alpha_logits, const float* d_beta_logits, void* stream);

/*
 * The projections around the core (Sec. 3.1: Q = x W_q, K = x W_k, V = x W_v; Eq. 6: gate logits x W_g;
 * Eq. 7: y = O W_o), so that the context is a drop-in attention module: x, y are [B, L, d] with
 * d = H * D, and Q, K, V, O are the same memory read as [B, L, H, D].  Tensor-core contexts (bf16 I/O,
 * D = 128) only.  All weights are bf16, row-major, indexed (in, out): W_q, W_k, W_v, W_o [d, d],
 * W_g [d, H].
 *   arl2_projection_workspace_bytes  bytes of the caller-owned packing buffer (256-byte aligned)
 *   arl2_set_projections             copies W_q | W_k | W_v | W_g side by side into the packing buffer
 *                                    (one GEMM then yields all four results) and keeps the W_o pointer;
 *                                    the buffers must stay valid until replaced or the context is destroyed
 *   arl2_project_in                  d_q, d_k, d_v [B, L, H, D] bf16 and d_gate_logits [B, L, H] fp32 from
 *                                    d_x [B, L, d] bf16 -- one launch of a tcgen05 GEMM kernel
 *   arl2_project_out                 d_y [B, L, d] bf16 = d_o [B, L, H, D] W_o -- one launch
 * fp32 accumulation in tensor memory; results are rounded to bf16 (the gate logits stay fp32).
 */
size_t arl2_projection_workspace_bytes(const arl2_config* cfg);
int arl2_set_projections(arl2_ctx* ctx, const void* d_wq, const void* d_wk, const void* d_wv, const void* d_wg,
                         const void* d_wo, void* d_pack, size_t pack_bytes, void* stream);
int arl2_project_in(arl2_ctx* ctx, const void* d_x, void* d_q, void* d_k, void* d_v, float* d_gate_logits,
                    void* stream);
int arl2_project_out(arl2_ctx* ctx, const void* d_o, void* d_y, void* stream);

/* S <- 0 for stream `stream_index` (0..B-1) or all streams (-1): Algorithm 1, first line. */
int arl2_reset(arl2_ctx* ctx, int32_t stream_index, void* stream);

/*
 * Checkpoint / resume.  `dst` / `src` hold [B, H, D, D] fp32 and may be host or device
 * memory (cudaMemcpyDefault).  set_state also refreshes the operand copy of S.
 */
int arl2_get_state(arl2_ctx* ctx, float* dst, void* stream);
int arl2_set_state(arl2_ctx* ctx, const float* src, void* stream);

/*
 * Synchronise `stream` and return the device status word: ARL2_OK, or ARL2_ERR_TIMEOUT
 * if a bounded wait inside a kernel expired (the kernel then returned early; its output
 * is undefined, the context stays usable).  The word is cleared by the call.
 */
int arl2_sync_status(arl2_ctx* ctx, void* stream);

/*
 * Test hook for the time-out path (no counterpart in the paper): from the next launch on, every
 * bounded wait inside this context's tensor-core kernels gives up after `polls` polls (0 .. 65534;
 * see ARL2_FLAG_DEBUG_WAIT_LIMIT, which sets the same limit at creation); negative = back to the
 * default bound.  A denoise pass that timed out leaves its output undefined and S untouched; a
 * commit whose partial-sum kernel timed out leaves S untouched as well (the reduction that
 * follows it sees the recorded error and does nothing).
 */
int arl2_debug_set_wait_limit(arl2_ctx* ctx, int32_t polls);

/*
 * Measurement hook (no counterpart in the paper).  `ev_before` / `ev_after` are
 * cudaEvent_t handles (as void*) or NULL.  While set, the NEXT arl2_denoise_step records
 * them on its stream immediately before and after its dominant kernel (the fused
 * attention kernel, not the K rotation pass), then forgets them.  Lets a caller time that
 * kernel alone without a profiler.
 */
int arl2_set_profile_events(arl2_ctx* ctx, void* ev_before, void* ev_after);

/*
 * The state commit without any device allocation and without a context or workspace
 * (the paper has no counterpart; this is a service to constrained callers).
 *
 * Some callers of this library may not allocate device memory at the point where they must
 * commit: a plugin whose host owns the memory pool and forbids cudaMalloc, code running while
 * another component is capturing work on the stream, a process that was handed exactly the
 * layer's tensors and nothing else.  arl2_commit needs a workspace for the partial sums of its
 * split reduction; this entry point keeps those partial sums in an array built into the
 * library image instead (ARL2_STATIC_SCRATCH_BYTES per GPU, resident on every GPU that loads
 * the library until the process exits) and calls no cudaMalloc, cudaFree or allocating routine.
 *
 * Computes exactly what arl2_commit computes (plain-FMA kernels, fp32 or bf16 I/O):
 *   S[b,h] <- sigmoid(a[b,h]) S[b,h] + sum_l K'_l^T V'_l   on d_state [B,H,D,D] fp32 in place.
 * d_wphi_k / d_wphi_v: [H,D,D] (in,out) io_dtype or NULL; d_rope_cos / d_rope_sin: [L,D/2] fp32
 * or both NULL.  cfg->flags and cfg->softmax_scale are ignored.
 *
 * Limits and rules
 *   - B*H*ceil(L/512)*D*D*4 bytes must fit in ARL2_STATIC_SCRATCH_BYTES; larger shapes are
 *     rejected with ARL2_ERR_WORKSPACE and a message saying so (use arl2_commit then).
 *   - The first call on each device looks up the array's device address (the device must be
 *     current, as for any launch); make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps the previous call's contents.
 *     Nothing in it needs clearing (every slot read is written first by the same call), but
 *     two calls that overlap on the GPU (different streams, no ordering) race on it: order them.
 *   - d_state, d_k_clean, d_v_clean and the rope tables must be 16-byte aligned (a slice that
 *     starts in the middle of a row is refused with ARL2_ERR_INVALID_ARG before any launch).
 */
#define ARL2_STATIC_SCRATCH_BYTES (8u << 20)
int arl2_commit_static_scratch(const arl2_config* cfg, void* d_state, const void* d_k_clean,
                               const void* d_v_clean, const float* d_decay_logits,
                               const void* d_wphi_k, const void* d_wphi_v,
                               const float* d_rope_cos, const float* d_rope_sin, void* stream);

/* Number of kernel launches this context has issued so far (all entry points). */
uint64_t arl2_launch_count(const arl2_ctx* ctx);

/* Which kernel family serves arl2_denoise_step for this context: "tcgen05" or "simt". */
const char* arl2_step_kernel_name(const arl2_ctx* ctx);

/* Frees the host context only; no device buffer is touched and nothing is synchronised
   (the caller makes sure its streams are done with the workspace before reusing it). */
void arl2_destroy(arl2_ctx* ctx);

/* Thread-local message describing the last error returned on this thread ("" if none). */
const char* arl2_last_error(void);

/* Library version string. */
const char* arl2_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ARL2_H */
