/*
 * libflashdiff -- region-selective denoising step of a diffusion transformer on one B200.
 *
 * C ABI.  Unless a parameter says "host", every pointer is a DEVICE pointer owned by the
 * caller.  The library allocates no device memory: all scratch lives in the workspace the
 * caller hands to fd_create.  Every call enqueues its work on `cuda_stream` (a cudaStream_t
 * passed as void*; NULL = the default stream), performs no device-to-host synchronisation and
 * returns as soon as the work is queued; stream order is the only ordering.
 *
 * Errors a host can see (null or misaligned pointers, shapes beyond the limits given at
 * creation, unsupported head sizes) return a status with nothing launched.  Problems only the
 * device can see (a label outside [0,R], a bounded wait that ran out) never trap: the kernel
 * records a code in the workspace and skips the offending work.  No call reads that word back by
 * itself (that would be a synchronisation): fd_poll_status synchronises the stream and returns
 * it, and fd_destroy returns whatever is still unpolled.
 *
 * Test-only switches, read from the environment when a context is created; they select older or
 * restricted forms of a kernel and are not part of the interface: FD_PDL=0 (fully serialised
 * launches), FD_TC_PAIR=0 (single-CTA GEMM tiles), FD_TMA_RESID=0 (per-thread residual
 * reductions), FD_ATT_SPLIT=0|2 (never / always cut attention items along the keys),
 * FD_TC_MAX_CTAS=n (cap on persistent CTAs), FD_ATT_PAIR=1 (CTA-pair attention kernel at head dim 128), and, read at
 * every step, FD_TC_GROUPED=0 (dual stream: one launch per stream and projection instead of one grouped launch) and
 * FD_QK_FUSED=0 (QK-RMSNorm / rotary embedding in a kernel of their own instead of the QKV projection's epilogue).
 */
#ifndef FLASHDIFF_H_
#define FLASHDIFF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fd_ctx fd_ctx; /* opaque; created by fd_create, released by fd_destroy */

typedef enum {
    FD_OK = 0,
    FD_ERR_INVALID_ARG = 1, /* null / misaligned pointer, negative size                    */
    FD_ERR_SHAPE = 2,       /* shape beyond the limits of fd_config or inconsistent         */
    FD_ERR_STATE = 3,       /* device-side check failed (bad label, bad index)              */
    FD_ERR_WORKSPACE = 4,   /* workspace too small or misaligned                            */
    FD_ERR_UNSUPPORTED = 5, /* configuration this build has no kernel for                   */
    FD_ERR_CUDA = 6,        /* a CUDA runtime / driver call failed; see fd_last_error       */
    FD_ERR_TIMEOUT = 7      /* a bounded device-side wait expired                           */
} fd_status;

typedef enum { FD_F32 = 0, FD_BF16 = 1 } fd_dtype;

/* Which kernels run the dense contractions. */
typedef enum {
    FD_ENGINE_AUTO = 0,  /* tensor cores for FD_BF16, CUDA cores for FD_F32                 */
    FD_ENGINE_SIMT = 1,  /* CUDA-core GEMM and attention (any dtype; validation path)       */
    FD_ENGINE_TC = 2     /* tcgen05 / TMEM / TMA kernels (FD_BF16 only)                     */
} fd_engine;

/* Model shape and limits; copied at creation (host struct). */
typedef struct {
    int32_t n_blocks;    /* L                                                               */
    int32_t hidden;      /* H = n_heads * head_dim                                          */
    int32_t n_heads;
    int32_t head_dim;
    int32_t mlp_dim;     /* M                                                               */
    int32_t cond_dim;    /* Hc, width of the conditioning vector                            */
    int32_t max_batch;   /* largest B of any later call                                     */
    int32_t max_tokens;  /* largest N (tokens per request) of any later call                */
    int32_t max_regions; /* largest R of any later call                                     */
    int32_t dtype;       /* fd_dtype of x, cond, y, kv_cache and all weights                */
    int32_t engine;      /* fd_engine                                                       */
    float ln_eps;        /* LayerNorm epsilon (1e-6 in DiT)                                 */
    float gate_eta;      /* eta of the gate weight, Appendix A.1 Eq. (gate-weight)          */
    int32_t max_skip_k;  /* K of the forced reactivation, Appendix A.1                      */
} fd_config;

/*
 * Weights of all blocks (host struct of DEVICE pointers), borrowed until fd_destroy.
 * Row-major with the input dimension contiguous, block index outermost, element type
 * fd_config.dtype.  The six adaLN chunks of w_ada / b_ada are, in order: shift_msa,
 * scale_msa, gate_msa, shift_mlp, scale_mlp, gate_mlp.  All pointers 16-byte aligned.
 */
typedef struct {
    const void *w_qkv, *b_qkv; /* [L,3H,H], [L,3H]  rows: Q then K then V                   */
    const void *w_o, *b_o;     /* [L,H,H],  [L,H]                                           */
    const void *w_fc1, *b_fc1; /* [L,M,H],  [L,M]                                           */
    const void *w_fc2, *b_fc2; /* [L,H,M],  [L,H]                                           */
    const void *w_ada, *b_ada; /* [L,6H,Hc],[L,6H]                                          */
} fd_weights;

/* Bytes of device scratch fd_create needs for this configuration (0 if the config is bad). */
size_t fd_workspace_bytes(const fd_config* cfg);

/*
 * Creates a context on the current CUDA device.  `workspace` (256-byte aligned, at least
 * fd_workspace_bytes(cfg) bytes) is borrowed until fd_destroy and must not be touched by the
 * caller in between.  Builds the TMA descriptors of the weights and of the workspace tensors.
 * Synchronises the device once (set-up only).
 */
fd_status fd_create(const fd_config* cfg, const fd_weights* weights, void* workspace,
                    size_t workspace_bytes, fd_ctx** out);

/*
 * Patch Partitioner (paper Sec. 4.1; Appendix A.3, Eq. otsu and the hierarchical-extension
 * remark): groups the N tokens of each request into R regions from an early-step attention
 * map.  Saliency S_j is the mean over `salient_cols` of attn_map[b,j,:]; the map is min-max
 * normalised and quantised to 16 bits; a node is bisected at the threshold that maximises the
 * between-class variance (focus: value >= threshold); its region budget is shared by
 * r_f = argmin_r |r - R n_f/(n_f+n_c)|; both halves are split again until R regions exist.
 * A cut is admissible only if each side can hold its regions with min_region_tokens ..
 * max_region_tokens tokens per region (max_region_tokens <= 0: unbounded); a node without an
 * admissible cut is chopped in token order into equal chunks.  Ties: lowest threshold,
 * smallest r.  Regions are numbered by their smallest token index.
 *
 *   attn_map      [B,N,T] f32         salient_cols  [T_s] i32 or NULL (= all T columns)
 *   labels_out    [B,N]   i32         region_sizes_out [B,R] i32 or NULL
 * Needs 1 <= R <= N <= max_tokens, R <= max_regions, B <= max_batch, N < 65536.
 */
fd_status fd_partition_regions(fd_ctx* ctx, const float* attn_map, int B, int N, int T,
                               const int32_t* salient_cols, int T_s, int R, int min_region_tokens,
                               int max_region_tokens, int32_t* labels_out,
                               int32_t* region_sizes_out, void* cuda_stream);

/*
 * Patch Gate (paper Sec. 4.2; Appendix A.1 Eq. delta-i, Eq. gate-weight, Eq.
 * forced-reactivation; Algorithm 1, PatchGate) on the change of the latent between two
 * neighbouring steps.  For every region i of request b:
 *   - if the region ran at the previous step (prev_active = 1): delta_i = root mean square of
 *     z_cur - z_prev over the region's tokens and D channels; otherwise delta_i stays frozen;
 *   - w_i = (delta_i + eta) / sum_j (delta_j + eta);
 *   - active iff w_i >= eps[b], or the region was skipped max_skip_k steps in a row;
 *   - skip_count and prev_active are updated for the next evaluation.
 * Tokens with label R are always active and take no part in the gate.
 *
 *   z_cur, z_prev [B,N,D] f32 (16-byte aligned)   labels [B,N] i32 in [0,R]   eps [B] f32
 *   delta_state [B,R] f32, skip_count [B,R] i32, prev_active [B,R] u8   (in/out)
 *   score_out [B,R] f32 (= delta), weight_out [B,R] f32, mask_out [B,R] u8
 */
fd_status fd_region_activity(fd_ctx* ctx, const float* z_cur, const float* z_prev,
                             const int32_t* labels, int B, int N, int D, int R, const float* eps,
                             float* delta_state, int32_t* skip_count, uint8_t* prev_active,
                             float* score_out, float* weight_out, uint8_t* mask_out,
                             void* cuda_stream);

/*
 * One denoising step of the block stack on the active regions only (paper Sec. 3 "Adaptive
 * execution": active patches are refined, skipped patches reuse cached states; Sec. 5: active
 * patches run against the previous step's K/V and refresh only their own K/V; Appendix A.6).
 *   1. tokens whose region is active (mask[b,labels[b,j]] != 0, or label R) are compacted into
 *      the ascending list active_idx_out (values b*N+j) with offsets cu_active_out [B+1];
 *   2. per block: gather, LayerNorm + adaLN modulation, QKV projection; Q stays compact, the
 *      K and V rows of active tokens overwrite kv_cache[l,b,0/1,j,:]; all other rows keep the
 *      values of the step at which their token last ran;
 *   3. each active query attends to all N keys of its request (fresh and cached);
 *   4. out-projection, gated residual, LayerNorm + modulation, tanh-GELU MLP, gated residual;
 *   5. after the last block the rows are scattered to y[b,j,:]; all other rows of y keep their
 *      cached output.
 * The first step on fresh kv_cache / y must use an all-ones mask (the warm-up steps).
 *
 *   x [B,N,H], cond [B,Hc], y [B,N,H], kv_cache [L,B,2,N,H]  of fd_config.dtype, 16-byte aligned
 *   labels [B,N] i32, mask [B,R] u8
 *   active_idx_out [B*N] i32 (capacity), cu_active_out [B+1] i32
 * Needs 1 <= R <= N <= max_tokens, R <= max_regions, B <= max_batch; the i32 arrays 4-byte aligned.
 */
fd_status fd_regional_step(fd_ctx* ctx, const void* x, const void* cond, const int32_t* labels,
                           const uint8_t* mask, int B, int N, int R, void* kv_cache, void* y,
                           int32_t* active_idx_out, int32_t* cu_active_out, void* cuda_stream);

/*
 * Block variants of the models the paper evaluates (Sec. 6.1; FLUX.1-dev, SD3-Medium and Wan2.1 normalise queries
 * and keys and / or rotate them by position).  The paper does not define them; the conventions here are those of the
 * published architectures:
 *   QK-RMSNorm  every head slice x [head_dim] of a query / key row becomes
 *               x / sqrt(mean(x^2) + qk_norm_eps) * w,  w = q_norm_w[l] for queries, k_norm_w[l] for keys of block l
 *               (one weight vector per block, shared by all heads);
 *   RoPE        then the channel pairs (2i, 2i+1) of every head are rotated by the angle of the token's position:
 *               (a, b) -> (a cos - b sin, a sin + b cos) with cos = rope_cos[j, i], sin = rope_sin[j, i], j the token's
 *               index inside its request (the caller tabulates the angles, so 1-D, axial or constant-for-text positions
 *               are all expressible).
 * Applied to the fresh Q and K rows of every block right after the QKV projection; the cache keeps keys in this final
 * form, so rows of skipped tokens never need re-rotation.  V is unchanged.
 *   q_norm_w, k_norm_w [L, head_dim] of fd_config.dtype, both or neither (NULL = no normalisation)
 *   rope_cos, rope_sin [max_tokens, head_dim/2] f32, both or neither (NULL = no rotation; needs an even head_dim)
 * DEVICE pointers, 4-byte aligned (8-byte for f32 weights), borrowed until the next call or fd_destroy.  v = NULL switches
 * every variant off.  Takes effect for the steps queued after the call returns.
 */
typedef struct {
    const void* q_norm_w;
    const void* k_norm_w;
    float qk_norm_eps;
    const float* rope_cos;
    const float* rope_sin;
    const void* q_norm_w_text; /* [L, head_dim]: QK-norm weights of the second stream (fd_set_text_stream), both or */
    const void* k_norm_w_text; /* neither; NULL = the second stream shares q_norm_w / k_norm_w                    */
} fd_block_variants;
fd_status fd_set_block_variants(fd_ctx* ctx, const fd_block_variants* v);

/*
 * Dual-stream blocks (the joint text-image architecture of the paper's FLUX.1-dev and SD3-Medium models; no
 * definition in the paper, this is the published structure): the tokens of a request belong to one of two streams,
 * and a token's stream selects the weights of everything that acts per token -- the adaLN conditioning (w_ada,
 * b_ada), the QKV projection, the QK-norm weights, the out-projection and the MLP -- while the attention stays joint
 * over all tokens of the request.  The second stream is the always-active tokens (label R: the text tokens of a
 * joint text-image request); `text_weights` has the layout of fd_weights and is borrowed until the next call or
 * fd_destroy.  NULL returns to a single stream.  Each projection then walks every row tile with the first stream's
 * weights and, in the same launch, the row tiles that hold rows of the second stream with the second stream's
 * weights; a tile's epilogue finishes only the rows of its own stream.
 */
fd_status fd_set_text_stream(fd_ctx* ctx, const fd_weights* text_weights);

/*
 * Cross-attention to a fixed context (the text conditioning of the paper's Wan2.1 and PixArt-style blocks; no equation
 * of the paper covers it, the reading is the published block structure of those models).  When set, every block
 * does, between the self-attention update and the MLP branch and for the active rows only,
 *     r <- r + W_o . Attn(LN(r) W_q^T + b_q, K_ctx, V_ctx) + b_o
 * with LN the plain LayerNorm of the block (ln_eps; no scale, shift or adaLN modulation), Attn the per-head
 * softmax(q k^T / sqrt(head_dim)) over the n_ctx context tokens of the row's request, and no gate.  The context's
 * keys and values are the caller's (a text encoder's states, projected once per prompt): they do not depend on
 * the step, so region skipping leaves them alone, and a skipped row keeps its cached block output as before.
 * DEVICE pointers in the storage type, 16-byte aligned, owned by the caller and alive while set:
 *   w_q, w_o [L, H, H] (out, in), b_q, b_o [L, H], ctx_kv [L, ctx_batch, 2, n_ctx, H] (keys then values; heads
 *   side by side as in the self-attention cache).  n_ctx >= 1.  A step with B != ctx_batch fails with
 *   FD_ERR_SHAPE.  In a dual-stream context both streams use this one set.  NULL switches it off.  Host call, no
 *   launch; takes effect from the next step.
 */
typedef struct fd_cross_attention {
    const void* w_q;
    const void* b_q;
    const void* w_o;
    const void* b_o;
    const void* ctx_kv;
    int n_ctx;
    int ctx_batch;
} fd_cross_attention;
fd_status fd_set_cross_attention(fd_ctx* ctx, const fd_cross_attention* cross);

/*
 * FP8 operands for the QKV, fc1 and fc2 projections (8-bit inference of the paper's models; the paper does not
 * cover it, the convention is this library's).  Both operands of those three products are OCP E4M3 values (4
 * exponent bits, bias 7, 3 mantissa bits, largest magnitude 448, no infinities):
 *   weights     quantised by the caller, row o of W standing for s[o] * w8[o, :]
 *               (w8_* DEVICE, E4M3 bytes, [L, 3H, H], [L, M, H], [L, H, M]; s_* DEVICE f32 [L, 3H], [L, M], [L, H]);
 *   activations quantised by the library where they are produced (the two modulated LayerNorm outputs, the GELU
 *               output) as E4M3(value * (1 / a)), round to nearest even, saturating, with one scale a per tensor and
 *               block: a_scale, a HOST array [L, 3] (inputs of QKV, fc1, fc2), copied by this call;
 *   result      (exact products, fp32 accumulation) * (a * s[o]) + bias, then as without FP8.
 * The attention, the out-projection, the cross-attention and all vector work stay in bf16 / fp32.  Tensor-core
 * engine with bf16 storage only, hidden and mlp_dim multiples of 192 or 256 (else FD_ERR_UNSUPPORTED).  Pointers
 * 16-byte aligned, owned by the caller and alive while set.  NULL switches it off.  Host call, no launch; takes effect
 * from the next step.
 * With a second stream (fd_set_text_stream) that stream's three projections need 8-bit operands of their own, given
 * by fd_set_fp8_text_stream in the same form (its own quantised weights, row scales and activation scales; a row is
 * quantised with the scale of the stream it belongs to); a step that finds FP8 operands and a second stream but not
 * the second stream's operands fails with FD_ERR_UNSUPPORTED.
 */
typedef struct fd_fp8_operands {
    const void* w8_qkv;
    const float* s_qkv;
    const void* w8_fc1;
    const float* s_fc1;
    const void* w8_fc2;
    const float* s_fc2;
    const float* a_scale;
} fd_fp8_operands;
fd_status fd_set_fp8_operands(fd_ctx* ctx, const fd_fp8_operands* fp8);
fd_status fd_set_fp8_text_stream(fd_ctx* ctx, const fd_fp8_operands* fp8_text);

/*
 * The Patch Gate on the paper's own signal (Sec. 4.2): the refinement importance of a patch is the block mean of
 * the self-attention matrix over the patch,  R_i = (1/|A_i|^2) sum_{u,v in A_i} SA[u,v],  and the gate weights are
 * the normalised changes  Delta_i = |R_i - Rbar_i|  (Rbar_i = the importance at the patch's last executed step;
 * a skipped patch keeps its Delta_i).  SA is taken from the FIRST block of the step, softmax probabilities averaged
 * over heads.
 *
 * fd_regional_step_mass is fd_regional_step that additionally writes
 *   region_mass_out [B,R] f64 (DEVICE):  sum over the ACTIVE queries u of region i and over the keys v of region i
 *   of SA[u,v] (zero for regions that did not run; tokens with label R belong to no region).
 * Both engines accumulate the mass inside the first block's attention kernel.
 *
 * fd_region_activity_attn turns it into the next step's mask: for every region executed at the step that produced
 * region_mass (prev_active = 1),  R_i = region_mass / region_sizes^2,  Delta_i = |R_i - Rbar_i|,  Rbar_i <- R_i;
 * weights, threshold, forced reactivation and the skip_count / prev_active updates are those of fd_region_activity.
 *   region_sizes [B,R] i32 (tokens per region, as fd_partition_regions returns them)
 *   state in/out: rbar_state, delta_state [B,R] f32 (start at zero), skip_count [B,R] i32, prev_active [B,R] u8
 *   outputs [B,R]: importance_out f32 (Rbar after the update), weight_out f32, mask_out u8
 */
fd_status fd_regional_step_mass(fd_ctx* ctx, const void* x, const void* cond, const int32_t* labels,
                                const uint8_t* mask, int B, int N, int R, void* kv_cache, void* y,
                                int32_t* active_idx_out, int32_t* cu_active_out, double* region_mass_out,
                                void* cuda_stream);
fd_status fd_region_activity_attn(fd_ctx* ctx, const double* region_mass, const int32_t* region_sizes, int B, int R,
                                  const float* eps, float* rbar_state, float* delta_state, int32_t* skip_count,
                                  uint8_t* prev_active, float* importance_out, float* weight_out, uint8_t* mask_out,
                                  void* cuda_stream);

/*
 * Sampler closure around the step: patch embedding before it, final layer and latent update after it
 * (Appendix A.1, Eq. sf-update: an active patch moves along its fresh drift, a skipped patch along
 * the drift cached at its most recent active step).  With these two calls a gated multi-step loop
 *     x = embed(z);  mask = gate(z, z_prev);  y = step(x, mask);  z_next = update(z, y)
 * runs entirely on the device.  Both maps are per token, so a "patch" is the set of tokens with its label.
 *
 * Weights (host struct of DEVICE pointers, element type fd_config.dtype, 16-byte aligned, borrowed for
 * the duration of the call):
 *   w_in [H,D], b_in [H], pos [N,H]   patch embedding  x[b,j,:] = z[b,j,:] w_in^T + b_in + pos[j,:]
 *   w_out [D,H], b_out [D]            final layer      drift = LayerNorm(y row, no affine, fd_config.ln_eps) w_out^T + b_out
 * D = latent_dim: a multiple of 4, at most 256.
 */
typedef struct {
    const void *w_in, *b_in, *pos;
    const void *w_out, *b_out;
    int32_t latent_dim;
} fd_sampler_weights;

/*   z [B,N,D] f32  ->  x_out [B,N,H] of fd_config.dtype (all tokens; the step reads the active ones).  */
fd_status fd_embed_latent(fd_ctx* ctx, const fd_sampler_weights* sw, const float* z, int B, int N, void* x_out,
                          void* cuda_stream);

/*
 * One application of Eq. sf-update after fd_regional_step:
 *   for every active token (active_idx / cu_active as the step wrote them): drift[b,j,:] = final layer of y[b,j,:];
 *   for every token: z_next[b,j,:] = z[b,j,:] + h[b] * drift[b,j,:]   (the cached drift where the token was skipped).
 *   z, z_next, drift_cache [B,N,D] f32 (z_next may be z); y [B,N,H] of fd_config.dtype; h [B] f32;
 *   active_idx [>= A] i32, cu_active [B+1] i32 (DEVICE; A = cu_active[B] is read on the device).
 * drift_cache is in/out state: rows of active tokens are overwritten, the others are only read, so the first
 * call must follow an all-active step.
 */
fd_status fd_update_latent(fd_ctx* ctx, const fd_sampler_weights* sw, const float* z, const void* y,
                           const int32_t* active_idx, const int32_t* cu_active, const float* h, int B, int N,
                           float* drift_cache, float* z_next, void* cuda_stream);

/*
 * The gate for callers that cannot allocate device memory (no counterpart in the paper; added for
 * embedding).  Some hosts of this library may not call cudaMalloc at all: a plug-in running inside
 * an inference server whose memory pool was sized and frozen at start-up, code on a latency-critical
 * thread where an allocation would serialise the whole device, or a process that has already handed
 * every byte of the GPU to its own arena.  Such a caller cannot provide the workspace fd_create
 * wants, so this entry point needs neither a context nor a workspace: it computes exactly what
 * fd_region_activity computes (same kernels, same argument meaning), with its per-region
 * accumulators in a fixed array that is part of the library image.
 *
 *  - Limit: B * R <= FD_NOALLOC_MAX_REGION_SLOTS; larger problems are refused with FD_ERR_SHAPE
 *    and nothing is launched.  The array (about 200 KB) is resident on every GPU that loads the
 *    library, from load until the process exits.
 *  - The first call on each device looks up the array's device address (with that device current).
 *    Make that first call outside any stream capture.
 *  - All calls on one device share the array and it keeps what the last call left in it; every
 *    call clears the part it uses before use.  Two calls whose GPU work overlaps (different
 *    streams without ordering, or different host threads) race on it: serialise them.
 *  - No cudaMalloc / cudaFree or any other allocating routine is called, by this function or the
 *    kernels it launches.
 *  - eta and max_skip_k take the place of the values a context would hold.
 *  - status_out: optional DEVICE int32 that receives, in stream order, 0, FD_ERR_STATE if a label was
 *    outside [0,R] (such tokens are skipped), or FD_ERR_TIMEOUT if a bounded wait of the streaming
 *    reduction ran out (the result is then incomplete); may be NULL.
 */
#define FD_NOALLOC_MAX_REGION_SLOTS 16384
fd_status fd_region_activity_noalloc(const float* z_cur, const float* z_prev, const int32_t* labels, int B,
                                     int N, int D, int R, const float* eps, float eta, int max_skip_k,
                                     float* delta_state, int32_t* skip_count, uint8_t* prev_active,
                                     float* score_out, float* weight_out, uint8_t* mask_out,
                                     int32_t* status_out, void* cuda_stream);

/*
 * Reads the device-side status word (synchronises `cuda_stream`).  Returns FD_OK, or the first
 * device-side problem recorded since the last poll (FD_ERR_STATE / FD_ERR_TIMEOUT), and clears it.
 */
fd_status fd_poll_status(fd_ctx* ctx, void* cuda_stream);

/*
 * Self-test of the bounded device-side waits: launches one thread that waits on a barrier nothing ever
 * signals.  The wait gives up after its poll limit (about a second), the kernel records FD_ERR_TIMEOUT and
 * returns normally; the next fd_poll_status reports FD_ERR_TIMEOUT and the context stays usable.
 */
fd_status fd_selftest_bounded_wait(fd_ctx* ctx, void* cuda_stream);

/* Number of kernels the library has launched through this context so far (host counter). */
int64_t fd_launch_count(const fd_ctx* ctx);

/*
 * Optional per-kernel timing.  While enabled, every kernel group the library launches is bracketed
 * by CUDA events on the caller's stream.  fd_profile_read synchronises `cuda_stream`, adds the
 * elapsed milliseconds and the kernel counts per group into the two HOST arrays of
 * FD_PROF_GROUPS entries, and forgets the recorded events.
 */
enum {
    FD_PROF_ACTIVITY = 0, /* activity reduce + gate          */
    FD_PROF_COMPACT = 1,  /* compaction (count + write)      */
    FD_PROF_ADALN = 2,    /* adaLN conditioning vectors      */
    FD_PROF_LN = 3,       /* gather + LayerNorm + modulation */
    FD_PROF_GEMM_QKV = 4,
    FD_PROF_ATTENTION = 5,
    FD_PROF_GEMM_OUT = 6,
    FD_PROF_GEMM_FC1 = 7,
    FD_PROF_GEMM_FC2 = 8,
    FD_PROF_PARTITION = 9,
    FD_PROF_SAMPLER = 10, /* patch embedding, final layer, latent update */
    FD_PROF_QK_VARIANTS = 11, /* QK-RMSNorm + rotary embedding (block variants) */
    FD_PROF_CROSS = 12,   /* cross-attention: LayerNorm, query projection, attention, out-projection */
    FD_PROF_GROUPS = 13
};
/*
 * Inspection of the step's intermediate buffers (they live in the caller's workspace): returns the DEVICE address and
 * the size in bytes of one of them, as the last fd_regional_step left it (valid rows: the step's active rows, compact
 * order).  For tests and debugging; nothing is launched and nothing is copied.
 *   FD_BUF_ACT     [rows, H]   the last modulated-LayerNorm output: storage type, or E4M3 bytes with FP8 operands
 *   FD_BUF_HIDDEN  [rows, M]   the last block's MLP hidden activations: storage type, or E4M3 bytes with FP8 operands
 *   FD_BUF_RESID   [rows, H]   f32 residual stream after the last block (tensor-core engine)
 *   FD_BUF_Q       [rows, q_ld] the last block's query rows, storage type; q_ld = bytes / (rows capacity * element size):
 *                              n_heads * head_dim, except that the tensor-core attention stores a 72-wide head in 80
 *                              columns (the last 8 zero)
 *   FD_BUF_ATTN    [rows, H]   the last block's self-attention output (or the cross-attention's, when that is set)
 */
enum { FD_BUF_ACT = 0, FD_BUF_HIDDEN = 1, FD_BUF_RESID = 2, FD_BUF_Q = 3, FD_BUF_ATTN = 4 };
fd_status fd_debug_buffer(fd_ctx* ctx, int which, void** device_ptr_out, size_t* bytes_out);

fd_status fd_profile_enable(fd_ctx* ctx, int enable);
fd_status fd_profile_read(fd_ctx* ctx, void* cuda_stream, float* ms_out, int32_t* kernels_out);

/*
 * Host-side batch former (Sec. 4.3, patch monotasks).  Pure host code: every pointer below is HOST memory, no
 * context, no CUDA call, no allocation; safe to call from any thread.
 *
 * fd_sched_pack -- the least-maximum-load rule (the equation of Sec. 4.3, "Monotask Packing").  Monotasks are
 * assigned one after another in the given order; monotask j of cost[j] goes to
 *     g* = argmin_g  max_g' ( load[g'] + cost[j] if g' == g else load[g'] ).
 * Among devices that tie on that maximum, home[j] (the device that already holds patches of the same request;
 * -1 for a warm-up monotask, which has none) wins if it is one of them, else the one with the smallest own load,
 * else the smallest index.  load [n_devices] f64 is read and updated in place; assign_out [n_tasks] receives g*.
 * O(n_devices) per monotask.  Errors: FD_ERR_INVALID_ARG for null pointers, n_devices < 1, n_tasks < 0, a
 * negative or non-finite cost or load, or home[j] >= n_devices (nothing is written in that case).
 *
 * fd_sched_form_batch -- which requests run the next device step.  A request's step is one unit (its active
 * patches run together; switching happens only at step boundaries, i.e. when this is called).  Requests are
 * visited by (priority descending, arrival ascending, index ascending); a request is taken if its active_tokens
 * still fit into what is left of token_budget and its state is resident or a residency slot (max_resident minus the
 * number of resident requests) is free, in which case it takes the slot; a request that does not fit is passed over
 * and lower-priority ones may use the leftover.  A request without active tokens is taken only if it is resident.
 *   priority, arrival [n] i32/i64; active_tokens [n] i32 (>= 0); resident [n] u8 in/out; chosen_out [n] u8.
 * Errors: FD_ERR_INVALID_ARG for null pointers, n < 0, negative tokens or budget, max_resident < 0.
 */
fd_status fd_sched_pack(int n_devices, double* load, int n_tasks, const double* cost, const int32_t* home,
                        int32_t* assign_out);
fd_status fd_sched_form_batch(int n, const int32_t* priority, const int64_t* arrival, const int32_t* active_tokens,
                              uint8_t* resident, int64_t token_budget, int max_resident, uint8_t* chosen_out);

/*
 * Adaptive patch granularity (Sec. 4.1): performance as a function of the number of patches R is unimodal, and R is
 * tuned online by a bounded binary search on the performance observed for past requests.  Pure host code; the state
 * is a plain struct owned by the caller (HOST memory).
 *   fd_rsearch_init    R in [r_min, r_max], first R to run = r_start; initial step = half the range, rounded up.
 *   fd_rsearch_update  observed_perf (higher is better) belongs to the R returned last (the first call: to r_start).
 *                      Better than the accepted R's -> the candidate becomes the accepted R, same direction and step;
 *                      not better -> the direction flips and the step halves (never below 1).  The next candidate is
 *                      accepted + direction * step clamped to the range; one that equals the accepted R counts as not
 *                      better without being run.  Two failures in a row at step 1 end the search (converged = 1): the
 *                      accepted R is returned from then on.  *next_r receives the R to run next.
 * Errors: FD_ERR_INVALID_ARG for null pointers, r_min < 1, r_min > r_max, r_start outside the range, a NaN performance.
 */
typedef struct {
    int32_t r_min, r_max;
    int32_t accepted, candidate; /* accepted R and the one being evaluated */
    int32_t step, dir;           /* dir = +1 / -1 */
    int32_t have_ref, fails_at_one, converged;
    double ref_perf;             /* performance observed with the accepted R */
} fd_rsearch;
fd_status fd_rsearch_init(fd_rsearch* st, int r_min, int r_max, int r_start);
fd_status fd_rsearch_update(fd_rsearch* st, double observed_perf, int32_t* next_r);

/* Releases the context (host memory only; the workspace goes back to the caller).  Synchronises the
 * device first and returns FD_OK, or a device-side status (FD_ERR_STATE / FD_ERR_TIMEOUT) that was
 * recorded and never polled; the context is released either way. */
fd_status fd_destroy(fd_ctx* ctx);

/* Text of the last error of this context (host string owned by the context; NULL ctx: text of
 * the last failed fd_create on this thread). */
const char* fd_last_error(const fd_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* FLASHDIFF_H_ */
