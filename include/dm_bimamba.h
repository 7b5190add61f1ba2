/*
 * dm_bimamba.h -- C ABI of the B200 (sm_100a) bidirectional Mamba-2 mixer used as the denoiser
 * backbone of a masked-diffusion language model (DiffuMamba, Sec. 3.2 and App. A.1).
 *
 * General rules for every entry point
 *   - Unless a parameter says "host", every data pointer is a DEVICE pointer owned by the caller.
 *     The structs themselves (configs, weight tables, state tables) live in HOST memory and are read
 *     during the call only; the library keeps no pointer after the call returns.
 *   - All tensors are dense, row-major, contiguous.  Matrices are [out_features, in_features].
 *   - `dtype` selects the storage type of activations, matrices, conv parameters, norm weights and the
 *     conv state (DM_F32 or DM_BF16).  Accumulation is always fp32; per-head scalars (dt_bias, A_log, D)
 *     and the SSM state are always fp32.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = the default stream)
 *     and the call returns without synchronising.  The library allocates no device memory: scratch
 *     comes from the caller's `workspace` (query its size first; 256-byte aligned).
 *   - Return value: DM_OK (0) or a negative dm_status.  Arguments are checked before anything is
 *     launched; a rejected call has no effect.  dm_last_error_message() gives a text for the last
 *     failure on the calling thread.
 *   - Column order of one direction's in_proj output (App. C, "D_in"):
 *         [ z : d_inner | x : d_inner | B : n_groups*d_state | C : n_groups*d_state | dt : n_heads ].
 *     conv_ch = d_inner + 2*n_groups*d_state channels (x, B, C) pass through the depthwise conv.
 */
#ifndef DM_BIMAMBA_H_
#define DM_BIMAMBA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DM_OK = 0,
    DM_ERR_INVALID_ARG = -1,   /* NULL pointer, non-positive size, misaligned pointer, aliasing states */
    DM_ERR_UNSUPPORTED = -2,   /* a shape the kernels do not cover (see dm_mixer_cfg) */
    DM_ERR_WORKSPACE = -3,     /* workspace NULL, misaligned or smaller than the queried size */
    DM_ERR_CUDA = -4,          /* a CUDA runtime call failed (launch configuration, driver) */
    DM_ERR_TIMEOUT = -5        /* a bounded device-side wait gave up (reported by dm_check) */
} dm_status;

enum { DM_F32 = 0, DM_BF16 = 1 };
enum { DM_FLAG_GATED_RMSNORM = 1, DM_FLAG_CONV_BIAS = 2, DM_FLAG_D_SKIP = 4,
       /* App. A.1 hyper-parameter "bidirectional weight tie" (False in the paper's runs): the two directions share in_proj and
          out_proj (w[0].w_in, w[0].w_out; the ones of w[1] are not read) and keep their own conv, step-size, decay, skip and norm
          parameters.  The shared in_proj is then computed once and the sum of the directions is taken before the one out_proj:
          Mamba(x) = W_out (g-> + g<-), with each direction's gated-norm scale applied to its g first. */
       DM_FLAG_TIED_PROJ = 8 };
enum { DM_DIR_FWD = 1, DM_DIR_REV = 2, DM_DIR_BOTH = 3 };

/* Sizes of one mixer call, in the paper's notation (Sec. 3.2: x in R^{B x L x d}; App. A.1
 * hyper-parameter table: expansion factor, state dimension, conv dimension; App. C: heads via D_in).
 * Supported: d_conv in [2,4]; n_groups == 1; headdim = expand*d_model/n_heads in {32, 64};
 * d_state in {16, 32, 64, 128, 256} with headdim*d_state/16 <= 1024.  Other shapes return
 * DM_ERR_UNSUPPORTED. */
typedef struct {
    int32_t batch;      /* B */
    int32_t seqlen;     /* L; for dm_bimamba_block_step the length G of the active block */
    int32_t d_model;    /* d */
    int32_t expand;     /* d_inner = expand * d_model */
    int32_t d_state;    /* N, states per channel */
    int32_t d_conv;     /* k, width of the depthwise conv */
    int32_t n_heads;    /* H; the decay and step size are scalars per head */
    int32_t n_groups;   /* groups sharing B and C */
    int32_t dtype;      /* DM_F32 | DM_BF16 */
    int32_t flags;      /* DM_FLAG_* */
    int32_t dir_mask;   /* DM_DIR_BOTH; one direction alone is meant for invariant tests */
    int32_t chunk;      /* tokens per scan chunk; 0 = library default.  Results do not depend on it
                           beyond rounding order.  bf16 with d_state <= 128 runs the chunked form of the
                           recurrence and takes 0, 128 (tensor-core kernel; the default above 64 tokens)
                           or 32 (CUDA-core kernel; the default up to 64 tokens, i.e. for the blocks of
                           block-autoregressive decoding) -- other values: DM_ERR_UNSUPPORTED.  fp32, and
                           d_state 256, run the sequential form, where any chunk > 0 only sizes the
                           staging buffers. */
    float   norm_eps;   /* epsilon of the gated RMS norm */
} dm_mixer_cfg;

/* One direction's parameters (the two directions are untied: App. A.1 "bidirectional weight tie: False"). */
typedef struct {
    const void  *w_in;     /* [d_in_proj, d_model]  dtype */
    const void  *conv_w;   /* [conv_ch, d_conv]     dtype; tap d_conv-1 multiplies the current token */
    const void  *conv_b;   /* [conv_ch]             dtype; ignored unless DM_FLAG_CONV_BIAS */
    const float *dt_bias;  /* [n_heads] */
    const float *A_log;    /* [n_heads]; A = -exp(A_log) */
    const float *D;        /* [n_heads]; ignored unless DM_FLAG_D_SKIP */
    const void  *norm_w;   /* [d_inner] dtype; ignored unless DM_FLAG_GATED_RMSNORM */
    const void  *w_out;    /* [d_model, d_inner]    dtype */
} dm_dir_weights;

typedef struct {
    const void    *norm_w;     /* [d_model] dtype: RMSNorm pre-norm weight of the layer */
    dm_dir_weights dir[2];     /* [0] left-to-right, [1] right-to-left */
} dm_layer_weights;

typedef struct {
    dm_mixer_cfg mixer;        /* batch/seqlen describe the token tensor of the step */
    int32_t n_layers;
    int32_t vocab;             /* rows of embed and w_vocab */
    float   rms_eps;
} dm_stack_cfg;

typedef struct {
    const void             *embed;         /* [vocab, d_model] dtype */
    const dm_layer_weights *layers;        /* HOST array of n_layers entries */
    const void             *final_norm_w;  /* [d_model] dtype */
    const void             *w_vocab;       /* [vocab, d_model] dtype */
} dm_stack_weights;

/* The timestep-conditioned block of App. A.1 around the mixer (used by dm_denoise_step_cond):
 *     y_mixer = x + g1 * Mamba(AdaLN1(x; tau)),     y_mlp = y_mixer + g2 * MLP(AdaLN2(y_mixer; tau)),
 *     AdaLN(x; tau) = gamma * (x - mean(x)) / sqrt(var(x) + ln_eps) + beta   over the channels of each token,
 *     [beta1 | gamma1 | g1 | beta2 | gamma2 | g2] = W_cond tau + b_cond      (6 * d_model values per sequence),
 *     MLP(u) = W_down GELU(W_up u + b_up) + b_down   (GELU in its tanh form).
 * The paper's equations show gamma and beta only; its FLOP table counts 6 * d_model modulation outputs
 * per layer, read here as a third vector per sublayer that gates the sublayer's output (g = 1 gives the
 * equations as printed). */
typedef struct {
    int32_t d_ff;      /* hidden width of the MLP (the paper: 2 * d_model) */
    int32_t d_cond;    /* width of the timestep embedding tau (the paper: 128) */
    float   ln_eps;
} dm_block_cfg;

typedef struct {
    const void  *w_cond;   /* [6 * d_model, d_cond] dtype */
    const float *b_cond;   /* [6 * d_model] fp32 or NULL */
    const void  *w_up;     /* [d_ff, d_model] dtype */
    const float *b_up;     /* [d_ff] fp32 or NULL */
    const void  *w_down;   /* [d_model, d_ff] dtype */
    const float *b_down;   /* [d_model] fp32 or NULL */
} dm_block_weights;

/* Carried state of one layer in block mode (Sec. 4.3): only the left-to-right direction has one.
 * *_in == NULL means zeros (no prefix yet); *_out == NULL means "do not commit".  in and out must not
 * be the same buffer. */
typedef struct {
    const float *ssm_in;    /* [B, H, P, N] fp32 */
    const void  *conv_in;   /* [B, d_conv-1, conv_ch] dtype: the d_conv-1 pre-conv rows before the block */
    float       *ssm_out;
    void        *conv_out;
} dm_layer_state;

/* Text for a status code (static storage, never NULL). */
const char *dm_status_string(int status);

/* Text describing the last failure on the calling thread (static thread-local storage). */
const char *dm_last_error_message(void);

/* Scratch sizes in bytes for the calls below with the same configuration. */
int dm_bimamba_workspace_bytes(const dm_mixer_cfg *cfg, size_t *bytes);
int dm_denoise_workspace_bytes(const dm_stack_cfg *cfg, size_t *bytes);

/* Synchronises `cuda_stream` and returns the deferred device status (DM_OK, DM_ERR_TIMEOUT when a
 * bounded wait inside a kernel expired, DM_ERR_CUDA for a sticky CUDA error).  Clears the status. */
int dm_check(void *cuda_stream);

/* The bidirectional mixer, Sec. 3.2:  y = Mamba(x) = h-> + h<-  for x [B, L, d_model].
 * Each direction is a complete Mamba-2 layer (App. C table): in_proj, depthwise conv + SiLU over
 * (x,B,C), Delta = softplus(dt + dt_bias), a = exp(Delta*A), the recurrence
 * h_t = a_t h_{t-1} + Delta_t x_t (x) B_t,  y_t = h_t C_t + D x_t, gate by SiLU(z) (then the gated
 * RMS norm when flagged), out_proj.  The right-to-left layer runs the same operator over the
 * sequence in reverse order (anti-causal conv, recurrence from t = L-1 down to 0).
 *   w[0], w[1]: left-to-right and right-to-left parameters.   x, y: [B, L, d_model] dtype; y != x. */
int dm_bimamba_forward(const dm_mixer_cfg *cfg, const dm_dir_weights w[2],
                       const void *x, void *y,
                       void *workspace, size_t workspace_bytes, void *cuda_stream);

/* One pass over the active block in block-autoregressive decoding, Sec. 4.3: cfg->seqlen = G.
 * The left-to-right layer starts from the carried state of the committed prefix (ssm_state_in,
 * conv_state_in; NULL = zeros) and, when the *_out pointers are given, writes the state after the
 * block's last token.  The right-to-left layer starts from zero and sees the block only.
 *   x_blk, y_blk: [B, G, d_model] dtype.  conv_state_out holds the last d_conv-1 rows of
 *   concat(conv_state_in, pre-conv xBC of the block) -- exact copies, also when G < d_conv-1. */
int dm_bimamba_block_step(const dm_mixer_cfg *cfg, const dm_dir_weights w[2],
                          const void *x_blk,
                          const float *ssm_state_in, const void *conv_state_in,
                          float *ssm_state_out, void *conv_state_out,
                          void *y_blk,
                          void *workspace, size_t workspace_bytes, void *cuda_stream);

/* One denoising step of the layer stack, App. A.1:  z = OutputProj(B_N(... B_1(E(x_t)))) with
 * r_0 = E[tokens], r_{l+1} = r_l + Mamba_l(RMSNorm(r_l) * norm_w_l), logits = W_vocab (RMSNorm(r_N) * w_f).
 *   tokens: [B, L] int32 ids in [0, vocab).   logits: [B, L, vocab] dtype, or NULL.
 *   argmax_out: [B, L] int32 = index of the largest logit (lowest index on ties), or NULL.
 *   states: HOST array of n_layers entries, or NULL for full-sequence denoising; when given, every
 *   layer runs as dm_bimamba_block_step with that layer's state pointers. */
int dm_denoise_step(const dm_stack_cfg *cfg, const dm_stack_weights *weights,
                    const int32_t *tokens, void *logits, int32_t *argmax_out,
                    const dm_layer_state *states,
                    void *workspace, size_t workspace_bytes, void *cuda_stream);

/* dm_denoise_step with the timestep-conditioned block of App. A.1 in every layer (see dm_block_cfg):
 *     r_0 = E[tokens];  r_{l+1} = Block_l(r_l, tau);  logits = W_vocab RMSNorm(r_N) * final_norm_w.
 * block_weights: HOST array of cfg->n_layers entries (device pointers inside); weights->layers[l].norm_w
 * is not used.  tau: [B, d_cond] fp32 on the device, the timestep embedding of each sequence (the output
 * of the paper's timestep MLP, computed by the caller).  Everything else as in dm_denoise_step, block
 * mode included; the workspace size comes from dm_denoise_cond_workspace_bytes. */
int dm_denoise_cond_workspace_bytes(const dm_stack_cfg *cfg, const dm_block_cfg *blk, size_t *bytes);
int dm_denoise_step_cond(const dm_stack_cfg *cfg, const dm_block_cfg *blk, const dm_stack_weights *weights,
                         const dm_block_weights *block_weights, const int32_t *tokens, const float *tau,
                         void *logits, int32_t *argmax_out, const dm_layer_state *states,
                         void *workspace, size_t workspace_bytes, void *cuda_stream);

/* One reverse step of the masked diffusion, Sec. 2 Eq. 3, from noise level t to s < t: the denoiser runs on
 * tokens_in (as dm_denoise_step when blk == NULL, else as dm_denoise_step_cond), then every position
 *   - that is not mask_id keeps its token;
 *   - that is masked stays masked when u_keep[pos] < keep_prob (= s / t);
 *   - otherwise receives the inverse-CDF draw at u_cat[pos] from softmax(logits[pos, 0..vocab_real)) with mask_id
 *     excluded (the model never predicts the mask token): the first v whose cumulative probability exceeds
 *     u_cat[pos].  Both uniforms are in [0, 1) and come from the caller, so the step is a function of its inputs.
 * Only the drawn positions go through the vocabulary projection (their number is never brought to the host), and
 * the logits are not stored.  tokens_in, tokens_out [B, L] int32 (different buffers); u_keep, u_cat [B, L] fp32;
 * all on the device.  The probabilities are accumulated in fp32 in vocabulary order; a draw whose u_cat falls
 * within rounding distance of a boundary of the cumulative distribution may land on either neighbour. */
typedef struct {
    int32_t mask_id;      /* id of [MASK], < vocab */
    int32_t vocab_real;   /* ids [0, vocab_real) can be drawn; rows of w_vocab beyond are padding */
    float   keep_prob;    /* s / t of this step, in [0, 1] */
} dm_sample_cfg;
int dm_denoise_sample_workspace_bytes(const dm_stack_cfg *cfg, const dm_block_cfg *blk, size_t *bytes);
int dm_denoise_sample_step(const dm_stack_cfg *cfg, const dm_block_cfg *blk, const dm_stack_weights *weights,
                           const dm_block_weights *block_weights, const int32_t *tokens_in, const float *tau,
                           const dm_sample_cfg *sample, const float *u_keep, const float *u_cat,
                           int32_t *tokens_out, const dm_layer_state *states,
                           void *workspace, size_t workspace_bytes, void *cuda_stream);

/* A whole generation, Sec. 2 Eq. 3 with Sec. 4.3's step count (K = L / p denoising steps for p tokens per step): K
 * reverse steps along the noise levels t_k = 1 - (1 - t_eps) k / K (k = 0..K; App. A.1's sampling eps is 1e-3), step k
 * being dm_denoise_sample_step with keep_prob = (float)(t_{k+1} / t_k) computed in double, followed by one clean-up
 * pass with keep_prob = 0 that draws every position still masked at noise level t_eps: K + 1 denoiser evaluations, all
 * enqueued on `cuda_stream` by this one call, nothing read back to the host in between (the number of positions a
 * step draws stays on the device), so the call can be recorded into a CUDA graph and replayed.
 *   tokens_in  [B, L] int32: the start (all mask_id for unconditional generation; unmasked positions are a prompt and
 *              are never changed).   tokens_out [B, L] int32, a different buffer: the result, free of mask_id.
 *   u_keep, u_cat [K + 1, B, L] fp32 in [0, 1): the uniforms of every step (the caller's generator), see
 *              dm_denoise_sample_step.   tau [K + 1, B, d_cond] fp32: the timestep embedding of every step's t_k, only
 *              with blk != NULL (the timestep MLP is the caller's), else NULL.
 *   trace      [K + 1, B, L] int32 or NULL: when given, the tokens after every step (trace[K] equals tokens_out).
 * Workspace: dm_generate_workspace_bytes. */
typedef struct {
    int32_t steps;        /* K >= 1 */
    float   t_eps;        /* in (0, 1) */
    int32_t mask_id;      /* as dm_sample_cfg */
    int32_t vocab_real;
} dm_generate_cfg;
int dm_generate_workspace_bytes(const dm_stack_cfg *cfg, const dm_block_cfg *blk, size_t *bytes);
int dm_generate(const dm_stack_cfg *cfg, const dm_block_cfg *blk, const dm_stack_weights *weights,
                const dm_block_weights *block_weights, const dm_generate_cfg *gen, const int32_t *tokens_in,
                const float *tau, const float *u_keep, const float *u_cat, int32_t *tokens_out, int32_t *trace,
                void *workspace, size_t workspace_bytes, void *cuda_stream);

/* The attention mixer of the hybrid variant, Sec. 3.3 (one attention mixer every N mixer blocks): full
 * (bidirectional, unmasked) multi-head self-attention over each sequence, no position encoding,
 *     y = concat_h softmax(Q_h K_h^T / sqrt(d_h)) V_h  W_o^T,   [Q | K | V] = x W_qkv^T.
 * x, y [B, L, d_model] dtype (y != x); w_qkv [3 * d_model, d_model] with rows [Q | K | V], each split into
 * n_heads consecutive blocks of d_h = d_model / n_heads; w_o [d_model, d_model].  bf16 only, d_h = 64 or 80 (the
 * paper's 1.3B hybrid: 24 heads at d_model = 1920) only (DM_ERR_UNSUPPORTED otherwise).  The scores never leave the SM (running-maximum softmax over key tiles);
 * P is rounded to bf16 before P V, accumulation is fp32.  The hybrid stack (which layers are attention) is
 * dm_denoise_step_hybrid below. */
int dm_attention_workspace_bytes(int32_t batch, int32_t seqlen, int32_t d_model, int32_t dtype, size_t *bytes);
int dm_attention_forward(int32_t batch, int32_t seqlen, int32_t d_model, int32_t n_heads, int32_t dtype,
                         const void *w_qkv, const void *w_o, const void *x, void *y,
                         void *workspace, size_t workspace_bytes, void *cuda_stream);

/* The hybrid stack, Sec. 3.3 / App. A.3: layer l uses the attention mixer when l is a multiple of attn_period
 * (one attention mixer followed by attn_period - 1 bidirectional Mamba mixers; the paper fixes 5) and the
 * bidirectional Mamba mixer otherwise; attn_period = 0 means no attention layer.  Around either mixer the layer is
 * the RMSNorm pre-norm + residual of dm_denoise_step (blk == NULL) or the timestep-conditioned block of
 * dm_denoise_step_cond (blk, block_weights, tau given).  attn_weights: HOST array of cfg->n_layers entries, read
 * only where the layer is attention (the Mamba weights of those layers are not read).  Full-sequence mode; block
 * mode is dm_denoise_step_hybrid_block.  bf16, attention heads of width 64 or 80. */
typedef struct {
    int32_t attn_period;   /* N: layers 0, N, 2N, ... are attention; 0 = none */
    int32_t attn_heads;    /* d_model = 64 * attn_heads or 80 * attn_heads */
} dm_hybrid_cfg;
typedef struct {
    const void *w_qkv;     /* [3 * d_model, d_model] dtype, rows [Q | K | V] */
    const void *w_o;       /* [d_model, d_model] dtype */
} dm_attn_weights;
/* Key/value cache of one attention layer in block mode (Sec. 4.3): rows [0, len) hold the committed prefix.  A step
 * writes the block's keys and values to rows [len, len + G) -- whether or not the caller then commits them by
 * advancing len -- and its queries attend to rows [0, len + G), unmasked. */
typedef struct {
    void   *k_cache;   /* [B, cap, d_model] dtype */
    void   *v_cache;   /* [B, cap, d_model] dtype */
    int32_t len;       /* committed rows */
    int32_t cap;       /* rows allocated; len + G <= cap */
} dm_attn_state;
int dm_denoise_hybrid_workspace_bytes(const dm_stack_cfg *cfg, const dm_block_cfg *blk, size_t *bytes);
int dm_denoise_step_hybrid(const dm_stack_cfg *cfg, const dm_block_cfg *blk, const dm_hybrid_cfg *hybrid,
                           const dm_stack_weights *weights, const dm_block_weights *block_weights,
                           const dm_attn_weights *attn_weights, const int32_t *tokens, const float *tau,
                           void *logits, int32_t *argmax_out,
                           void *workspace, size_t workspace_bytes, void *cuda_stream);

/* dm_denoise_step_hybrid in block mode (Sec. 4.3): cfg->mixer.seqlen = G tokens of the active block per sequence;
 * `states` carries the Mamba layers' states as in dm_denoise_step, `attn_states` (HOST array of cfg->n_layers entries,
 * read where the layer is attention) the attention layers' key/value caches. */
int dm_denoise_step_hybrid_block(const dm_stack_cfg *cfg, const dm_block_cfg *blk, const dm_hybrid_cfg *hybrid,
                                 const dm_stack_weights *weights, const dm_block_weights *block_weights,
                                 const dm_attn_weights *attn_weights, const int32_t *tokens, const float *tau,
                                 void *logits, int32_t *argmax_out, const dm_layer_state *states,
                                 const dm_attn_state *attn_states,
                                 void *workspace, size_t workspace_bytes, void *cuda_stream);

/* dm_attention_forward for the active block of block-autoregressive decoding, with a key/value cache (dm_attn_state's
 * convention): the block's keys and values are written to rows [cache_len, cache_len + block_len) of the caches and
 * the block's queries attend to rows [0, cache_len + block_len).  Workspace as dm_attention_workspace_bytes(batch,
 * block_len, ...). */
int dm_attention_block_step(int32_t batch, int32_t block_len, int32_t d_model, int32_t n_heads, int32_t dtype,
                            const void *w_qkv, const void *w_o, const void *x_blk,
                            void *k_cache, void *v_cache, int32_t cache_len, int32_t cache_cap, void *y_blk,
                            void *workspace, size_t workspace_bytes, void *cuda_stream);

/* One dense projection as the mixer uses it (App. C counts 2mn FLOPs per token for a weight W in R^{m x n}):
 *     y[r, :] = row_scale[r] * (W x[r, :]) + addend[r, :]
 * x [rows, in_features] dtype; w [out_features, in_features] dtype; y [rows, out_features] of y_dtype
 * (DM_F32 or DM_BF16); row_scale [rows] fp32 or NULL (= 1); addend [rows, out_features] fp32 or NULL (= 0),
 * which may be y itself when y_dtype is DM_F32.  bf16 inputs run on the tensor cores when in_features is a
 * multiple of 8 and the pointers are 16-byte aligned, otherwise (and for fp32) on the CUDA cores. */
int dm_linear(int dtype, const void *x, const void *w, void *y, int y_dtype,
              int64_t rows, int32_t in_features, int32_t out_features,
              const float *row_scale, const float *addend, void *cuda_stream);

/* Same as dm_bimamba_forward, but x and y are HOST buffers (pageable or pinned; pinned lets the copies
 * overlap): the call copies x to the device, runs the mixer and copies y back, then synchronises
 * `cuda_stream`.  Batch rows are independent, so the batch is cut into up to 8 pieces of whole rows (about 4096 tokens or more each) and the
 * copy-in of the next piece and the copy-out of the previous one run on two internal streams (created on
 * the first call on a device) while the current piece is computed on `cuda_stream`; the work is ordered
 * after whatever was enqueued on `cuda_stream` before.  Calls on the same device must not overlap.
 * `workspace` must hold dm_bimamba_workspace_bytes + 2*B*L*d_model*sizeof(dtype) bytes. */
int dm_bimamba_forward_host(const dm_mixer_cfg *cfg, const dm_dir_weights w[2],
                            const void *x_host, void *y_host,
                            void *workspace, size_t workspace_bytes, void *cuda_stream);

/* The mixer without a caller workspace (the paper has no counterpart: this is a deployment aid).
 * For callers that cannot hand the library device memory of their own: code running where cudaMalloc is
 * not allowed or would stall the device (a serving loop that has given all free memory to its own pool, a
 * plug-in host that forbids allocation, a latency-critical path, since cudaMalloc synchronises the
 * device).  Same computation and arguments as dm_bimamba_forward, but every intermediate lives in a fixed
 * array of DM_STATIC_WORKSPACE_BYTES that is part of the library image: each GPU that loads the library
 * holds that much memory until the process exits.  The call allocates and frees nothing.
 *   - A configuration whose dm_bimamba_workspace_bytes exceeds DM_STATIC_WORKSPACE_BYTES is rejected
 *     with DM_ERR_WORKSPACE before anything is launched (use dm_bimamba_forward with your own buffer).
 *   - The first call on each device looks up the array's device address (with that device current);
 *     make that first call outside any stream capture.
 *   - All calls on a device share the one array and it keeps the previous call's contents.  Every call
 *     overwrites each region before reading it, so nothing needs clearing, but two calls whose kernels
 *     can overlap on the GPU (different streams, no dependency between them) race on it: serialise them. */
#define DM_STATIC_WORKSPACE_BYTES ((size_t)32 << 20)
int dm_bimamba_forward_static(const dm_mixer_cfg *cfg, const dm_dir_weights w[2],
                              const void *x, void *y, void *cuda_stream);

/* Self-test of the bounded device-side waits (no counterpart in the paper).  Every hand-off inside the pipelined kernels
 * is a wait with a time limit; when one runs out, the CTA stores DM_ERR_TIMEOUT in the device status word, its other
 * roles leave through an abort flag, and TMEM is freed before the CTA returns.  This call launches one small CTA that
 * goes through exactly that sequence on purpose: one warp waits, for limit_us microseconds, on a barrier nothing arrives
 * at; a second warp, holding TMEM columns, waits on another such barrier and must be released by the first one's abort.
 * Nothing faults or hangs.  Afterwards dm_check(cuda_stream) returns DM_ERR_TIMEOUT once (and clears it), and
 * out[0..2] (DEVICE, 3 x uint64) hold: 1 if the first wait gave up, 1 if the second was released by the abort flag,
 * and the nanoseconds the second one waited. */
int dm_selftest_wait_timeout(uint32_t limit_us, uint64_t *out, void *cuda_stream);

/* Self-test switch for the same failure path inside the tensor-core scan (no counterpart in the paper).  While on, a mixer call
 * whose scan would do its prep work inside the scan launch (one long sequence: fewer scan CTAs than SMs, more than eight chunks)
 * launches the scan without the CTAs of that role: the flags its load warps wait for from the ninth chunk on are never raised,
 * the waits run out after their regular limit (2 s), and every role of every CTA has to leave through the abort path -- loads in
 * flight waited for, TMEM freed.  The call itself returns DM_OK; dm_check then reports DM_ERR_TIMEOUT; y is unspecified.  Nothing
 * faults or hangs.  Process-wide; switch it off again. */
int dm_selftest_withhold_prep(int on);

/* Number of kernels this library has launched from this process since load (for benchmarks). */
uint64_t dm_kernel_launch_count(void);

/* Measurement aid (no counterpart in the paper).  While enabled, every mixer call records CUDA event
 * pairs on its stream around its three stages: in_proj (one span per direction), the fused
 * conv+scan+gate launch, out_proj (one span per direction).  dm_profile_read waits for the recorded
 * events, writes the summed device time in milliseconds and the number of spans per stage into the HOST
 * arrays ms[DM_STAGE_COUNT], spans[DM_STAGE_COUNT], and forgets them.  Not for use during stream capture. */
enum { DM_STAGE_IN_PROJ = 0, DM_STAGE_SCAN = 1, DM_STAGE_OUT_PROJ = 2, DM_STAGE_COUNT = 3 };
int dm_profile_enable(int on);
int dm_profile_read(float *ms, uint64_t *spans);

#ifdef __cplusplus
}
#endif
#endif /* DM_BIMAMBA_H_ */
