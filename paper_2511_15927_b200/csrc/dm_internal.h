// Internal declarations shared by the translation units of libdm_bimamba.so (not part of the ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "dm_bimamba.h"

namespace dm {

// Every kernel launch goes through this counter (dm_kernel_launch_count()).
void count_launch(int n = 1);

// Device status word written by kernels whose bounded waits expire; read and cleared by dm_check().
int *device_status_ptr();

inline size_t dtype_size(int dtype) { return dtype == DM_BF16 ? 2 : 4; }
inline size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }

// ---------------------------------------------------------------------------------------------
// GEMM:  C[m, n] = row_scale[m] * sum_k A[m, k] * B[n, k]  +  addend[m, n]
// A [M, K] (lda), B [N, K] (ldb): in_dtype.  C [M, N] (ldc): c_dtype.  row_scale [M] fp32 or NULL.
// addend [M, N] (ld_add) fp32 or NULL; it may alias C when c_dtype is DM_F32 and ldc == ld_add.
// ---------------------------------------------------------------------------------------------
struct GemmArgs {
    const void *A; int64_t lda;
    const void *B; int64_t ldb;
    void *C; int64_t ldc;
    int in_dtype, c_dtype;
    int M, N, K;
    const float *row_scale;
    const float *addend; int64_t ld_add;
    int silu_cols;           // output columns [0, silu_cols) get SiLU applied (0 = none)
    // Epilogue order: v = acc * row_scale[r] + col_bias[c];  v = act(v);  v *= col_scale[(r / cs_rows) * ld_cs + c];  v += addend[r, c]
    const float *col_bias;   // [N] or NULL
    int gelu;                // GELU (tanh form) on every output column
    const float *col_scale;  // [ceil(M / cs_rows), ld_cs] or NULL: one scale vector per group of cs_rows consecutive rows
    int cs_rows;
    int64_t ld_cs;           // row pitch of col_scale (0 = N)
    const int *m_dev;        // device int or NULL: only rows [0, clamp(*m_dev - m_off, 0, M)) are computed (row count known on the device only)
    int m_off;
};
cudaError_t gemm_simple(const GemmArgs &a, cudaStream_t s);
// Tensor-core path (tcgen05 + TMEM + TMA).  Returns cudaErrorNotSupported for shapes it does not take.
cudaError_t gemm_tcgen05(const GemmArgs &a, cudaStream_t s);
bool gemm_tcgen05_supports(const GemmArgs &a);
// Two problems of equal M, N, K and output type in one launch (same tile loop, one tail round).  The problems must be independent
// of each other: neither reads what the other writes.
bool gemm_tcgen05_pair_supports(const GemmArgs &a, const GemmArgs &b);
cudaError_t gemm_tcgen05_pair(const GemmArgs &a, const GemmArgs &b, cudaStream_t s);
// The same pair with each product cut in two along K (fp32 outputs only): the first half of a's product goes to a.C (with its addend and bias),
// the second half to a_hi (same pitch), likewise b; the caller adds the halves.  _pays: the shapes for which that fills the GPU better.
bool gemm_tcgen05_pair_splitk_pays(const GemmArgs &a, const GemmArgs &b);
cudaError_t gemm_tcgen05_pair_splitk(const GemmArgs &a, const GemmArgs &b, float *a_hi, float *b_hi, cudaStream_t s);

// ---------------------------------------------------------------------------------------------
// Fused conv + SiLU + discretisation + selective scan + gate, both directions in one launch.
// ---------------------------------------------------------------------------------------------
struct ScanDir {
    const void *conv_w, *conv_b, *norm_w;
    const float *dt_bias, *A_log, *D;
};
struct ScanArgs {
    int B, L, d_inner, H, P, N, k;
    int d_in_proj;           // row pitch of zx in elements (>= 2 d_inner + 2 N + H; the columns beyond are padding)
    int conv_ch;
    int dtype, flags, dir_mask, chunk;
    const void *zx;          // [2][B*L][d_in_proj] dtype: in_proj output of each direction
    int zx_tied;             // both directions read zx[0] (shared in_proj, DM_FLAG_TIED_PROJ)
    int z_gated;             // the z columns of zx already hold SiLU(z) (applied by the in_proj epilogue); the tensor-core scan requires it
    void *g;                 // [2][B*L][d_inner]   dtype: gated output (times norm_w when the norm is on)
    float *ssq;              // [2][B*L][H] per-head sum of squares of the gated output (norm on), or NULL
    ScanDir dir[2];
    const float *ssm_in;     // [B,H,P,N] or NULL   (left-to-right direction only)
    const void *conv_in;     // [B,k-1,conv_ch] or NULL
    float *ssm_out;          // [B,H,P,N] or NULL
};
size_t scan_seq_workspace_bytes(const ScanArgs &a);
cudaError_t scan_sequential(const ScanArgs &a, void *ws, cudaStream_t s);
bool scan_ssd_supports(const ScanArgs &a);
// chunk values the chunked bf16 path takes (0 = default, 32 = CUDA-core kernel, 128 = tensor-core kernel); other paths take any chunk > 0
bool scan_ssd_chunk_ok(int dtype, int d_state, int chunk);
void scan_ssd_selftest_withhold(int on);
size_t scan_ssd_workspace_bytes(const ScanArgs &a);
cudaError_t scan_ssd(const ScanArgs &a, void *ws, cudaStream_t s);

// Bidirectional multi-head attention over qkv [B*L, 3 d] (columns [Q | K | V], heads contiguous inside each) -> out [B*L, d];
// bf16, head width 64.
bool attention_supports(int dtype, int d, int n_heads);
// k_cache != NULL: block mode -- the block's K, V are appended at rows [cache_len, cache_len + L) of the caches [B, cache_cap, d]
// and the queries attend to the first cache_len + L rows.
cudaError_t attention_forward(const void *qkv, void *out, int B, int L, int d, int n_heads, void *k_cache, void *v_cache,
                              int cache_len, int cache_cap, cudaStream_t s);

// ---------------------------------------------------------------------------------------------
// Small row-wise kernels
// ---------------------------------------------------------------------------------------------
// rstd[dir][t] = rsqrt(sum_h ssq[dir][t][h] / d_inner + eps)
cudaError_t rstd_from_ssq(const float *ssq, float *rstd, int rows, int H, int d_inner, float eps, cudaStream_t s);
// r[t, :] = embed[tokens[t], :]  (fp32 residual stream)
cudaError_t embed_gather(const void *embed, int dtype, const int32_t *tokens, float *r, int T, int d, int vocab, cudaStream_t s);
// u[t, :] = r[t, :] * rsqrt(mean(r[t]^2) + eps) * w
cudaError_t rmsnorm_rows(const float *r, const void *w, void *u, int dtype, int T, int d, float eps, cudaStream_t s);
// u[t, :] = gamma[t / L, :] * (r[t, :] - mean) / sqrt(var + eps) + beta[t / L, :]   (gamma, beta: rows of pitch ld_mod)
cudaError_t adaln_rows(const float *r, const float *gamma, const float *beta, int64_t ld_mod, void *u, int dtype, int T, int L, int d,
                       float eps, cudaStream_t s);
// mod[b, :] = b_cond + W_cond tau[b, :]   (W_cond [n_out, d_c] dtype, b_cond [n_out] fp32 or NULL, tau [B, d_c] fp32)
cudaError_t modulation_rows(const float *tau, const void *w_cond, const float *b_cond, float *mod, int dtype, int B, int n_out, int d_c,
                            cudaStream_t s);
// Reverse step (Sec. 2, Eq. 3): tokens_out = tokens_in; idx[0..*count) = positions drawn this step (masked and u_keep >= keep_prob)
cudaError_t select_drawn(const int32_t *tokens_in, const float *u_keep, float keep_prob, int mask_id, int32_t *tokens_out, int32_t *idx,
                         int *count, int T, cudaStream_t s);
// dst[j, :] = src[idx[j], :] for j < *count
cudaError_t gather_rows(const void *src, const int32_t *idx, const int *count, void *dst, int dtype, int T, int d, cudaStream_t s);
// tokens_out[idx[row0 + r]] = inverse-CDF draw at u_cat from softmax(logits[r, 0..vocab_real) without mask_id), r < rows, row0 + r < *count
cudaError_t draw_rows(const void *logits, int64_t ld, int dtype, const int32_t *idx, const int *count, int row0, int rows,
                      const float *u_cat, int mask_id, int vocab_real, int32_t *tokens_out, cudaStream_t s);
// out[t] = argmax_v logits[t, v], lowest index on ties
cudaError_t argmax_rows(const void *logits, int dtype, int32_t *out, int T, int V, cudaStream_t s);
// y[i] = (dtype) (a[i] + b[i])
// y[t, :] = addend[t, :] + s0[t] (p0[t, :] + q0[t, :]) + s1[t] (p1[t, :] + q1[t, :])  (q0, q1: second halves of a product split along K, or NULL) with s_dir[t] = rsqrt(sum_h ssq_dir[t, h] / d_inner + eps_g) (1 when ssq_dir is NULL);
// u != NULL: also u[t, :] = w * y[t, :] * rsqrt(mean(y[t, :]^2) + eps).  One block per token; sum_partials_norm_supports(d) says whether d fits.
bool sum_partials_norm_supports(int d);
cudaError_t sum_partials_norm(const float *p0, const float *p1, const float *q0, const float *q1, const float *ssq0, const float *ssq1, int H, int d_inner, float eps_g,
                              const float *addend, int64_t ld_add, void *y, int y_dtype, const void *w, void *u, int u_dtype, int64_t T, int d,
                              float eps, cudaStream_t s);
// Tied projections: g0[t, :] = s0[t] * g0[t, :] + s1[t] * g1[t, :]  (s = rstd of each direction, or 1 when rstd is NULL), in place over g0
cudaError_t combine_directions(void *g0, const void *g1, const float *rstd0, const float *rstd1, int dtype, int64_t T, int d_inner, cudaStream_t s);
// conv_out[b] = last k-1 rows of concat(conv_in[b] (or zeros), xBC columns of zx[b, 0..L-1])
cudaError_t conv_state_update(const void *zx_fwd, const void *conv_in, void *conv_out, int dtype, int B, int L,
                              int k, int d_inner, int conv_ch, int d_in_proj, cudaStream_t s);

// One CTA whose waits run out by design (see selftest.cu); out: 3 x uint64 on the device
cudaError_t selftest_wait_timeout(unsigned long long limit_ns, unsigned long long *out, cudaStream_t s);

}  // namespace dm
