// Small row-wise kernels around the mixer: embedding gather, RMSNorm, the gated norm's rstd, arg-max
// over the vocabulary, the carried conv state.  All are bandwidth-trivial next to the GEMMs and the scan.
#include "dm_internal.h"

namespace dm {
namespace {

template <typename T> __device__ __forceinline__ float ldf(const T *p);
template <> __device__ __forceinline__ float ldf<float>(const float *p) { return *p; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void stf(T *p, float v);
template <> __device__ __forceinline__ void stf<float>(float *p, float v) { *p = v; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float block_sum(float v, float *red) {
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarp = blockDim.x >> 5;
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float t = 0.f;
    for (int i = 0; i < nwarp; ++i) t += red[i];      // same order in every thread: deterministic
    return t;
}

// One warp per row: the lanes read the row's per-head sums side by side, then reduce in a fixed order.
__global__ void rstd_kernel(const float *__restrict__ ssq, float *__restrict__ rstd, int rows, int H, float inv_n, float eps) {
    const int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (r >= rows) return;
    float s = 0.f;
    for (int h = lane; h < H; h += 32) s += ssq[(int64_t)r * H + h];
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    if (lane == 0) rstd[r] = rsqrtf(s * inv_n + eps);
}

template <typename T>
__global__ void embed_kernel(const T *__restrict__ embed, const int32_t *__restrict__ tokens, float *__restrict__ r, int d, int vocab) {
    const int64_t t = blockIdx.x;
    int id = tokens[t];
    id = id < 0 ? 0 : (id >= vocab ? vocab - 1 : id);      // ids are validated on the host side of the tests; clamp keeps reads in bounds
    for (int c = threadIdx.x; c < d; c += blockDim.x) r[t * d + c] = ldf(embed + (int64_t)id * d + c);
}

// The two row kernels below keep the token's channels in registers between the statistics and the output (one read
// of r): thread i holds channels 4 (i + 256 k) .. +3 for k < ROW_K, which covers d <= 4096; wider rows are re-read.
constexpr int ROW_THREADS = 256, ROW_K = 4;

template <typename T> __device__ __forceinline__ void st4(T *p, float a, float b, float c, float d);
template <> __device__ __forceinline__ void st4<float>(float *p, float a, float b, float c, float d) { *reinterpret_cast<float4 *>(p) = make_float4(a, b, c, d); }
template <> __device__ __forceinline__ void st4<__nv_bfloat16>(__nv_bfloat16 *p, float a, float b, float c, float d) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
    *reinterpret_cast<uint2 *>(p) = make_uint2(*reinterpret_cast<uint32_t *>(&lo), *reinterpret_cast<uint32_t *>(&hi));
}

template <typename T>
__global__ void __launch_bounds__(ROW_THREADS)
rmsnorm_kernel(const float *__restrict__ r, const T *__restrict__ w, T *__restrict__ u, int d, float eps) {
    __shared__ float red[32];
    const int64_t t = blockIdx.x;
    const float *row = r + t * d;
    const bool fast = (d & 3) == 0 && d <= 4 * ROW_THREADS * ROW_K;
    float4 v[ROW_K];
    float s = 0.f;
    if (fast) {
#pragma unroll
        for (int k = 0; k < ROW_K; ++k) {
            const int c = 4 * (threadIdx.x + ROW_THREADS * k);
            v[k] = c < d ? *reinterpret_cast<const float4 *>(row + c) : make_float4(0.f, 0.f, 0.f, 0.f);
            s = fmaf(v[k].x, v[k].x, s); s = fmaf(v[k].y, v[k].y, s); s = fmaf(v[k].z, v[k].z, s); s = fmaf(v[k].w, v[k].w, s);
        }
    } else {
        for (int c = threadIdx.x; c < d; c += blockDim.x) { const float x = row[c]; s = fmaf(x, x, s); }
    }
    s = block_sum(s, red);
    const float rs = rsqrtf(s / (float)d + eps);
    if (fast) {
#pragma unroll
        for (int k = 0; k < ROW_K; ++k) {
            const int c = 4 * (threadIdx.x + ROW_THREADS * k);
            if (c < d) st4(u + t * d + c, v[k].x * rs * ldf(w + c), v[k].y * rs * ldf(w + c + 1), v[k].z * rs * ldf(w + c + 2), v[k].w * rs * ldf(w + c + 3));
        }
    } else {
        for (int c = threadIdx.x; c < d; c += blockDim.x) stf(u + t * d + c, row[c] * rs * ldf(w + c));
    }
}

// u[t, :] = gamma[b, :] * (r[t, :] - mean) / sqrt(var + eps) + beta[b, :], b = t / L  (App. A.1, Eq. "AdaLN");
// gamma and beta are rows of the per-sequence modulation table (row pitch ld_mod).
template <typename T>
__global__ void __launch_bounds__(ROW_THREADS)
adaln_kernel(const float *__restrict__ r, const float *__restrict__ gamma, const float *__restrict__ beta, int64_t ld_mod,
             T *__restrict__ u, int L, int d, float eps) {
    __shared__ float red[32];
    const int64_t t = blockIdx.x, b = t / L;
    const float *row = r + t * d, *g = gamma + b * ld_mod, *be = beta + b * ld_mod;
    const bool fast = (d & 3) == 0 && d <= 4 * ROW_THREADS * ROW_K;
    float4 v[ROW_K];
    float s = 0.f;
    if (fast) {
#pragma unroll
        for (int k = 0; k < ROW_K; ++k) {
            const int c = 4 * (threadIdx.x + ROW_THREADS * k);
            v[k] = c < d ? *reinterpret_cast<const float4 *>(row + c) : make_float4(0.f, 0.f, 0.f, 0.f);
            s += (v[k].x + v[k].y) + (v[k].z + v[k].w);
        }
    } else {
        for (int c = threadIdx.x; c < d; c += blockDim.x) s += row[c];
    }
    const float mu = block_sum(s, red) / (float)d;
    float q = 0.f;
    if (fast) {
#pragma unroll
        for (int k = 0; k < ROW_K; ++k) {
            const int c = 4 * (threadIdx.x + ROW_THREADS * k);
            if (c < d) {
                const float a0 = v[k].x - mu, a1 = v[k].y - mu, a2 = v[k].z - mu, a3 = v[k].w - mu;
                q = fmaf(a0, a0, q); q = fmaf(a1, a1, q); q = fmaf(a2, a2, q); q = fmaf(a3, a3, q);
            }
        }
    } else {
        for (int c = threadIdx.x; c < d; c += blockDim.x) { const float x = row[c] - mu; q = fmaf(x, x, q); }
    }
    const float rs = rsqrtf(block_sum(q, red) / (float)d + eps);
    if (fast) {
#pragma unroll
        for (int k = 0; k < ROW_K; ++k) {
            const int c = 4 * (threadIdx.x + ROW_THREADS * k);
            if (c < d)
                st4(u + t * d + c, fmaf(g[c], (v[k].x - mu) * rs, be[c]), fmaf(g[c + 1], (v[k].y - mu) * rs, be[c + 1]),
                    fmaf(g[c + 2], (v[k].z - mu) * rs, be[c + 2]), fmaf(g[c + 3], (v[k].w - mu) * rs, be[c + 3]));
        }
    } else {
        for (int c = threadIdx.x; c < d; c += blockDim.x) stf(u + t * d + c, fmaf(g[c], (row[c] - mu) * rs, be[c]));
    }
}

// mod[b, j] = bias[j] + sum_c w[j, c] tau[b, c]: the modulation vectors of one layer (App. A.1: (gamma, beta) = W_cond tau).
// One warp per output element.
template <typename T>
__global__ void modulation_kernel(const float *__restrict__ tau, const T *__restrict__ w, const float *__restrict__ bias,
                                  float *__restrict__ mod, int n_out, int d_c) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31, b = blockIdx.y;
    if (warp >= n_out) return;
    float s = 0.f;
    for (int c = lane; c < d_c; c += 32) s = fmaf(ldf(w + (int64_t)warp * d_c + c), tau[(int64_t)b * d_c + c], s);
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    if (lane == 0) mod[(int64_t)b * n_out + warp] = s + (bias ? bias[warp] : 0.f);
}

template <typename T>
__global__ void argmax_kernel(const T *__restrict__ logits, int32_t *__restrict__ out, int V) {
    __shared__ float bv[32];
    __shared__ int bi[32];
    const int64_t t = blockIdx.x;
    float best = -INFINITY; int idx = 0x7fffffff;
    const T *row = logits + t * V;
    constexpr int PER = 16 / (int)sizeof(T);            // elements per 16-byte load
    if ((reinterpret_cast<uintptr_t>(row) & 15u) == 0) {
        const int nvec = V / PER;
        for (int i = threadIdx.x; i < nvec; i += blockDim.x) {
            const uint4 q = *reinterpret_cast<const uint4 *>(row + (int64_t)i * PER);
            const T *e = reinterpret_cast<const T *>(&q);
#pragma unroll
            for (int j = 0; j < PER; ++j) {                 // increasing v inside the thread: strict > keeps the lowest index
                const float x = ldf(e + j);
                if (x > best) { best = x; idx = i * PER + j; }
            }
        }
        for (int v = nvec * PER + threadIdx.x; v < V; v += blockDim.x) {
            const float x = ldf(row + v);
            if (x > best || (x == best && v < idx)) { best = x; idx = v; }
        }
    } else {
        for (int v = threadIdx.x; v < V; v += blockDim.x) {
            const float x = ldf(row + v);
            if (x > best || (x == best && v < idx)) { best = x; idx = v; }
        }
    }
    for (int off = 16; off > 0; off >>= 1) {
        const float ob = __shfl_xor_sync(0xffffffffu, best, off);
        const int oi = __shfl_xor_sync(0xffffffffu, idx, off);
        if (ob > best || (ob == best && oi < idx)) { best = ob; idx = oi; }
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarp = blockDim.x >> 5;
    if (lane == 0) { bv[warp] = best; bi[warp] = idx; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < nwarp; ++i)
            if (bv[i] > best || (bv[i] == best && bi[i] < idx)) { best = bv[i]; idx = bi[i]; }
        out[t] = idx == 0x7fffffff ? 0 : idx;
    }
}

// Row r (0..k-2) of the new conv state of batch row b is row L + r - (k-1) of the block when that is
// >= 0, otherwise row (k-1) + (L + r - (k-1)) of the old state (or zero).
template <typename T>
__global__ void conv_state_kernel(const T *__restrict__ zx, const T *__restrict__ conv_in, T *__restrict__ conv_out,
                                  int L, int k, int d_inner, int conv_ch, int d_in_proj) {
    const int b = blockIdx.y, r = blockIdx.z;
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= conv_ch) return;
    const int src = L + r - (k - 1);
    T v;
    if (src >= 0) v = zx[((int64_t)b * L + src) * d_in_proj + d_inner + c];
    else if (conv_in) v = conv_in[((int64_t)b * (k - 1) + (k - 1 + src)) * conv_ch + c];
    else { stf(&v, 0.f); }
    conv_out[((int64_t)b * (k - 1) + r) * conv_ch + c] = v;
}

// Short inputs (block decoding), one block of threads per token: the two directions' out_proj partials are summed with the gated norm's
// row scale of each direction applied here (the scale of a row commutes with the projection: Mamba(x) = s-> (g-> W->^T) + s<- (g<- W<-^T),
// Sec. 3.2), the residual is added, and -- when the caller's next step is an RMSNorm of the result -- that norm is applied to the row
// while it is still in registers.  ssq0/ssq1 = per-head sums of squares of the directions' gated outputs (NULL: no gated norm);
// q0, q1 = the second halves of the partials when the products were split along K (both or neither); addend may alias y; u = NULL: no norm.  Needs d % 4 == 0 and d <= 4 * ROW_THREADS * ROW_K.
template <typename TY, typename TU>
__global__ void __launch_bounds__(ROW_THREADS)
sum_partials_norm_kernel(const float *__restrict__ p0, const float *__restrict__ p1, const float *__restrict__ q0, const float *__restrict__ q1,
                         const float *__restrict__ ssq0, const float *__restrict__ ssq1,
                         int H, float inv_n, float eps_g, const float *addend, int64_t ld_add, TY *y, const TU *__restrict__ w, TU *__restrict__ u,
                         int d, float eps) {
    __shared__ float red[32];
    __shared__ float sc[2];
    const int64_t t = blockIdx.x;
    if (threadIdx.x < 64) {                      // warps 0 and 1: the two directions' scales, summed in the order of rstd_kernel
        const int dir = threadIdx.x >> 5, lane = threadIdx.x & 31;
        const float *q = dir ? ssq1 : ssq0;
        float v = 0.f;
        if (q) for (int h = lane; h < H; h += 32) v += q[t * H + h];
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
        if (lane == 0) sc[dir] = q ? rsqrtf(v * inv_n + eps_g) : 1.f;
    }
    __syncthreads();
    const float s0 = sc[0], s1 = sc[1];
    float4 v[ROW_K];
    float ss = 0.f;
#pragma unroll
    for (int k = 0; k < ROW_K; ++k) {
        const int c = 4 * (threadIdx.x + ROW_THREADS * k);
        v[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < d) {
            float4 a = __ldg(reinterpret_cast<const float4 *>(p0 + t * d + c)), b = __ldg(reinterpret_cast<const float4 *>(p1 + t * d + c));
            if (q0) {                            // products split along K: the second halves
                const float4 a2 = __ldg(reinterpret_cast<const float4 *>(q0 + t * d + c)), b2 = __ldg(reinterpret_cast<const float4 *>(q1 + t * d + c));
                a.x += a2.x; a.y += a2.y; a.z += a2.z; a.w += a2.w;
                b.x += b2.x; b.y += b2.y; b.z += b2.z; b.w += b2.w;
            }
            float4 r = addend ? *reinterpret_cast<const float4 *>(addend + t * ld_add + c) : make_float4(0.f, 0.f, 0.f, 0.f);
            r.x = fmaf(s1, b.x, fmaf(s0, a.x, r.x)); r.y = fmaf(s1, b.y, fmaf(s0, a.y, r.y));
            r.z = fmaf(s1, b.z, fmaf(s0, a.z, r.z)); r.w = fmaf(s1, b.w, fmaf(s0, a.w, r.w));
            st4(y + t * d + c, r.x, r.y, r.z, r.w);
            v[k] = r;
            ss = fmaf(r.x, r.x, ss); ss = fmaf(r.y, r.y, ss); ss = fmaf(r.z, r.z, ss); ss = fmaf(r.w, r.w, ss);
        }
    }
    if (!u) return;
    ss = block_sum(ss, red);
    const float rs = rsqrtf(ss / (float)d + eps);
#pragma unroll
    for (int k = 0; k < ROW_K; ++k) {
        const int c = 4 * (threadIdx.x + ROW_THREADS * k);
        if (c < d) st4(u + t * d + c, v[k].x * rs * ldf(w + c), v[k].y * rs * ldf(w + c + 1), v[k].z * rs * ldf(w + c + 2), v[k].w * rs * ldf(w + c + 3));
    }
}

// g0 <- s0 g0 + s1 g1, one block of threads per row (tied projections: the sum of the directions before the shared out_proj);
// 16-byte accesses when the rows allow it (VEC = elements per 16 bytes, or 1)
template <typename T, int VEC>
__global__ void __launch_bounds__(256) combine_kernel(T *__restrict__ g0, const T *__restrict__ g1, const float *__restrict__ r0,
                                                       const float *__restrict__ r1, int64_t rows, int d_inner) {
    for (int64_t t = blockIdx.x; t < rows; t += gridDim.x) {
        const float s0 = r0 ? r0[t] : 1.f, s1 = r1 ? r1[t] : 1.f;
        T *a = g0 + t * d_inner;
        const T *b = g1 + t * d_inner;
        for (int c = threadIdx.x * VEC; c < d_inner; c += blockDim.x * VEC) {
            if constexpr (VEC == 1) {
                stf(a + c, fmaf(s0, ldf(a + c), s1 * ldf(b + c)));
            } else {
                uint4 va = *reinterpret_cast<const uint4 *>(a + c);
                const uint4 vb = __ldg(reinterpret_cast<const uint4 *>(b + c));
                uint32_t *wa = reinterpret_cast<uint32_t *>(&va);
                const uint32_t *wb = reinterpret_cast<const uint32_t *>(&vb);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if constexpr (sizeof(T) == 2) {
                        const float lo = fmaf(s0, __uint_as_float(wa[e] << 16), s1 * __uint_as_float(wb[e] << 16));
                        const float hi = fmaf(s0, __uint_as_float(wa[e] & 0xFFFF0000u), s1 * __uint_as_float(wb[e] & 0xFFFF0000u));
                        const __nv_bfloat162 pk = __floats2bfloat162_rn(lo, hi);
                        wa[e] = *reinterpret_cast<const uint32_t *>(&pk);
                    } else {
                        wa[e] = __float_as_uint(fmaf(s0, __uint_as_float(wa[e]), s1 * __uint_as_float(wb[e])));
                    }
                }
                *reinterpret_cast<uint4 *>(a + c) = va;
            }
        }
    }
}

}  // namespace

cudaError_t rstd_from_ssq(const float *ssq, float *rstd, int rows, int H, int d_inner, float eps, cudaStream_t s) {
    rstd_kernel<<<(rows + 7) / 8, 256, 0, s>>>(ssq, rstd, rows, H, 1.f / (float)d_inner, eps);
    count_launch();
    return cudaGetLastError();
}

cudaError_t embed_gather(const void *embed, int dtype, const int32_t *tokens, float *r, int T, int d, int vocab, cudaStream_t s) {
    if (dtype == DM_BF16) embed_kernel<<<T, 256, 0, s>>>(static_cast<const __nv_bfloat16 *>(embed), tokens, r, d, vocab);
    else embed_kernel<<<T, 256, 0, s>>>(static_cast<const float *>(embed), tokens, r, d, vocab);
    count_launch();
    return cudaGetLastError();
}

cudaError_t rmsnorm_rows(const float *r, const void *w, void *u, int dtype, int T, int d, float eps, cudaStream_t s) {
    if (dtype == DM_BF16) rmsnorm_kernel<<<T, 256, 0, s>>>(r, static_cast<const __nv_bfloat16 *>(w), static_cast<__nv_bfloat16 *>(u), d, eps);
    else rmsnorm_kernel<<<T, 256, 0, s>>>(r, static_cast<const float *>(w), static_cast<float *>(u), d, eps);
    count_launch();
    return cudaGetLastError();
}

cudaError_t adaln_rows(const float *r, const float *gamma, const float *beta, int64_t ld_mod, void *u, int dtype, int T, int L, int d,
                       float eps, cudaStream_t s) {
    if (dtype == DM_BF16) adaln_kernel<<<T, 256, 0, s>>>(r, gamma, beta, ld_mod, static_cast<__nv_bfloat16 *>(u), L, d, eps);
    else adaln_kernel<<<T, 256, 0, s>>>(r, gamma, beta, ld_mod, static_cast<float *>(u), L, d, eps);
    count_launch();
    return cudaGetLastError();
}

cudaError_t modulation_rows(const float *tau, const void *w_cond, const float *b_cond, float *mod, int dtype, int B, int n_out, int d_c,
                            cudaStream_t s) {
    dim3 grid((n_out * 32 + 255) / 256, B);
    if (dtype == DM_BF16) modulation_kernel<<<grid, 256, 0, s>>>(tau, static_cast<const __nv_bfloat16 *>(w_cond), b_cond, mod, n_out, d_c);
    else modulation_kernel<<<grid, 256, 0, s>>>(tau, static_cast<const float *>(w_cond), b_cond, mod, n_out, d_c);
    count_launch();
    return cudaGetLastError();
}

cudaError_t argmax_rows(const void *logits, int dtype, int32_t *out, int T, int V, cudaStream_t s) {
    if (dtype == DM_BF16) argmax_kernel<<<T, 256, 0, s>>>(static_cast<const __nv_bfloat16 *>(logits), out, V);
    else argmax_kernel<<<T, 256, 0, s>>>(static_cast<const float *>(logits), out, V);
    count_launch();
    return cudaGetLastError();
}

cudaError_t conv_state_update(const void *zx_fwd, const void *conv_in, void *conv_out, int dtype, int B, int L,
                              int k, int d_inner, int conv_ch, int d_in_proj, cudaStream_t s) {
    dim3 grid((conv_ch + 255) / 256, B, k - 1);
    if (dtype == DM_BF16)
        conv_state_kernel<<<grid, 256, 0, s>>>(static_cast<const __nv_bfloat16 *>(zx_fwd), static_cast<const __nv_bfloat16 *>(conv_in),
                                               static_cast<__nv_bfloat16 *>(conv_out), L, k, d_inner, conv_ch, d_in_proj);
    else
        conv_state_kernel<<<grid, 256, 0, s>>>(static_cast<const float *>(zx_fwd), static_cast<const float *>(conv_in),
                                               static_cast<float *>(conv_out), L, k, d_inner, conv_ch, d_in_proj);
    count_launch();
    return cudaGetLastError();
}

bool sum_partials_norm_supports(int d) { return d % 4 == 0 && d <= 4 * ROW_THREADS * ROW_K; }

cudaError_t sum_partials_norm(const float *p0, const float *p1, const float *q0, const float *q1, const float *ssq0, const float *ssq1, int H, int d_inner, float eps_g,
                              const float *addend, int64_t ld_add, void *y, int y_dtype, const void *w, void *u, int u_dtype, int64_t T, int d,
                              float eps, cudaStream_t s) {
    if (!sum_partials_norm_supports(d) || (q0 == nullptr) != (q1 == nullptr)) return cudaErrorInvalidValue;
    const float inv_n = 1.f / (float)d_inner;
    const int grid = (int)T;
#define DM_SPN(TY, TU) sum_partials_norm_kernel<TY, TU><<<grid, ROW_THREADS, 0, s>>>(p0, p1, q0, q1, ssq0, ssq1, H, inv_n, eps_g, addend, ld_add, \
        static_cast<TY *>(y), static_cast<const TU *>(w), static_cast<TU *>(u), d, eps)
    if (y_dtype == DM_F32) { if (u_dtype == DM_BF16) DM_SPN(float, __nv_bfloat16); else DM_SPN(float, float); }
    else { if (u_dtype == DM_BF16) DM_SPN(__nv_bfloat16, __nv_bfloat16); else DM_SPN(__nv_bfloat16, float); }
#undef DM_SPN
    count_launch();
    return cudaGetLastError();
}

cudaError_t combine_directions(void *g0, const void *g1, const float *rstd0, const float *rstd1, int dtype, int64_t T, int d_inner, cudaStream_t s) {
    const int blocks = (int)(T < 148 * 8 ? T : 148 * 8);
    const size_t es = dtype_size(dtype);
    const bool vec = ((size_t)d_inner * es) % 16 == 0 && ((reinterpret_cast<uintptr_t>(g0) | reinterpret_cast<uintptr_t>(g1)) & 15u) == 0;
    if (dtype == DM_BF16) {
        auto *a = static_cast<__nv_bfloat16 *>(g0);
        auto *b = static_cast<const __nv_bfloat16 *>(g1);
        if (vec) combine_kernel<__nv_bfloat16, 8><<<blocks, 256, 0, s>>>(a, b, rstd0, rstd1, T, d_inner);
        else combine_kernel<__nv_bfloat16, 1><<<blocks, 256, 0, s>>>(a, b, rstd0, rstd1, T, d_inner);
    } else {
        auto *a = static_cast<float *>(g0);
        auto *b = static_cast<const float *>(g1);
        if (vec) combine_kernel<float, 4><<<blocks, 256, 0, s>>>(a, b, rstd0, rstd1, T, d_inner);
        else combine_kernel<float, 1><<<blocks, 256, 0, s>>>(a, b, rstd0, rstd1, T, d_inner);
    }
    count_launch();
    return cudaGetLastError();
}

}  // namespace dm
