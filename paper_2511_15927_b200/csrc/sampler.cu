// Reverse step of the masked diffusion (Sec. 2, Eq. 3) after the denoiser: which positions are drawn this step,
// their rows gathered for the vocabulary projection, and the draw itself from the projected logits.
//   - a position that is not [MASK] is carried over;
//   - a masked position stays masked iff u_keep < s/t;
//   - otherwise its token is the inverse-CDF sample at u_cat of softmax(logits) with the mask token (and any
//     vocabulary padding) excluded: the first v whose cumulative probability exceeds u_cat.
// Only the drawn positions go through the vocabulary projection; their number stays on the device (the GEMM and the
// kernels below read it there), so a step needs no host synchronisation.
#include "dm_internal.h"

namespace dm {
namespace {

template <typename T> __device__ __forceinline__ float ldv(const T *p);
template <> __device__ __forceinline__ float ldv<float>(const float *p) { return *p; }
template <> __device__ __forceinline__ float ldv<__nv_bfloat16>(const __nv_bfloat16 *p) { return __bfloat162float(*p); }

constexpr int SEL_THREADS = 1024;

// One block: tokens_out = tokens_in; idx[0..count) = the positions drawn this step, in increasing order; *count.
__global__ void __launch_bounds__(SEL_THREADS)
select_drawn_kernel(const int32_t *__restrict__ tokens_in, const float *__restrict__ u_keep, float keep_prob, int mask_id,
                    int32_t *__restrict__ tokens_out, int32_t *__restrict__ idx, int *__restrict__ count, int T) {
    __shared__ int part[SEL_THREADS];
    const int tid = threadIdx.x;
    const int per = (T + SEL_THREADS - 1) / SEL_THREADS, t0 = tid * per, t1 = min(T, t0 + per);
    int n = 0;
    for (int t = t0; t < t1; ++t) {
        const int tok = tokens_in[t];
        tokens_out[t] = tok;
        n += (tok == mask_id && !(u_keep[t] < keep_prob)) ? 1 : 0;
    }
    part[tid] = n;
    __syncthreads();
    for (int off = 1; off < SEL_THREADS; off <<= 1) {       // inclusive scan (integers: exact in any order)
        const int v = tid >= off ? part[tid - off] : 0;
        __syncthreads();
        part[tid] += v;
        __syncthreads();
    }
    int pos = part[tid] - n;
    for (int t = t0; t < t1; ++t)
        if (tokens_in[t] == mask_id && !(u_keep[t] < keep_prob)) idx[pos++] = t;
    if (tid == SEL_THREADS - 1) *count = part[tid];
}

// dst[j, :] = src[idx[j], :] for j < *count
template <typename T>
__global__ void gather_rows_kernel(const T *__restrict__ src, const int32_t *__restrict__ idx, const int *__restrict__ count,
                                   T *__restrict__ dst, int d) {
    const int j = blockIdx.x;
    if (j >= *count) return;
    const T *s = src + (int64_t)idx[j] * d;
    T *o = dst + (int64_t)j * d;
    for (int c = threadIdx.x; c < d; c += blockDim.x) o[c] = s[c];
}

constexpr int DRAW_THREADS = 256;

__device__ __forceinline__ float block_reduce(float v, float *red, bool is_max) {
    for (int off = 16; off > 0; off >>= 1) {
        const float o = __shfl_xor_sync(0xffffffffu, v, off);
        v = is_max ? fmaxf(v, o) : v + o;
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float t = red[0];
    for (int i = 1; i < DRAW_THREADS / 32; ++i) t = is_max ? fmaxf(t, red[i]) : t + red[i];
    return t;
}

// One block per drawn row of the chunk: row r of `logits` belongs to position idx[row0 + r].  Each thread owns one
// contiguous segment of the vocabulary, so that the cumulative sums run in vocabulary order.
template <typename T>
__global__ void __launch_bounds__(DRAW_THREADS)
draw_rows_kernel(const T *__restrict__ logits, int64_t ld, const int32_t *__restrict__ idx, const int *__restrict__ count, int row0,
                 const float *__restrict__ u_cat, int mask_id, int vocab_real, int32_t *__restrict__ tokens_out) {
    __shared__ float red[DRAW_THREADS / 32];
    __shared__ float seg[DRAW_THREADS];
    __shared__ int chosen;
    const int r = blockIdx.x;
    if (row0 + r >= *count) return;
    const int pos = idx[row0 + r];
    const T *z = logits + (int64_t)r * ld;
    const int tid = threadIdx.x;
    const int per = (vocab_real + DRAW_THREADS - 1) / DRAW_THREADS, v0 = min(vocab_real, tid * per), v1 = min(vocab_real, v0 + per);
    float m = -INFINITY;
    for (int v = v0; v < v1; ++v) if (v != mask_id) m = fmaxf(m, ldv(z + v));
    m = block_reduce(m, red, true);
    float s = 0.f;
    for (int v = v0; v < v1; ++v) if (v != mask_id) s += __expf(ldv(z + v) - m);
    seg[tid] = s;
    if (tid == 0) chosen = -1;
    __syncthreads();
    // the segment sums in order (256 of them: one thread adds them up and finds the segment that contains the target)
    __shared__ float before;     // mass before the chosen segment
    __shared__ float target_s;
    if (tid == 0) {
        float total = 0.f;
        for (int i = 0; i < DRAW_THREADS; ++i) total += seg[i];
        const float target = u_cat[pos] * total;
        float acc = 0.f;
        int k = 0;
        for (; k < DRAW_THREADS - 1; ++k) {
            if (acc + seg[k] > target) break;
            acc += seg[k];
        }
        // k is the first segment whose cumulative mass exceeds the target (or the last one); skip back over empty tails
        while (k > 0 && seg[k] == 0.f) --k;
        chosen = k; before = acc; target_s = target;
    }
    __syncthreads();
    if (tid == chosen) {
        float acc = before;
        int pick = -1, last = -1;
        for (int v = v0; v < v1; ++v) {
            if (v == mask_id) continue;
            const float p = __expf(ldv(z + v) - m);
            if (p > 0.f) last = v;
            acc += p;
            if (acc > target_s && p > 0.f) { pick = v; break; }
        }
        tokens_out[pos] = pick >= 0 ? pick : last;          // rounding at the very end of the range: the last token with mass
    }
}

}  // namespace

cudaError_t select_drawn(const int32_t *tokens_in, const float *u_keep, float keep_prob, int mask_id, int32_t *tokens_out, int32_t *idx,
                         int *count, int T, cudaStream_t s) {
    select_drawn_kernel<<<1, SEL_THREADS, 0, s>>>(tokens_in, u_keep, keep_prob, mask_id, tokens_out, idx, count, T);
    count_launch();
    return cudaGetLastError();
}

cudaError_t gather_rows(const void *src, const int32_t *idx, const int *count, void *dst, int dtype, int T, int d, cudaStream_t s) {
    if (dtype == DM_BF16) gather_rows_kernel<<<T, 128, 0, s>>>(static_cast<const __nv_bfloat16 *>(src), idx, count, static_cast<__nv_bfloat16 *>(dst), d);
    else gather_rows_kernel<<<T, 128, 0, s>>>(static_cast<const float *>(src), idx, count, static_cast<float *>(dst), d);
    count_launch();
    return cudaGetLastError();
}

cudaError_t draw_rows(const void *logits, int64_t ld, int dtype, const int32_t *idx, const int *count, int row0, int rows,
                      const float *u_cat, int mask_id, int vocab_real, int32_t *tokens_out, cudaStream_t s) {
    if (dtype == DM_BF16)
        draw_rows_kernel<<<rows, DRAW_THREADS, 0, s>>>(static_cast<const __nv_bfloat16 *>(logits), ld, idx, count, row0, u_cat, mask_id, vocab_real, tokens_out);
    else
        draw_rows_kernel<<<rows, DRAW_THREADS, 0, s>>>(static_cast<const float *>(logits), ld, idx, count, row0, u_cat, mask_id, vocab_real, tokens_out);
    count_launch();
    return cudaGetLastError();
}

}  // namespace dm
