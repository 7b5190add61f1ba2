// Fused depthwise conv + SiLU, discretisation, selective scan and gate on the CUDA cores, both
// directions in one launch.  One CTA owns one (batch row, direction, head) and walks the sequence in
// logical time (left-to-right for the forward layer, right-to-left for the reverse layer: the reverse
// layer is the same operator on the reversed sequence, done here by index arithmetic only).
//
// The CTA is split in two groups that work on different chunks of TC tokens at the same time:
//   scan threads (the first P * LPC):  the state h[p][n] of the head lives in their registers: channel p is served
//       by LPC adjacent lanes, each holding N / LPC states; the C-contraction is finished with warp shuffles.  They
//       run the token loop of chunk i from shared memory and leave y_t = h_t C_t + D x_t there.
//   loader threads (the last 128):  meanwhile they write chunk i-1's gated output (g = y SiLU(z) [* norm_w], per-head
//       sum of squares) and prepare chunk i+1: conv + SiLU of this head's x channels with one global load per output
//       (a sliding window along time per channel), B' and C' copied from scratch, z, Delta and the decay.
// One __syncthreads per chunk hands the buffers over.  The first chunk is prepared, and the last one finished, by all
// threads.  B' and C' (conv + SiLU of the B and C columns, shared by all heads) come from a small launch of their own.
//
// This is the exact (fp32) form of the recurrence: the kernel for fp32 I/O (whose 1e-4 tolerance rules out bf16
// products) and for d_state above 128; bf16 I/O with d_state <= 128 runs the chunked kernels of scan_ssd.cu, block
// decoding with carried state included.
#include "dm_internal.h"

namespace dm {
namespace {

constexpr int NL = 128;            // loader threads
constexpr int NSEG = 4;            // time segments per conv channel (parallelism of the sliding windows)

template <typename T> __device__ __forceinline__ float ldf(const T *p);
template <> __device__ __forceinline__ float ldf<float>(const float *p) { return __ldg(p); }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16 *p) {
    return __bfloat162float(*p);
}
template <typename T> __device__ __forceinline__ void stf(T *p, float v);
template <> __device__ __forceinline__ void stf<float>(float *p, float v) { *p = v; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

// 16 bytes of T -> floats (VEC = 16 / sizeof(T) elements)
template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int VEC = 4;
    static __device__ __forceinline__ void load(const float *p, float *o) {
        const float4 v = __ldg(reinterpret_cast<const float4 *>(p));
        o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
    }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int VEC = 8;
    static __device__ __forceinline__ void load(const __nv_bfloat16 *p, float *o) {
        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(p));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) { o[2 * i] = __uint_as_float(w[i] << 16); o[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u); }
    }
};

__device__ __forceinline__ float silu_f(float v) { return __fdividef(v, 1.f + __expf(-v)); }     // ~1e-6 relative: inside the fp32 tolerance
__device__ __forceinline__ float softplus_f(float v) { return fmaxf(v, 0.f) + log1pf(expf(-fabsf(v))); }

// B' and C' of every token: conv + SiLU of the 2N shared columns, in logical time order semantics (the reverse layer
// looks at later rows), fp32, layout [dir][B*L][2N].  Thread = one column of one run of `rows` consecutive tokens.
template <typename T>
__global__ void __launch_bounds__(256)
bc_prep_kernel(const ScanArgs a, const int dir0, float *__restrict__ bc, const int rows) {
    const int N2 = 2 * a.N, L = a.L, k = a.k;
    const int dir = dir0 + blockIdx.z, b = blockIdx.y;
    const bool rev = dir == 1;
    const ScanDir &w = a.dir[dir];
    const int64_t T_all = (int64_t)a.B * L;
    const T *zx = static_cast<const T *>(a.zx) + ((int64_t)(a.zx_tied ? 0 : dir) * T_all + (int64_t)b * L) * a.d_in_proj;
    const T *conv_in = (!rev && a.conv_in) ? static_cast<const T *>(a.conv_in) + (int64_t)b * (k - 1) * a.conv_ch : nullptr;
    float *out = bc + ((int64_t)dir * T_all + (int64_t)b * L) * N2;
    const bool has_bias = (a.flags & DM_FLAG_CONV_BIAS) && w.conv_b != nullptr;
    const int tau0 = blockIdx.x * rows;
    for (int col = threadIdx.x; col < N2; col += blockDim.x) {
        const int cc = a.d_inner + col;
        auto raw = [&](int tau) -> float {
            if (tau >= L) return 0.f;
            if (tau >= 0) return ldf(zx + (int64_t)(rev ? L - 1 - tau : tau) * a.d_in_proj + a.d_inner + cc);
            return conv_in ? ldf(conv_in + (int64_t)(k - 1 + tau) * a.conv_ch + cc) : 0.f;
        };
        float wl[4];
#pragma unroll
        for (int m = 0; m < 4; ++m) wl[m] = m < k ? ldf(static_cast<const T *>(w.conv_w) + (int64_t)cc * k + (k - 1 - m)) : 0.f;
        const float bias = has_bias ? ldf(static_cast<const T *>(w.conv_b) + cc) : 0.f;
        float h1 = raw(tau0 - 1), h2 = k > 2 ? raw(tau0 - 2) : 0.f, h3 = k > 3 ? raw(tau0 - 3) : 0.f;
#pragma unroll 4
        for (int i = 0; i < rows; ++i) {
            const int tau = tau0 + i;
            if (tau >= L) break;
            const float cur = raw(tau);
            float v = bias;
            v = fmaf(wl[3], h3, v); v = fmaf(wl[2], h2, v); v = fmaf(wl[1], h1, v); v = fmaf(wl[0], cur, v);
            out[(int64_t)(rev ? L - 1 - tau : tau) * N2 + col] = silu_f(v);
            h3 = h2; h2 = h1; h1 = cur;
        }
    }
}

// NQ = float4 groups of state per lane (N / LPC / 4): 4 for N <= 128, 8 for N = 256.
template <typename T, int NQ>
__global__ void __launch_bounds__(512 + NL)
scan_seq_kernel(const ScanArgs a, const int dir0, const int TC, const int LPC, const float *__restrict__ bc_all) {
    extern __shared__ __align__(16) float smem[];
    const int P = a.P, N = a.N, L = a.L, k = a.k;
    const int NS = P * LPC;                            // scan threads
    const int h = blockIdx.x, b = blockIdx.z;
    const int dir = dir0 + blockIdx.y;                 // 0 = left-to-right, 1 = right-to-left
    const bool rev = dir == 1;
    const int tid = threadIdx.x;

    // two stages of { xs[TC][P] conv(x), zs[TC][P] z, Bs[TC][N], Cs[TC][N], dl[TC] Delta, da[TC] exp(Delta A) }, then ys[2][TC][P],
    // then xr[(TC+3)][P]: the pre-conv x rows of the chunk being prepared (3 rows of history first)
    const int stage_floats = TC * (2 * P + 2 * N + 2);
    float *ys_all = smem + 2 * stage_floats;
    float *xr = ys_all + 2 * TC * P;
    constexpr int VEC = Vec16<T>::VEC;
    // 16-byte loads need every row slice to start on a 16-byte boundary
    const bool vec_ok = ((a.d_in_proj * (int)sizeof(T)) % 16 == 0) && (((int64_t)a.d_inner * sizeof(T)) % 16 == 0) &&
                        ((P * (int)sizeof(T)) % 16 == 0) && ((reinterpret_cast<uintptr_t>(a.zx) & 15u) == 0);
    auto xs_of = [&](int s) { return smem + s * stage_floats; };

    const ScanDir &w = a.dir[dir];
    const T *conv_w = static_cast<const T *>(w.conv_w);
    const T *conv_b = static_cast<const T *>(w.conv_b);
    const T *norm_w = static_cast<const T *>(w.norm_w);
    const bool has_bias = (a.flags & DM_FLAG_CONV_BIAS) && conv_b != nullptr;
    const bool norm_on = (a.flags & DM_FLAG_GATED_RMSNORM) != 0;

    const int64_t T_all = (int64_t)a.B * L;
    const T *zx = static_cast<const T *>(a.zx) + ((int64_t)(a.zx_tied ? 0 : dir) * T_all + (int64_t)b * L) * a.d_in_proj;
    T *gout = static_cast<T *>(a.g) + ((int64_t)dir * T_all + (int64_t)b * L) * a.d_inner;
    float *ssq = a.ssq ? a.ssq + ((int64_t)dir * T_all + (int64_t)b * L) * a.H : nullptr;
    const T *conv_in = (!rev && a.conv_in) ? static_cast<const T *>(a.conv_in) + (int64_t)b * (k - 1) * a.conv_ch : nullptr;
    const float *bc = bc_all + ((int64_t)dir * T_all + (int64_t)b * L) * (2 * N);
    const int nchunks = (L + TC - 1) / TC;
    const int nall = blockDim.x;

    const float Ah = -expf(w.A_log[h]);
    const float dtb = w.dt_bias[h];
    // pre-conv value of conv channel cc at logical time tau (tau < 0: carried rows or zeros)
    auto raw = [&](int tau, int cc) -> float {
        if (tau >= 0) {
            const int t = rev ? L - 1 - tau : tau;
            return ldf(zx + (int64_t)t * a.d_in_proj + a.d_inner + cc);
        }
        return (conv_in && k - 1 + tau >= 0) ? ldf(conv_in + (int64_t)(k - 1 + tau) * a.conv_ch + cc) : 0.f;
    };
    // everything the token loop of chunk ci reads, by threads lt = 0..nthr-1
    auto prepare = [&](int ci, int lt, int nthr) {
        const int s = ci & 1, tau0 = ci * TC, tc = min(TC, L - tau0);
        float *xs = xs_of(s), *zs = xs + TC * P, *Bs = zs + TC * P, *Cs = Bs + TC * N, *dl = Cs + TC * N, *da = dl + TC;
        // ---- phase 1: global -> shared with independent loads: pre-conv x rows (3 rows of history first), z, B', C'
        const int upr = P / VEC;                           // 16-byte units per row slice
        if (vec_ok) {
#pragma unroll 4
            for (int u = lt; u < (tc + 3) * upr; u += nthr) {
                const int r = u / upr, c = (u - r * upr) * VEC, tau = tau0 + r - 3;
                float o[VEC];
                if (tau >= 0) {
                    Vec16<T>::load(zx + (int64_t)(rev ? L - 1 - tau : tau) * a.d_in_proj + a.d_inner + h * P + c, o);
                } else {
#pragma unroll
                    for (int e = 0; e < VEC; ++e) o[e] = raw(tau, h * P + c + e);
                }
#pragma unroll
                for (int e = 0; e < VEC; ++e) xr[r * P + c + e] = o[e];
            }
#pragma unroll 4
            for (int u = lt; u < tc * upr; u += nthr) {
                const int i = u / upr, c = (u - i * upr) * VEC;
                const int t = rev ? L - 1 - (tau0 + i) : tau0 + i;
                float o[VEC];
                Vec16<T>::load(zx + (int64_t)t * a.d_in_proj + h * P + c, o);
#pragma unroll
                for (int e = 0; e < VEC; ++e) zs[i * P + c + e] = o[e];
            }
        } else {
            for (int e = lt; e < (tc + 3) * P; e += nthr) {
                const int r = e / P, c = e - r * P;
                xr[r * P + c] = raw(tau0 + r - 3, h * P + c);
            }
            for (int e = lt; e < tc * P; e += nthr) {
                const int i = e / P, c = e - i * P;
                const int t = rev ? L - 1 - (tau0 + i) : tau0 + i;
                zs[i * P + c] = ldf(zx + (int64_t)t * a.d_in_proj + h * P + c);
            }
        }
        const int n4 = N / 2;                              // float4 per token row of [B' | C']
#pragma unroll 4
        for (int e = lt; e < tc * n4; e += nthr) {
            const int i = e / n4, c4 = e - i * n4;
            const int t = rev ? L - 1 - (tau0 + i) : tau0 + i;
            const float4 v = __ldg(reinterpret_cast<const float4 *>(bc + (int64_t)t * 2 * N) + c4);
            float *dst = c4 * 4 < N ? Bs + i * N + c4 * 4 : Cs + i * N + (c4 * 4 - N);
            *reinterpret_cast<float4 *>(dst) = v;
        }
        if (nthr == nall) __syncthreads();
        else asm volatile("bar.sync 1, %0;" ::"n"(NL) : "memory");
        // ---- phase 2: conv + SiLU of this head's x channels from shared memory: task = (time segment, channel)
        const int seglen = (tc + NSEG - 1) / NSEG;
        for (int task = lt; task < NSEG * P; task += nthr) {
            const int seg = task / P, col = task - seg * P;
            const int i0 = seg * seglen, i1 = min(tc, i0 + seglen);
            if (i0 >= i1) continue;
            const int cc = h * P + col;
            float wl[4];                                   // wl[m] multiplies the row m steps back in time
#pragma unroll
            for (int m = 0; m < 4; ++m) wl[m] = m < k ? ldf(conv_w + (int64_t)cc * k + (k - 1 - m)) : 0.f;
            const float bias = has_bias ? ldf(conv_b + cc) : 0.f;
            const float *xc = xr + 3 * P + col;              // xc[i * P] = pre-conv value at chunk row i
            float h1 = xc[(i0 - 1) * P], h2 = xc[(i0 - 2) * P], h3 = xc[(i0 - 3) * P];
#pragma unroll 4
            for (int i = i0; i < i1; ++i) {
                const float cur = xc[i * P];
                float v = bias;
                v = fmaf(wl[3], h3, v); v = fmaf(wl[2], h2, v); v = fmaf(wl[1], h1, v); v = fmaf(wl[0], cur, v);
                xs[i * P + col] = silu_f(v);
                h3 = h2; h2 = h1; h1 = cur;
            }
        }
        for (int i = lt; i < tc; i += nthr) {
            const int t = rev ? L - 1 - (tau0 + i) : tau0 + i;
            const float dlt = softplus_f(ldf(zx + (int64_t)t * a.d_in_proj + a.d_inner + a.conv_ch + h) + dtb);
            dl[i] = dlt;
            da[i] = expf(dlt * Ah);
        }
    };
    // gated output of chunk ci: one warp per token, lanes over the channels; by warps lw = 0..nwarp-1
    auto finish = [&](int ci, int lw, int nwarp, int lane) {
        const int s = ci & 1, tau0 = ci * TC, tc = min(TC, L - tau0);
        const float *zs = xs_of(s) + TC * P, *ys = ys_all + s * TC * P;
        for (int i = lw; i < tc; i += nwarp) {
            const int t = rev ? L - 1 - (tau0 + i) : tau0 + i;
            float sacc = 0.f;
            for (int c = lane; c < P; c += 32) {
                float gv = ys[i * P + c] * silu_f(zs[i * P + c]);
                sacc = fmaf(gv, gv, sacc);
                if (norm_on && norm_w) gv *= ldf(norm_w + h * P + c);
                stf(gout + (int64_t)t * a.d_inner + h * P + c, gv);
            }
            for (int off = 16; off > 0; off >>= 1) sacc += __shfl_xor_sync(0xffffffffu, sacc, off);
            if (lane == 0 && ssq) ssq[(int64_t)t * a.H + h] = sacc;
        }
    };
    prepare(0, tid, nall);                                 // first chunk: everybody
    __syncthreads();

    if (tid >= NS) {
        // ------------------------------------------------------------------ loader group
        const int lt = tid - NS;
        for (int ci = 0; ci < nchunks; ++ci) {
            if (ci > 0) finish(ci - 1, lt >> 5, NL / 32, lt & 31);
            asm volatile("bar.sync 1, %0;" ::"n"(NL) : "memory");     // the stage read by finish() is the one prepare() refills
            if (ci + 1 < nchunks) prepare(ci + 1, lt, NL);
            __syncthreads();
        }
    } else {
        // ------------------------------------------------------------------ scan group
        const int p = tid / LPC, j = tid - p * LPC;
        const float Dh = (a.flags & DM_FLAG_D_SKIP) ? w.D[h] : 0.f;
        // state slice of this lane: float4 index f = q*LPC + j, q = 0..NQ-1
        float hst[4 * NQ];
        if (!rev && a.ssm_in) {
            const float *h0 = a.ssm_in + (((int64_t)b * a.H + h) * P + p) * N;
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                const float4 v = *reinterpret_cast<const float4 *>(h0 + (q * LPC + j) * 4);
                hst[4 * q] = v.x; hst[4 * q + 1] = v.y; hst[4 * q + 2] = v.z; hst[4 * q + 3] = v.w;
            }
        } else {
#pragma unroll
            for (int q = 0; q < 4 * NQ; ++q) hst[q] = 0.f;
        }
        for (int ci = 0; ci < nchunks; ++ci) {
            const int s = ci & 1, tc = min(TC, L - ci * TC);
            const float *xs = xs_of(s), *Bs = xs + 2 * TC * P, *Cs = Bs + TC * N, *dl = Cs + TC * N, *da = dl + TC;
            float *ys = ys_all + s * TC * P;
            // h_t = a_t h_{t-1} + Delta_t x_t (x) B_t ;  y_t = h_t C_t + D x_t
#pragma unroll 2
            for (int i = 0; i < tc; ++i) {
                const float av = da[i];
                const float xv = xs[i * P + p];
                const float dx = dl[i] * xv;
                const float4 *B4 = reinterpret_cast<const float4 *>(Bs + i * N);
                const float4 *C4 = reinterpret_cast<const float4 *>(Cs + i * N);
                float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;      // four partial sums keep the dependent chain short
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    const float4 bv = B4[q * LPC + j], cv = C4[q * LPC + j];
                    hst[4 * q + 0] = fmaf(av, hst[4 * q + 0], dx * bv.x); a0 = fmaf(hst[4 * q + 0], cv.x, a0);
                    hst[4 * q + 1] = fmaf(av, hst[4 * q + 1], dx * bv.y); a1 = fmaf(hst[4 * q + 1], cv.y, a1);
                    hst[4 * q + 2] = fmaf(av, hst[4 * q + 2], dx * bv.z); a2 = fmaf(hst[4 * q + 2], cv.z, a2);
                    hst[4 * q + 3] = fmaf(av, hst[4 * q + 3], dx * bv.w); a3 = fmaf(hst[4 * q + 3], cv.w, a3);
                }
                float acc = (a0 + a1) + (a2 + a3);
                for (int off = LPC >> 1; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
                if (j == 0) ys[i * P + p] = fmaf(Dh, xv, acc);
            }
            __syncthreads();
        }
        if (!rev && a.ssm_out) {
            float *ho = a.ssm_out + (((int64_t)b * a.H + h) * P + p) * N;
#pragma unroll
            for (int q = 0; q < NQ; ++q)
                *reinterpret_cast<float4 *>(ho + (q * LPC + j) * 4) =
                    make_float4(hst[4 * q], hst[4 * q + 1], hst[4 * q + 2], hst[4 * q + 3]);
        }
    }
    finish(nchunks - 1, tid >> 5, nall >> 5, tid & 31);    // last chunk: everybody (the loop's last barrier made y visible)
}

}  // namespace

size_t scan_seq_workspace_bytes(const ScanArgs &a) {
    return align_up((size_t)2 * a.B * a.L * 2 * a.N * sizeof(float));      // B', C' of both directions, fp32
}

cudaError_t scan_sequential(const ScanArgs &a, void *ws, cudaStream_t s) {
    if (!ws) return cudaErrorInvalidValue;
    if (a.N % 16 || a.P % 32) return cudaErrorNotSupported;
    const int NQ = a.N > 128 ? 8 : 4;
    const int LPC = a.N / (4 * NQ);                     // lanes per channel: 1, 2, 4 or 8
    const int NS = a.P * LPC;
    if (LPC < 1 || (LPC & (LPC - 1)) || LPC > 8 || NS > 512 || NS < 32 || a.N != 4 * NQ * LPC) return cudaErrorNotSupported;
    const int ndir = (a.dir_mask == DM_DIR_BOTH) ? 2 : 1;
    const int dir0 = (a.dir_mask == DM_DIR_REV) ? 1 : 0;
    int TC = a.chunk > 0 ? a.chunk : 32;
    if (TC > a.L) TC = a.L;
    size_t smem;
    for (;;) {
        smem = ((size_t)TC * (2 * (2 * a.P + 2 * a.N + 2) + 2 * a.P) + (size_t)(TC + 3) * a.P) * sizeof(float);
        if (smem <= 160 * 1024 || TC == 1) break;
        TC = (TC + 1) / 2;
    }
    typedef void (*Kern)(const ScanArgs, const int, const int, const int, const float *);
    Kern kern;
    if (a.dtype == DM_BF16) kern = NQ == 8 ? (Kern)scan_seq_kernel<__nv_bfloat16, 8> : (Kern)scan_seq_kernel<__nv_bfloat16, 4>;
    else kern = NQ == 8 ? (Kern)scan_seq_kernel<float, 8> : (Kern)scan_seq_kernel<float, 4>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    float *bc = static_cast<float *>(ws);
    const int rows = 32;
    dim3 pgrid((a.L + rows - 1) / rows, a.B, ndir);
    if (a.dtype == DM_BF16) bc_prep_kernel<__nv_bfloat16><<<pgrid, 256, 0, s>>>(a, dir0, bc, rows);
    else bc_prep_kernel<float><<<pgrid, 256, 0, s>>>(a, dir0, bc, rows);
    count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    dim3 grid(a.H, ndir, a.B);
    kern<<<grid, NS + NL, smem, s>>>(a, dir0, TC, LPC, bc);
    count_launch();
    return cudaGetLastError();
}

}  // namespace dm
