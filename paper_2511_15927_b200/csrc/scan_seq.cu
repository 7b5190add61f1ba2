// Fused depthwise conv + SiLU, discretisation, selective scan and gate on the CUDA cores, both
// directions in one launch.  One CTA owns one (batch row, direction, head) and walks the sequence in
// logical time (left-to-right for the forward layer, right-to-left for the reverse layer: the reverse
// layer is the same operator on the reversed sequence, done here by index arithmetic only).
//
// The state h[p][n] of a head lives in registers: channel p is served by LPC = N/16 adjacent lanes,
// each holding 16 states; the C-contraction is finished with warp shuffles.  Per chunk of tokens the
// CTA first prepares conv(x), conv(B), conv(C), Delta and the decay in shared memory, then runs the
// token loop without any block-wide barrier, then writes the gated output with coalesced stores.
//
// This is the exact (fp32) form of the recurrence; it is the kernel for fp32 I/O, for small d_state
// (where it is bandwidth-bound), and for short blocks in block-autoregressive decoding.
#include "dm_internal.h"

namespace dm {
namespace {

template <typename T> __device__ __forceinline__ float ldf(const T *p);
template <> __device__ __forceinline__ float ldf<float>(const float *p) { return __ldg(p); }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16 *p) {
    return __bfloat162float(*p);
}
template <typename T> __device__ __forceinline__ void stf(T *p, float v);
template <> __device__ __forceinline__ void stf<float>(float *p, float v) { *p = v; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float silu_f(float v) { return v / (1.f + expf(-v)); }
__device__ __forceinline__ float softplus_f(float v) { return fmaxf(v, 0.f) + log1pf(expf(-fabsf(v))); }

template <typename T>
__global__ void __launch_bounds__(1024)
scan_seq_kernel(const ScanArgs a, const int dir0, const int TC) {
    extern __shared__ __align__(16) float smem[];
    const int P = a.P, N = a.N, L = a.L, k = a.k;
    const int LPC = N / 16;
    const int h = blockIdx.x, b = blockIdx.z;
    const int dir = dir0 + blockIdx.y;                 // 0 = left-to-right, 1 = right-to-left
    const bool rev = dir == 1;
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int p = tid / LPC, j = tid % LPC;

    float *xs = smem;                  // [TC][P]  conv(x) of this head
    float *zs = xs + TC * P;           // [TC][P]  z, overwritten by the gated output
    float *Bs = zs + TC * P;           // [TC][N]
    float *Cs = Bs + TC * N;           // [TC][N]
    float *dl = Cs + TC * N;           // [TC] Delta
    float *da = dl + TC;               // [TC] exp(Delta * A)

    const ScanDir &w = a.dir[dir];
    const T *conv_w = static_cast<const T *>(w.conv_w);
    const T *conv_b = static_cast<const T *>(w.conv_b);
    const T *norm_w = static_cast<const T *>(w.norm_w);
    const bool has_bias = (a.flags & DM_FLAG_CONV_BIAS) && conv_b != nullptr;
    const bool norm_on = (a.flags & DM_FLAG_GATED_RMSNORM) != 0;
    const float Dh = (a.flags & DM_FLAG_D_SKIP) ? w.D[h] : 0.f;
    const float Ah = -expf(w.A_log[h]);
    const float dtb = w.dt_bias[h];

    const int64_t T_all = (int64_t)a.B * L;
    const T *zx = static_cast<const T *>(a.zx) + ((int64_t)dir * T_all + (int64_t)b * L) * a.d_in_proj;
    T *gout = static_cast<T *>(a.g) + ((int64_t)dir * T_all + (int64_t)b * L) * a.d_inner;
    float *ssq = a.ssq ? a.ssq + ((int64_t)dir * T_all + (int64_t)b * L) * a.H : nullptr;
    const T *conv_in = (!rev && a.conv_in) ? static_cast<const T *>(a.conv_in) + (int64_t)b * (k - 1) * a.conv_ch : nullptr;

    // state slice of this lane: float4 index f = q*LPC + j, q = 0..3
    float hst[16];
    if (!rev && a.ssm_in) {
        const float *h0 = a.ssm_in + (((int64_t)b * a.H + h) * P + p) * N;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float4 v = *reinterpret_cast<const float4 *>(h0 + (q * LPC + j) * 4);
            hst[4 * q] = v.x; hst[4 * q + 1] = v.y; hst[4 * q + 2] = v.z; hst[4 * q + 3] = v.w;
        }
    } else {
#pragma unroll
        for (int q = 0; q < 16; ++q) hst[q] = 0.f;
    }

    // pre-conv value of conv channel cc at logical time tau (tau < 0: carried rows or zeros)
    auto raw = [&](int tau, int cc) -> float {
        if (tau >= 0) {
            const int t = rev ? L - 1 - tau : tau;
            return ldf(zx + (int64_t)t * a.d_in_proj + a.d_inner + cc);
        }
        return conv_in ? ldf(conv_in + (int64_t)(k - 1 + tau) * a.conv_ch + cc) : 0.f;
    };
    auto conv_act = [&](int tau, int cc) -> float {
        float v = has_bias ? ldf(conv_b + cc) : 0.f;
        for (int jj = 0; jj < k; ++jj) v = fmaf(ldf(conv_w + (int64_t)cc * k + jj), raw(tau - (k - 1) + jj, cc), v);
        return silu_f(v);
    };

    for (int tau0 = 0; tau0 < L; tau0 += TC) {
        const int tc = min(TC, L - tau0);
        // ---- prologue: everything the token loop reads goes to shared memory
        for (int e = tid; e < tc * P; e += nthr) {
            const int i = e / P, c = e % P;
            const int t = rev ? L - 1 - (tau0 + i) : tau0 + i;
            xs[i * P + c] = conv_act(tau0 + i, h * P + c);
            zs[i * P + c] = ldf(zx + (int64_t)t * a.d_in_proj + h * P + c);
        }
        for (int e = tid; e < tc * 2 * N; e += nthr) {
            const int i = e / (2 * N), c = e % (2 * N);
            const float v = conv_act(tau0 + i, a.d_inner + c);
            if (c < N) Bs[i * N + c] = v; else Cs[i * N + c - N] = v;
        }
        for (int i = tid; i < tc; i += nthr) {
            const int t = rev ? L - 1 - (tau0 + i) : tau0 + i;
            const float dlt = softplus_f(ldf(zx + (int64_t)t * a.d_in_proj + a.d_inner + a.conv_ch + h) + dtb);
            dl[i] = dlt;
            da[i] = expf(dlt * Ah);
        }
        __syncthreads();
        // ---- token loop: h_t = a_t h_{t-1} + Delta_t x_t (x) B_t ;  y_t = h_t C_t + D x_t
        for (int i = 0; i < tc; ++i) {
            const float av = da[i];
            const float xv = xs[i * P + p];
            const float dx = dl[i] * xv;
            const float4 *B4 = reinterpret_cast<const float4 *>(Bs + i * N);
            const float4 *C4 = reinterpret_cast<const float4 *>(Cs + i * N);
            float acc = 0.f;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float4 bv = B4[q * LPC + j], cv = C4[q * LPC + j];
                hst[4 * q + 0] = fmaf(av, hst[4 * q + 0], dx * bv.x); acc = fmaf(hst[4 * q + 0], cv.x, acc);
                hst[4 * q + 1] = fmaf(av, hst[4 * q + 1], dx * bv.y); acc = fmaf(hst[4 * q + 1], cv.y, acc);
                hst[4 * q + 2] = fmaf(av, hst[4 * q + 2], dx * bv.z); acc = fmaf(hst[4 * q + 2], cv.z, acc);
                hst[4 * q + 3] = fmaf(av, hst[4 * q + 3], dx * bv.w); acc = fmaf(hst[4 * q + 3], cv.w, acc);
            }
            for (int off = LPC >> 1; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
            if (j == 0) {
                const float y = fmaf(Dh, xv, acc);
                zs[i * P + p] = y * silu_f(zs[i * P + p]);
            }
        }
        __syncthreads();
        // ---- epilogue: coalesced store of the gated output, per-token sum of squares for the norm
        for (int e = tid; e < tc * P; e += nthr) {
            const int i = e / P, c = e % P;
            const int t = rev ? L - 1 - (tau0 + i) : tau0 + i;
            float gv = zs[i * P + c];
            if (norm_on && norm_w) gv *= ldf(norm_w + h * P + c);
            stf(gout + (int64_t)t * a.d_inner + h * P + c, gv);
        }
        if (ssq) {
            const int warp = tid >> 5, lane = tid & 31, nwarp = nthr >> 5;
            for (int i = warp; i < tc; i += nwarp) {
                float sacc = 0.f;
                for (int c = lane; c < P; c += 32) { const float gv = zs[i * P + c]; sacc = fmaf(gv, gv, sacc); }
                for (int off = 16; off > 0; off >>= 1) sacc += __shfl_xor_sync(0xffffffffu, sacc, off);
                if (lane == 0) {
                    const int t = rev ? L - 1 - (tau0 + i) : tau0 + i;
                    ssq[(int64_t)t * a.H + h] = sacc;
                }
            }
        }
        __syncthreads();
    }
    if (!rev && a.ssm_out) {
        float *ho = a.ssm_out + (((int64_t)b * a.H + h) * P + p) * N;
#pragma unroll
        for (int q = 0; q < 4; ++q)
            *reinterpret_cast<float4 *>(ho + (q * LPC + j) * 4) =
                make_float4(hst[4 * q], hst[4 * q + 1], hst[4 * q + 2], hst[4 * q + 3]);
    }
}

}  // namespace

cudaError_t scan_sequential(const ScanArgs &a, cudaStream_t s) {
    const int LPC = a.N / 16;
    const int nthr = a.P * LPC;
    if (a.N % 16 || (LPC & (LPC - 1)) || LPC > 32 || a.P % 32 || nthr > 1024 || nthr < 32) return cudaErrorNotSupported;
    const int ndir = (a.dir_mask == DM_DIR_BOTH) ? 2 : 1;
    const int dir0 = (a.dir_mask == DM_DIR_REV) ? 1 : 0;
    int TC = a.chunk > 0 ? a.chunk : (a.N <= 32 ? 64 : 32);
    if (TC > a.L) TC = a.L;
    size_t smem;
    for (;;) {
        smem = (size_t)TC * (2 * a.P + 2 * a.N + 2) * sizeof(float);
        if (smem <= 200 * 1024 || TC == 1) break;
        TC = (TC + 1) / 2;
    }
    auto kern = a.dtype == DM_BF16 ? scan_seq_kernel<__nv_bfloat16> : scan_seq_kernel<float>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    dim3 grid(a.H, ndir, a.B);
    kern<<<grid, nthr, smem, s>>>(a, dir0, TC);
    count_launch();
    return cudaGetLastError();
}

}  // namespace dm
