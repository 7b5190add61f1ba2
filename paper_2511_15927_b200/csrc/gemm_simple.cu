// CUDA-core GEMM with fp32 accumulation.  It serves the fp32 I/O mode (whose 1e-4 tolerance rules out
// reduced-precision tensor products) and shapes the tensor-core kernel does not take.
#include "dm_internal.h"

namespace dm {
namespace {

constexpr int BM = 64, BN = 64, BK = 16, TM = 4, TN = 4;   // 256 threads, 4x4 outputs each

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename TIn, typename TOut>
__global__ void __launch_bounds__(256)
gemm_simple_kernel(const TIn *__restrict__ A, int64_t lda, const TIn *__restrict__ B, int64_t ldb,
                   TOut *C, int64_t ldc, int M, int N, int K,
                   const float *__restrict__ row_scale, const float *addend, int64_t ld_add, int silu_cols,
                   const float *__restrict__ col_bias, int gelu, const float *__restrict__ col_scale, int cs_rows, int64_t ld_cs, const int *__restrict__ m_dev, int m_off) {
    if (m_dev) M = min(M, max(0, *m_dev - m_off));
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int tid = threadIdx.x;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int tx = tid % 16, ty = tid / 16;
    float acc[TM][TN] = {};
    for (int k0 = 0; k0 < K; k0 += BK) {
        // 64 rows x 16 k per operand = 1024 elements, 4 per thread; consecutive threads walk k
        for (int e = tid; e < BM * BK; e += 256) {
            const int r = e / BK, kk = e % BK;
            const int gm = m0 + r, gk = k0 + kk;
            As[kk][r] = (gm < M && gk < K) ? to_f32(A[(int64_t)gm * lda + gk]) : 0.f;
            const int gn = n0 + r;
            Bs[kk][r] = (gn < N && gk < K) ? to_f32(B[(int64_t)gn * ldb + gk]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[TM], b[TN];
#pragma unroll
            for (int i = 0; i < TM; ++i) a[i] = As[kk][ty * TM + i];
#pragma unroll
            for (int j = 0; j < TN; ++j) b[j] = Bs[kk][tx * TN + j];
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        const int gm = m0 + ty * TM + i;
        if (gm >= M) continue;
        const float sc = row_scale ? row_scale[gm] : 1.f;
#pragma unroll
        for (int j = 0; j < TN; ++j) {
            const int gn = n0 + tx * TN + j;
            if (gn >= N) continue;
            float v = acc[i][j] * sc;
            if (col_bias) v += col_bias[gn];
            if (gn < silu_cols) v = v / (1.f + __expf(-v));
            if (gelu) v = 0.5f * v * (1.f + tanhf(0.7978845608028654f * (v + 0.044715f * v * v * v)));
            if (col_scale) v *= col_scale[(int64_t)(gm / cs_rows) * ld_cs + gn];
            if (addend) v += addend[(int64_t)gm * ld_add + gn];
            if constexpr (sizeof(TOut) == 4) C[(int64_t)gm * ldc + gn] = v;
            else C[(int64_t)gm * ldc + gn] = __float2bfloat16_rn(v);
        }
    }
}

template <typename TIn, typename TOut>
cudaError_t launch(const GemmArgs &a, cudaStream_t s) {
    dim3 grid((a.N + BN - 1) / BN, (a.M + BM - 1) / BM);
    gemm_simple_kernel<TIn, TOut><<<grid, 256, 0, s>>>(
        static_cast<const TIn *>(a.A), a.lda, static_cast<const TIn *>(a.B), a.ldb,
        static_cast<TOut *>(a.C), a.ldc, a.M, a.N, a.K, a.row_scale, a.addend, a.ld_add, a.silu_cols,
        a.col_bias, a.gelu, a.col_scale, a.cs_rows > 0 ? a.cs_rows : 1, a.ld_cs > 0 ? a.ld_cs : a.N, a.m_dev, a.m_off);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

cudaError_t gemm_simple(const GemmArgs &a, cudaStream_t s) {
    if (a.M <= 0 || a.N <= 0 || a.K <= 0) return cudaErrorInvalidValue;
    if ((a.M + BM - 1) / BM > 65535) return cudaErrorInvalidValue;
    if (a.in_dtype == DM_F32) {
        return a.c_dtype == DM_F32 ? launch<float, float>(a, s) : launch<float, __nv_bfloat16>(a, s);
    }
    return a.c_dtype == DM_F32 ? launch<__nv_bfloat16, float>(a, s) : launch<__nv_bfloat16, __nv_bfloat16>(a, s);
}

}  // namespace dm
