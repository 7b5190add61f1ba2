// bf16 x bf16 -> fp32 GEMM on the 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM,
// operands staged by TMA with the 128-byte swizzle, mbarrier pipeline), for the dense projections:
//     C[m, n] = row_scale[m] * sum_k A[m, k] * B[n, k] + addend[m, n]
// Persistent kernel, one CTA per SM, CTA tile 128 x BN, K step 64.  Warp roles: warp 0 issues the TMA
// loads, warp 1 owns TMEM and issues the MMAs, warps 2-5 drain the accumulator (double-buffered in
// TMEM, so the epilogue of one tile overlaps the main loop of the next).
//
// Every wait on an mbarrier is bounded by wall time; when one gives up the CTA raises an abort flag,
// stores DM_ERR_TIMEOUT in the device status word, waits (bounded) for its own TMA loads, frees its
// TMEM and returns.
#include <cuda.h>

#include "dm_internal.h"

namespace dm {
namespace {

constexpr int BM = 128, BK = 64;
constexpr int STAGES = 4;
constexpr int NUM_THREADS = 192;
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;   // 2 s

struct __align__(8) PipeBars {
    uint64_t full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2];
    uint32_t tmem_base;
    int abort;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint64_t globaltimer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the CTA is aborting (this wait or another one gave up).
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag, int *status) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = globaltimer_ns();
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 63u) {
            if (*abort_flag) return false;
            if (globaltimer_ns() - t0 > WAIT_LIMIT_NS) {
                *abort_flag = 1;
                atomicExch(status, (int)DM_ERR_TIMEOUT);
                return false;
            }
        }
    }
}

__device__ __forceinline__ void tma_load_2d(void *smem_dst, const CUtensorMap *map, int x, int y, uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(smem_dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}

// Shared-memory matrix descriptor: K-major tile whose rows are 128 bytes (64 bf16), 128-byte swizzle,
// 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_k_sw128(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);        // start address, 16-byte units
    d |= (uint64_t)1 << 16;                          // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                          // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                          // 128-byte swizzle
    return d;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t instr_desc_bf16(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld_32x32b_x32(uint32_t taddr, uint32_t *r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
          "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
          "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

struct EpiArgs {
    void *C; int64_t ldc; int c_is_f32;
    const float *row_scale; const float *addend; int64_t ld_add;
    int M, N, K;
};

template <int BN>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const EpiArgs ep, int *status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    constexpr uint32_t A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
    PipeBars *bars = reinterpret_cast<PipeBars *>(smem + STAGES * STAGE_BYTES);
    volatile int *abort_flag = &bars->abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_m = (ep.M + BM - 1) / BM, tiles_n = (ep.N + BN - 1) / BN;
    const int num_tiles = tiles_m * tiles_n;
    const int kblocks = (ep.K + BK - 1) / BK;
    constexpr uint32_t TMEM_COLS = 2 * BN;          // two accumulator buffers; 256 or 512 columns

    if (threadIdx.x == 0) {
        for (int i = 0; i < STAGES; ++i) { mbar_init(&bars->full[i], 1); mbar_init(&bars->empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&bars->tmem_full[i], 1); mbar_init(&bars->tmem_empty[i], 4); }
        bars->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (one lane)
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int m0 = (tile % tiles_m) * BM, n0 = (tile / tiles_m) * BN;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                    if (!(ok = mbar_wait(&bars->empty[s], ph ^ 1u, abort_flag, status))) break;
                    uint8_t *sa = smem + s * STAGE_BYTES, *sb = sa + A_BYTES;
                    mbar_expect_tx(&bars->full[s], STAGE_BYTES);
                    tma_load_2d(sa, &map_a, kb * BK, m0, &bars->full[s]);
                    tma_load_2d(sb, &map_b, kb * BK, n0, &bars->full[s]);
                }
            }
            if (!ok) {
                // aborting: give the loads already issued a bounded chance to land before the CTA goes away
                const uint32_t first = it > STAGES ? it - STAGES : 0;
                for (uint32_t j = first; j < it; ++j) {
                    const uint64_t t0 = globaltimer_ns();
                    while (!mbar_try_wait(&bars->full[j % STAGES], (j / STAGES) & 1u) && globaltimer_ns() - t0 < 100000000ull) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (one lane)
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc_bf16(BN);
            uint32_t it = 0, tcount = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tcount) {
                const uint32_t buf = tcount & 1u, bph = (tcount >> 1) & 1u;
                if (!(ok = mbar_wait(&bars->tmem_empty[buf], bph ^ 1u, abort_flag, status))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                    if (!(ok = mbar_wait(&bars->full[s], ph, abort_flag, status))) break;
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem + s * STAGE_BYTES), sb = sa + A_BYTES;
                    const uint64_t da = smem_desc_k_sw128(sa), db = smem_desc_k_sw128(sb);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)      // 32 bytes along K per MMA: +2 in 16-byte units
                        umma_bf16(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
                    umma_commit(&bars->empty[s]);          // frees the stage when these MMAs have read it
                }
                if (ok) umma_commit(&bars->tmem_full[buf]);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue: 4 warps, one TMEM lane quarter each
        const int q = warp & 3;                            // warps 2,3,4,5 -> quarters 2,3,0,1
        uint32_t tcount = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tcount) {
            const uint32_t buf = tcount & 1u, bph = (tcount >> 1) & 1u;
            const int m0 = (tile % tiles_m) * BM, n0 = (tile / tiles_m) * BN;
            ok = mbar_wait(&bars->tmem_full[buf], bph, abort_flag, status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const int row = m0 + q * 32 + lane;
            const bool row_ok = row < ep.M;
            const float sc = (ep.row_scale && row_ok) ? ep.row_scale[row] : 1.f;
            const float *add_row = ep.addend ? ep.addend + (int64_t)row * ep.ld_add : nullptr;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t r[32];
                tmem_ld_32x32b_x32(tmem_base + ((uint32_t)(q * 32) << 16) + buf * BN + c0, r);
                tmem_wait_ld();
                const int col = n0 + c0;
                if (!row_ok || col >= ep.N) continue;
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]) * sc;
                const bool full = col + 32 <= ep.N;
                if (add_row) {
                    if (full && (ep.ld_add & 3) == 0) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            const float4 a4 = *reinterpret_cast<const float4 *>(add_row + col + j);
                            v[j] += a4.x; v[j + 1] += a4.y; v[j + 2] += a4.z; v[j + 3] += a4.w;
                        }
                    } else {
                        for (int j = 0; j < 32; ++j) if (col + j < ep.N) v[j] += add_row[col + j];
                    }
                }
                if (ep.c_is_f32) {
                    float *crow = static_cast<float *>(ep.C) + (int64_t)row * ep.ldc + col;
                    if (full && (ep.ldc & 3) == 0) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) *reinterpret_cast<float4 *>(crow + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                    } else {
                        for (int j = 0; j < 32; ++j) if (col + j < ep.N) crow[j] = v[j];
                    }
                } else {
                    __nv_bfloat16 *crow = static_cast<__nv_bfloat16 *>(ep.C) + (int64_t)row * ep.ldc + col;
                    if (full && (ep.ldc & 7) == 0) {
#pragma unroll
                        for (int j = 0; j < 32; j += 8)
                            *reinterpret_cast<uint4 *>(crow + j) = make_uint4(pack_bf16(v[j], v[j + 1]), pack_bf16(v[j + 2], v[j + 3]),
                                                                             pack_bf16(v[j + 4], v[j + 5]), pack_bf16(v[j + 6], v[j + 7]));
                    } else {
                        for (int j = 0; j < 32; ++j) if (col + j < ep.N) crow[j] = __float2bfloat16_rn(v[j]);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->tmem_empty[buf]);
        }
    }
    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// 2-D bf16 tensor [rows, cols] with row pitch ld elements; box = [box_rows, 64 columns], 128-byte swizzle.
bool make_map(CUtensorMap *m, const void *base, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int sm_count() {
    static int n = 0;
    if (!n) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (n <= 0) n = 148;
    }
    return n;
}

template <int BN>
cudaError_t launch(const GemmArgs &a, cudaStream_t s) {
    CUtensorMap ma, mb;
    if (!make_map(&ma, a.A, a.M, a.K, a.lda, BM) || !make_map(&mb, a.B, a.N, a.K, a.ldb, BN)) return cudaErrorInvalidValue;
    constexpr size_t smem = STAGES * (size_t)(BM * BK * 2 + BN * BK * 2) + sizeof(PipeBars) + 1024;
    cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int *status = device_status_ptr();
    if (!status) return cudaErrorUnknown;
    const int tiles = ((a.M + BM - 1) / BM) * ((a.N + BN - 1) / BN);
    const int grid = tiles < sm_count() ? tiles : sm_count();
    EpiArgs ep{a.C, a.ldc, a.c_dtype == DM_F32 ? 1 : 0, a.row_scale, a.addend, a.ld_add, a.M, a.N, a.K};
    gemm_tc_kernel<BN><<<grid, NUM_THREADS, smem, s>>>(ma, mb, ep, status);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

bool gemm_tcgen05_supports(const GemmArgs &a) {
    if (a.in_dtype != DM_BF16) return false;
    if (a.M <= 0 || a.N <= 0 || a.K <= 0) return false;
    if ((a.lda % 8) || (a.ldb % 8)) return false;                                   // TMA: 16-byte row pitch
    if ((reinterpret_cast<uintptr_t>(a.A) & 15u) || (reinterpret_cast<uintptr_t>(a.B) & 15u)) return false;
    if (a.c_dtype == DM_BF16 ? (reinterpret_cast<uintptr_t>(a.C) & 15u) : (reinterpret_cast<uintptr_t>(a.C) & 15u)) return false;
    if (a.addend && (reinterpret_cast<uintptr_t>(a.addend) & 15u)) return false;
    return encode_fn() != nullptr;
}

cudaError_t gemm_tcgen05(const GemmArgs &a, cudaStream_t s) {
    if (!gemm_tcgen05_supports(a)) return cudaErrorNotSupported;
    // Narrow outputs take the 128-wide tile so that more CTAs get work.
    const int tiles256 = ((a.M + BM - 1) / BM) * ((a.N + 255) / 256);
    if (a.N <= 128 || tiles256 < sm_count()) return launch<128>(a, s);
    return launch<256>(a, s);
}

}  // namespace dm
