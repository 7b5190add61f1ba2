// bf16 x bf16 -> fp32 GEMM on the 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM,
// operands staged by TMA with the 128-byte swizzle, mbarrier pipeline), for the dense projections:
//     C[m, n] = row_scale[m] * sum_k A[m, k] * B[n, k] + addend[m, n]
// Persistent kernel, one CTA per SM, CTA tile 128 x BN, K step 64.  Warp roles: warp 0 issues the TMA
// loads, warp 1 owns TMEM and issues the MMAs, warps 2-5 drain the accumulator (double-buffered in
// TMEM, so the epilogue of one tile overlaps the main loop of the next).
// Tall tiles (MB = 2: 256 x 256, two 128-row accumulator blocks that share the B stage, all 512 TMEM columns as one buffer, eight
// epilogue warps) are for few rows and many columns, where every CTA has one tile anyway: each weight tile is then fetched by
// half as many CTAs, and what L2 delivers to the SMs is what bounds such a product.
//
// Every wait on an mbarrier is bounded by wall time; when one gives up the CTA raises an abort flag,
// stores DM_ERR_TIMEOUT in the device status word, waits (bounded) for its own TMA loads, frees its
// TMEM and returns.
#include "dm_internal.h"
#include "tc_ptx.cuh"

namespace dm {
namespace {

using namespace tc;

constexpr int BM = 128, BK = 64;
constexpr int MAX_STAGES = 6;
// pipeline depth: as many (A, B) stages as shared memory holds -- 4 x 48 KB with 256-column tiles, 6 x 32 KB with 128-column tiles (whose
// lower arithmetic intensity needs more bytes in flight per MMA clock)
__host__ __device__ constexpr int stages_for(int bn, int mb) { return mb == 2 ? 3 : bn == 128 ? 6 : 4; }
__host__ __device__ constexpr int threads_for(int mb) { return 64 + 128 * mb; }      // TMA warp, MMA warp, 4 epilogue warps per row block

struct __align__(8) PipeBars {
    uint64_t full[MAX_STAGES], empty[MAX_STAGES], tmem_full[2], tmem_empty[2];
    uint32_t tmem_base;
    int abort;
};

struct EpiArgs {
    void *C; int64_t ldc; int c_is_f32;
    const float *row_scale; const float *addend; int64_t ld_add;
    int M, N, K;
    int silu_cols;   // SiLU on output columns below this one
    const float *col_bias; int gelu; const float *col_scale; int cs_rows; int64_t ld_cs;   // see GemmArgs
    const int *m_dev; int m_off;
    int n_fast;      // tile order: consecutive tiles step along N (the A rows are streamed once, B stays in L2) or along M
    int k_off;       // first element along K of this problem's share (split K: the second half of a product is a problem of its own)
};

// Up to two products of the same M, N, K in one launch (the two directions' in_proj, or their out_proj on short inputs), each optionally
// cut in two along K (ksplit: problems 2 i and 2 i + 1 are the halves of product i, each with an output of its own that the caller adds): the tile
// loop runs over both, so that they share one tail round and -- for in_proj, whose A operand is the same x -- the rows of A in L2.
struct EpiPair { EpiArgs p[4]; int nprob; int ksplit; };

template <int BN, int MB>
__global__ void __launch_bounds__(threads_for(MB), 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a0, const __grid_constant__ CUtensorMap map_b0,
               const __grid_constant__ CUtensorMap map_a1, const __grid_constant__ CUtensorMap map_b1,
               const __grid_constant__ EpiPair epp, int *status) {
    const EpiArgs &ep = epp.p[0];              // sizes and tile order are common to both problems
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte aligned base, derived by offsetting the __shared__ array so that accesses stay shared-space loads and stores
    uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    constexpr int STAGES = stages_for(BN, MB);
    constexpr uint32_t A_BLOCK = BM * BK * 2, A_BYTES = MB * A_BLOCK, B_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
    constexpr int NBUF = MB == 1 ? 2 : 1;            // accumulator buffers
    PipeBars *bars = reinterpret_cast<PipeBars *>(smem + STAGES * STAGE_BYTES);
    volatile int *abort_flag = &bars->abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // rows to compute: all of them, or the count another kernel left on the device (tiles beyond it are skipped)
    const int M_eff = ep.m_dev ? min(ep.M, max(0, *ep.m_dev - ep.m_off)) : ep.M;
    const int tiles_m = (M_eff + MB * BM - 1) / (MB * BM), tiles_n = (ep.N + BN - 1) / BN;
    const int np = epp.nprob, tiles_np = tiles_n * np;         // the problems sit side by side along N
    const int num_tiles = tiles_m * tiles_np;
    // tile -> (row block, column block over both problems); the column block's problem is cb / tiles_n
    auto tile_mb = [&](int tile) { return ep.n_fast ? tile / tiles_np : tile % tiles_m; };
    auto tile_cb = [&](int tile) { return ep.n_fast ? tile % tiles_np : tile / tiles_m; };
    const int kblocks = (ep.K + BK - 1) / BK;
    constexpr uint32_t TMEM_COLS = 2 * BN;          // two accumulator buffers, or the two row blocks of a tall tile; 256 or 512 columns

    if (threadIdx.x == 0) {
        for (int i = 0; i < STAGES; ++i) { mbar_init(&bars->full[i], 1); mbar_init(&bars->empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&bars->tmem_full[i], 1); mbar_init(&bars->tmem_empty[i], 4 * MB); }
        bars->abort = 0;
        mbar_fence_init();
    }
    if (warp == 1) {
        tmem_alloc(&bars->tmem_base, TMEM_COLS);
    }
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem_base = bars->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (one lane)
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int cb = tile_cb(tile), prob = cb / tiles_n;
                const int m0 = tile_mb(tile) * MB * BM, n0 = (cb - prob * tiles_n) * BN;
                const int prod = epp.ksplit ? prob >> 1 : prob, k_off = epp.p[prob].k_off;
                const CUtensorMap *ma = prod ? &map_a1 : &map_a0, *mb = prod ? &map_b1 : &map_b0;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                    if (!(ok = mbar_wait(&bars->empty[s], ph ^ 1u, abort_flag, status))) break;
                    uint8_t *sa = smem + s * STAGE_BYTES, *sb = sa + A_BYTES;
                    mbar_expect_tx(&bars->full[s], STAGE_BYTES);
#pragma unroll
                    for (int i = 0; i < MB; ++i) tma_load_2d(sa + i * A_BLOCK, ma, k_off + kb * BK, m0 + i * BM, &bars->full[s]);
                    tma_load_2d(sb, mb, k_off + kb * BK, n0, &bars->full[s]);
                }
            }
            if (!ok) {
                // aborting: give the loads already issued a bounded chance to land before the CTA goes away
                const uint32_t first = it > STAGES ? it - STAGES : 0;
                for (uint32_t j = first; j < it; ++j) {
                    mbar_wait_quiet(&bars->full[j % STAGES], (j / STAGES) & 1u, 100000000ull);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (one lane)
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16(BM, BN, 0, 0);
            uint32_t it = 0, tcount = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tcount) {
                const uint32_t buf = NBUF == 2 ? tcount & 1u : 0u, bph = (NBUF == 2 ? tcount >> 1 : tcount) & 1u;
                if (!(ok = mbar_wait(&bars->tmem_empty[buf], bph ^ 1u, abort_flag, status))) break;
                fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                    if (!(ok = mbar_wait(&bars->full[s], ph, abort_flag, status))) break;
                    fence_after();
                    const uint32_t sa = smem_u32(smem + s * STAGE_BYTES), sb = sa + A_BYTES;
                    const uint64_t db = desc_k_sw128(sb);
#pragma unroll
                    for (int i = 0; i < MB; ++i) {          // row block i accumulates into columns [i BN, (i + 1) BN)
                        const uint64_t da = desc_k_sw128(sa + i * A_BLOCK);
#pragma unroll
                        for (int k = 0; k < BK / 16; ++k)      // 32 bytes along K per MMA: +2 in 16-byte units
                            umma_bf16(d_tmem + i * BN, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
                    }
                    umma_commit(&bars->empty[s]);          // frees the stage when these MMAs have read it
                }
                if (ok) umma_commit(&bars->tmem_full[buf]);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue: 4 warps per row block, one TMEM lane quarter each
        const int q = warp & 3;                            // warps 2,3,4,5 -> quarters 2,3,0,1
        const int rb = MB == 1 ? 0 : (warp - 2) >> 2;      // row block of a tall tile
        // 32-byte stores and loads (one full sector per thread) when every row of C / of the addend starts on a 32-byte boundary
        const int c_es = ep.c_is_f32 ? 4 : 2;
        uint32_t tcount = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tcount) {
            const uint32_t buf = NBUF == 2 ? tcount & 1u : 0u, bph = (NBUF == 2 ? tcount >> 1 : tcount) & 1u;
            const int cb = tile_cb(tile), prob = cb / tiles_n;
            const int m0 = tile_mb(tile) * MB * BM + rb * BM, n0 = (cb - prob * tiles_n) * BN;
            const EpiArgs &ep = epp.p[prob];               // this tile's problem: its output, scales and addend
            const bool wide_c = (reinterpret_cast<uintptr_t>(ep.C) & 31u) == 0 && ((ep.ldc * c_es) & 31) == 0;
            const bool wide_add = ep.addend && (reinterpret_cast<uintptr_t>(ep.addend) & 31u) == 0 && ((ep.ld_add * 4) & 31) == 0;
            ok = mbar_wait(&bars->tmem_full[buf], bph, abort_flag, status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            fence_after();
            const int row = m0 + q * 32 + lane;
            const bool row_ok = row < M_eff;
            const float sc = (ep.row_scale && row_ok) ? ep.row_scale[row] : 1.f;
            const float *add_row = ep.addend ? ep.addend + (int64_t)row * ep.ld_add : nullptr;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t r[32];
                tmem_ld_x32(tmem_base + ((uint32_t)(q * 32) << 16) + (MB == 1 ? buf : rb) * BN + c0, r);
                tmem_wait_ld();
                const int col = n0 + c0;
                if (!row_ok || col >= ep.N) continue;
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]) * sc;
                const bool full = col + 32 <= ep.N;
                if (ep.col_bias) {
                    if (full) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            const float4 b4 = *reinterpret_cast<const float4 *>(ep.col_bias + col + j);
                            v[j] += b4.x; v[j + 1] += b4.y; v[j + 2] += b4.z; v[j + 3] += b4.w;
                        }
                    } else {
                        for (int j = 0; j < 32; ++j) if (col + j < ep.N) v[j] += ep.col_bias[col + j];
                    }
                }
                if (col < ep.silu_cols) {                  // gate columns: SiLU here, where the ALUs idle, not in the scan
                    if (col + 32 <= ep.silu_cols) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) { const float hv = 0.5f * v[j]; v[j] = fmaf(hv, tanh_fast(hv), hv); }   // SiLU(v) = v/2 + v/2 tanh(v/2)
                    } else {
                        for (int j = 0; j < 32; ++j)
                            if (col + j < ep.silu_cols) { const float hv = 0.5f * v[j]; v[j] = fmaf(hv, tanh_fast(hv), hv); }
                    }
                }
                if (ep.gelu) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) {                  // GELU, tanh form
                        const float x = v[j], hx = 0.5f * x;
                        v[j] = fmaf(hx, tanh_fast(0.7978845608028654f * fmaf(0.044715f * x, x * x, x)), hx);
                    }
                }
                if (ep.col_scale) {
                    const float *cs = ep.col_scale + (int64_t)(row / ep.cs_rows) * ep.ld_cs + col;
                    if (full) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            const float4 c4 = *reinterpret_cast<const float4 *>(cs + j);
                            v[j] *= c4.x; v[j + 1] *= c4.y; v[j + 2] *= c4.z; v[j + 3] *= c4.w;
                        }
                    } else {
                        for (int j = 0; j < 32; ++j) if (col + j < ep.N) v[j] *= cs[j];
                    }
                }
                if (add_row) {
                    if (full && wide_add) {
#pragma unroll
                        for (int j = 0; j < 32; j += 8) {
                            uint32_t a8[8];
                            ld_global_256(add_row + col + j, a8);
#pragma unroll
                            for (int e = 0; e < 8; ++e) v[j + e] += __uint_as_float(a8[e]);
                        }
                    } else if (full && (ep.ld_add & 3) == 0) {
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
                    if (full && wide_c) {
#pragma unroll
                        for (int j = 0; j < 32; j += 8) {
                            uint32_t o[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e) o[e] = __float_as_uint(v[j + e]);
                            st_global_256(crow + j, o);
                        }
                    } else if (full && (ep.ldc & 3) == 0) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) *reinterpret_cast<float4 *>(crow + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                    } else {
                        for (int j = 0; j < 32; ++j) if (col + j < ep.N) crow[j] = v[j];
                    }
                } else {
                    __nv_bfloat16 *crow = static_cast<__nv_bfloat16 *>(ep.C) + (int64_t)row * ep.ldc + col;
                    if (full && wide_c) {
#pragma unroll
                        for (int j = 0; j < 32; j += 16) {
                            uint32_t o[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e) o[e] = pack_bf16(v[j + 2 * e], v[j + 2 * e + 1]);
                            st_global_256(crow + j, o);
                        }
                    } else if (full && (ep.ldc & 7) == 0) {
#pragma unroll
                        for (int j = 0; j < 32; j += 8)
                            *reinterpret_cast<uint4 *>(crow + j) = make_uint4(pack_bf16(v[j], v[j + 1]), pack_bf16(v[j + 2], v[j + 3]),
                                                                             pack_bf16(v[j + 4], v[j + 5]), pack_bf16(v[j + 6], v[j + 7]));
                    } else {
                        for (int j = 0; j < 32; ++j) if (col + j < ep.N) crow[j] = __float2bfloat16_rn(v[j]);
                    }
                }
            }
            fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->tmem_empty[buf]);
        }
    }
    // ---------------------------------------------------------------- teardown
    fence_before();
    __syncthreads();
    if (warp == 1) {
        fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// 2-D bf16 tensor [rows, cols] with row pitch ld elements; box = [box_rows, 64 columns], 128-byte swizzle.
bool make_map(CUtensorMap *m, const void *base, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
    const uint64_t dims[2] = {(uint64_t)cols, (uint64_t)rows};
    const uint64_t strides[1] = {(uint64_t)ld};
    const uint32_t box[2] = {(uint32_t)BK, (uint32_t)box_rows};
    return make_map_bf16(m, base, 2, dims, strides, box);
}

EpiArgs epi_of(const GemmArgs &a) {
    // The operand with more rows is streamed from HBM once; the other one is re-read by every wave of CTAs and should stay in L2.
    return EpiArgs{a.C, a.ldc, a.c_dtype == DM_F32 ? 1 : 0, a.row_scale, a.addend, a.ld_add, a.M, a.N, a.K, a.silu_cols,
                   a.col_bias, a.gelu, a.col_scale, a.cs_rows > 0 ? a.cs_rows : 1, a.ld_cs > 0 ? a.ld_cs : (int64_t)a.N, a.m_dev, a.m_off, a.M > a.N ? 1 : 0, 0};
}

// b == NULL: one product.  hi != NULL (two products, fp32 outputs): each product is cut in two along K; the first half goes to the
// product's own C with its addend and bias, the second half to hi[i] (same pitch), scaled like the first (the scales are linear).
template <int BN, int MB = 1>
cudaError_t launch(const GemmArgs &a, const GemmArgs *b, float *const *hi, cudaStream_t s) {
    CUtensorMap ma[2], mb[2];
    if (!make_map(&ma[0], a.A, a.M, a.K, a.lda, BM) || !make_map(&mb[0], a.B, a.N, a.K, a.ldb, BN)) return cudaErrorInvalidValue;
    ma[1] = ma[0]; mb[1] = mb[0];
    if (b && (!make_map(&ma[1], b->A, b->M, b->K, b->lda, BM) || !make_map(&mb[1], b->B, b->N, b->K, b->ldb, BN))) return cudaErrorInvalidValue;
    constexpr size_t smem = stages_for(BN, MB) * (size_t)(MB * BM * BK * 2 + BN * BK * 2) + sizeof(PipeBars) + 1024;
    cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<BN, MB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int *status = device_status_ptr();
    if (!status) return cudaErrorUnknown;
    EpiPair epp{};
    if (hi) {
        const GemmArgs *prod[2] = {&a, b};
        for (int i = 0; i < 2; ++i) {
            EpiArgs lo = epi_of(*prod[i]), up = lo;
            lo.K = up.K = prod[i]->K / 2;
            up.k_off = lo.K;
            up.C = hi[i]; up.addend = nullptr; up.col_bias = nullptr;
            epp.p[2 * i] = lo; epp.p[2 * i + 1] = up;
        }
        epp.nprob = 4; epp.ksplit = 1;
    } else {
        epp.p[0] = epi_of(a);
        epp.p[1] = b ? epi_of(*b) : epp.p[0];
        epp.nprob = b ? 2 : 1;
    }
    const int tiles = ((a.M + MB * BM - 1) / (MB * BM)) * ((a.N + BN - 1) / BN) * epp.nprob;
    const int grid = tiles < sm_count() ? tiles : sm_count();
    gemm_tc_kernel<BN, MB><<<grid, threads_for(MB), smem, s>>>(ma[0], mb[0], ma[1], mb[1], epp, status);
    count_launch();
    return cudaGetLastError();
}

// Tile width by rounds of CTAs: a 128 x 256 tile costs about 1.6 times a 128 x 128 one (it fetches 1.5 times the operands for
// twice the products), so the wide tile wins whenever it saves a round -- also when it leaves a single round partly empty.
bool wide_tile(const GemmArgs &a, int nprob) {
    const int tm = (a.M + BM - 1) / BM, sms = sm_count();
    const int rounds128 = (tm * ((a.N + 127) / 128) * nprob + sms - 1) / sms, rounds256 = (tm * ((a.N + 255) / 256) * nprob + sms - 1) / sms;
    return !(a.N <= 128 || 10 * rounds128 <= 16 * rounds256);
}

// Tall tiles pay when the wide tiles would need a second, partly filled round of CTAs and the tall ones fit in one: every CTA then has
// one tile either way, and the tall tile moves a third less operand data per product.
bool tall_tile(const GemmArgs &a, int nprob) {
    const int sms = sm_count(), cols = (a.N + 255) / 256;
    return a.M > BM && !a.m_dev && ((a.M + BM - 1) / BM) * cols * nprob > sms && ((a.M + 2 * BM - 1) / (2 * BM)) * cols * nprob <= sms;
}

}  // namespace

bool gemm_tcgen05_supports(const GemmArgs &a) {
    if (a.in_dtype != DM_BF16) return false;
    if (a.M <= 0 || a.N <= 0 || a.K <= 0) return false;
    if ((a.lda % 8) || (a.ldb % 8)) return false;                                   // TMA: 16-byte row pitch
    if ((reinterpret_cast<uintptr_t>(a.A) & 15u) || (reinterpret_cast<uintptr_t>(a.B) & 15u)) return false;
    if (a.c_dtype == DM_BF16 ? (reinterpret_cast<uintptr_t>(a.C) & 15u) : (reinterpret_cast<uintptr_t>(a.C) & 15u)) return false;
    if (a.addend && (reinterpret_cast<uintptr_t>(a.addend) & 15u)) return false;
    if (a.col_bias && (reinterpret_cast<uintptr_t>(a.col_bias) & 15u)) return false;
    if (a.col_scale && ((reinterpret_cast<uintptr_t>(a.col_scale) & 15u) || ((a.ld_cs > 0 ? a.ld_cs : (int64_t)a.N) & 3))) return false;
    return encode_fn() != nullptr;
}

cudaError_t gemm_tcgen05(const GemmArgs &a, cudaStream_t s) {
    if (!gemm_tcgen05_supports(a)) return cudaErrorNotSupported;
    if (tall_tile(a, 1)) return launch<256, 2>(a, nullptr, nullptr, s);
    return wide_tile(a, 1) ? launch<256>(a, nullptr, nullptr, s) : launch<128>(a, nullptr, nullptr, s);
}

bool gemm_tcgen05_pair_supports(const GemmArgs &a, const GemmArgs &b) {
    return gemm_tcgen05_supports(a) && gemm_tcgen05_supports(b) && a.M == b.M && a.N == b.N && a.K == b.K && !a.m_dev && !b.m_dev &&
           a.c_dtype == b.c_dtype;
}

cudaError_t gemm_tcgen05_pair(const GemmArgs &a, const GemmArgs &b, cudaStream_t s) {
    if (!gemm_tcgen05_pair_supports(a, b)) return cudaErrorNotSupported;
    if (tall_tile(a, 2)) return launch<256, 2>(a, &b, nullptr, s);
    return wide_tile(a, 2) ? launch<256>(a, &b, nullptr, s) : launch<128>(a, &b, nullptr, s);
}

// Few rows and a long K (the out_proj pair of block decoding): two products of 128 x 256 tiles fill less than half of the SMs, and 128 x 128
// tiles run their MMAs at about half rate (their operand traffic per product is twice that of the wide tile).  Halving K instead doubles
// the number of wide tiles.
bool gemm_tcgen05_pair_splitk_pays(const GemmArgs &a, const GemmArgs &b) {
    if (!gemm_tcgen05_pair_supports(a, b) || a.c_dtype != DM_F32 || a.K % (2 * BK) || a.gelu || b.gelu || a.silu_cols || b.silu_cols) return false;
    const int tiles = ((a.M + BM - 1) / BM) * ((a.N + 255) / 256) * 2;
    return a.N > 128 && 2 * tiles <= sm_count();
}

cudaError_t gemm_tcgen05_pair_splitk(const GemmArgs &a, const GemmArgs &b, float *a_hi, float *b_hi, cudaStream_t s) {
    if (!gemm_tcgen05_pair_splitk_pays(a, b) || !a_hi || !b_hi || ((reinterpret_cast<uintptr_t>(a_hi) | reinterpret_cast<uintptr_t>(b_hi)) & 15u))
        return cudaErrorNotSupported;
    float *const hi[2] = {a_hi, b_hi};
    return launch<256>(a, &b, hi, s);
}

}  // namespace dm
