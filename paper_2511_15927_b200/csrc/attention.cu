// Bidirectional multi-head attention for the hybrid variant (Sec. 3.3: one attention mixer every N mixer blocks):
//     O_h = softmax(Q_h K_h^T / sqrt(d_h)) V_h        full (non-causal), no position encoding, d_h = 64 or 80.
// One CTA per (128-query tile, head, sequence) walks the keys in tiles of 128 with the running-maximum form of the
// softmax, so the L x L score matrix never leaves the SM:
//     warp 0      TMA loads: the Q tile once, K and V tiles double-buffered
//     warp 1      one thread issues  S = Q K^T  (both operands K-major in shared memory, fp32 accumulator in TMEM) and
//                 O += P V  (A = P from TMEM as bf16, B = V [key][d_h] MN-major)
//     warps 2-5   one query row per thread: S row -> running max m and sum l, P = 2^(s - m) as bf16 into TMEM, O scaled by
//                 2^(m_old - m_new) in TMEM; at the end O / l -> bf16 -> global
// A CTA holds 256 TMEM columns (S 128, P 64, O 64) and 82 KB of shared memory, so two CTAs share an SM: while one is in
// its softmax (latency bound: one warp per scheduler), the other one's products and softmax fill the gaps.
// Heads of 80 channels (the paper's 1.3B hybrid, d = 1920 with 24 heads): every Q, K, V tile is two 64-column sub-tiles, the head's
// channels 0..63 and the 64 columns from channel 64 on, of which the products use the first 16 (the rest belongs to the next head, or is
// the zero fill beyond the tensor, and is never read): one more K step of 16 for S, one more product of 16 columns for O.  Twice the
// shared memory and 512 TMEM columns: one CTA per SM.
// Every wait is bounded; on expiry the CTA stores DM_ERR_TIMEOUT in the device status word and leaves.
#include "dm_internal.h"
#include "tc_ptx.cuh"

namespace dm {
using namespace tc;
namespace {

constexpr int BQ = 128, BK = 128, SUB = 64, NTHREADS = 192;       // SUB: columns of a sub-tile (128 bytes: one swizzle atom)
constexpr uint32_t TILE = BQ * SUB * 2;                     // 16 KB: 128 rows of 128 bytes
constexpr uint32_t TM_S = 0, TM_P = 128, TM_O = 192;      // S fp32 128 columns, P bf16 64, O fp32 64 or 80
constexpr uint32_t smem_bytes(int nt) { return 5 * nt * TILE + 1024 + 1024; }

struct Bars {
    uint64_t q_full, k_full[2], k_empty[2], v_full[2], v_empty[2], s_full, s_empty, p_full, o_done;
    uint32_t tmem_base;
    int abort;
};

struct AttnArgs {
    int B, Lq, Lk, d, H;         // Lq queries per sequence attend to Lk keys
    int kx0, vx0;                // column of head 0's keys / values in their tensor maps
    __nv_bfloat16 *out;          // [B*Lq, d]
    float scale_log2;            // log2(e) / sqrt(d_h)
};

// NT: sub-tiles per operand tile; 1 = heads of 64 channels, 2 = heads of 80
template <int NT>
__global__ void __launch_bounds__(NTHREADS, 3 - NT)
attention_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v, const AttnArgs a, int *status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    constexpr int DH = NT == 1 ? 64 : 80;
    constexpr uint32_t OPND = NT * TILE;                        // bytes of one operand tile
    constexpr uint32_t OFF_Q = 0, OFF_K = OPND, OFF_V = 3 * OPND, OFF_BAR = 5 * OPND;
    constexpr uint32_t TM_COLS = NT == 1 ? 256 : 512;
    Bars *bars = reinterpret_cast<Bars *>(smem + OFF_BAR);
    volatile int *abort_flag = &bars->abort;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int q0 = blockIdx.x * BQ, h = blockIdx.y, b = blockIdx.z;
    const int n_kv = (a.Lk + BK - 1) / BK;

    if (tid == 0) {
        mbar_init(&bars->q_full, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&bars->k_full[i], 1); mbar_init(&bars->k_empty[i], 1);
            mbar_init(&bars->v_full[i], 1); mbar_init(&bars->v_empty[i], 1);
        }
        mbar_init(&bars->s_full, 1); mbar_init(&bars->s_empty, 128);
        mbar_init(&bars->p_full, 128);
        mbar_init(&bars->o_done, 1);
        bars->abort = 0;
        mbar_fence_init();
    }
    if (warp == 1) tmem_alloc(&bars->tmem_base, TM_COLS);
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem = bars->tmem_base;
    auto WAIT = [&](uint64_t *bar, uint32_t parity) { return mbar_wait(bar, parity, abort_flag, status); };

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            mbar_expect_tx(&bars->q_full, OPND);
#pragma unroll
            for (int u = 0; u < NT; ++u) tma_load_3d(smem + OFF_Q + u * TILE, &map_q, h * DH + u * SUB, q0, b, &bars->q_full);
            int issued_k = 0, issued_v = 0;
            for (int j = 0; j < n_kv; ++j) {
                const int st = j & 1;
                const uint32_t ph = (j >> 1) & 1;
                if (!WAIT(&bars->k_empty[st], ph ^ 1)) break;
                mbar_expect_tx(&bars->k_full[st], OPND);
#pragma unroll
                for (int u = 0; u < NT; ++u) tma_load_3d(smem + OFF_K + st * OPND + u * TILE, &map_k, a.kx0 + h * DH + u * SUB, j * BK, b, &bars->k_full[st]);
                issued_k = j + 1;
                if (!WAIT(&bars->v_empty[st], ph ^ 1)) break;
                mbar_expect_tx(&bars->v_full[st], OPND);
#pragma unroll
                for (int u = 0; u < NT; ++u) tma_load_3d(smem + OFF_V + st * OPND + u * TILE, &map_v, a.vx0 + h * DH + u * SUB, j * BK, b, &bars->v_full[st]);
                issued_v = j + 1;
            }
            if (*abort_flag) {             // aborting: bounded wait for the loads still in flight
                mbar_wait_quiet(&bars->q_full, 0, 100000000ull);
                for (int j = max(0, issued_k - 2); j < issued_k; ++j) mbar_wait_quiet(&bars->k_full[j & 1], (j >> 1) & 1, 100000000ull);
                for (int j = max(0, issued_v - 2); j < issued_v; ++j) mbar_wait_quiet(&bars->v_full[j & 1], (j >> 1) & 1, 100000000ull);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t dQ = desc_lo_k(smem_u32(smem + OFF_Q));
            constexpr uint32_t I_S = idesc_bf16(128, 128, 0, 0), I_O = idesc_bf16(128, 64, 0, 1), I_O16 = idesc_bf16(128, 16, 0, 1);
            auto issue_pv = [&](int j) -> bool {          // O (+)= P(j) V(j)
                const int st = j & 1;
                const uint32_t ph = (j >> 1) & 1;
                if (!WAIT(&bars->p_full, (uint32_t)(j & 1)) || !WAIT(&bars->v_full[st], ph)) return false;
                fence_after();
                const uint32_t dV = desc_lo_mn(smem_u32(smem + OFF_V + st * OPND), TILE), tp = tmem + TM_P;
                if (j == 0) umma_ts<0>(tmem + TM_O, tp, dV, I_O); else umma_ts<1>(tmem + TM_O, tp, dV, I_O);
#pragma unroll
                for (int kk = 1; kk < 8; ++kk) umma_ts<1>(tmem + TM_O, tp + 8 * kk, dV + kk * 128, I_O);
                if constexpr (NT == 2) {                  // channels 64..79: the first 16 columns of the second sub-tile
                    const uint32_t dV2 = desc_lo_mn(smem_u32(smem + OFF_V + st * OPND + TILE), TILE);
                    if (j == 0) umma_ts<0>(tmem + TM_O + 64, tp, dV2, I_O16); else umma_ts<1>(tmem + TM_O + 64, tp, dV2, I_O16);
#pragma unroll
                    for (int kk = 1; kk < 8; ++kk) umma_ts<1>(tmem + TM_O + 64, tp + 8 * kk, dV2 + kk * 128, I_O16);
                }
                umma_commit(&bars->o_done);               // phase j: O holds tiles 0..j; P(j) and the V stage are free
                umma_commit(&bars->v_empty[st]);
                return true;
            };
            bool ok = WAIT(&bars->q_full, 0);
            for (int j = 0; j < n_kv && ok; ++j) {
                const int st = j & 1;
                const uint32_t ph = (j >> 1) & 1;
                if (!WAIT(&bars->k_full[st], ph) || !WAIT(&bars->s_empty, (uint32_t)((j & 1) ^ 1))) { ok = false; break; }
                fence_after();
                const uint32_t dK = desc_lo_k(smem_u32(smem + OFF_K + st * OPND)), ts = tmem + TM_S;
                umma_ss<0>(ts, dQ, dK, I_S);
#pragma unroll
                for (int kk = 1; kk < 4; ++kk) umma_ss<1>(ts, dQ + 2 * kk, dK + 2 * kk, I_S);
                if constexpr (NT == 2) umma_ss<1>(ts, dQ + (TILE >> 4), dK + (TILE >> 4), I_S);      // channels 64..79: one K step of the second sub-tiles
                umma_commit(&bars->s_full);
                umma_commit(&bars->k_empty[st]);
                if (j > 0) ok = issue_pv(j - 1);
            }
            if (ok) issue_pv(n_kv - 1);
        }
    } else {
        // ------------------------------------------------------------ softmax, O scaling, output
        const int q = warp & 3;                                   // TMEM lane quarter of this warp
        const int row = q * 32 + lane;                            // query row of the tile
        const uint32_t tlane = tmem + ((uint32_t)(q * 32) << 16);
        float m = -INFINITY, l = 0.f;
        bool ok = true;
        for (int j = 0; j < n_kv; ++j) {
            ok = ok && WAIT(&bars->s_full, (uint32_t)(j & 1));
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            fence_after();
            const uint32_t ts = tlane + TM_S, tp = tlane + TM_P;
            const int valid = min(BK, a.Lk - j * BK);             // keys of this tile inside the sequence
            // pass 1: the row maximum of the scaled scores
            float mx = -INFINITY;
#pragma unroll 1
            for (int c0 = 0; c0 < BK; c0 += 32) {
                uint32_t r[32];
                tmem_ld_x32(ts + c0, r);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) if (c0 + i < valid) mx = fmaxf(mx, __uint_as_float(r[i]));
            }
            const float m_new = fmaxf(m, mx * a.scale_log2);
            const float alpha = ex2f(m - m_new);                  // 0 on the first tile (m = -inf)
            // P is single-buffered: P V of the previous tile must have read it (that product also completes O for the scaling below)
            if (j > 0) {
                ok = WAIT(&bars->o_done, (uint32_t)((j - 1) & 1));
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                fence_after();
            }
            // pass 2: P = 2^(s - m_new) as bf16 into TMEM, and its row sum
            float sum = 0.f;
#pragma unroll 1
            for (int c0 = 0; c0 < BK; c0 += 32) {
                uint32_t r[32], pk[16];
                tmem_ld_x32(ts + c0, r);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const float p0 = c0 + i < valid ? ex2f(fmaf(__uint_as_float(r[i]), a.scale_log2, -m_new)) : 0.f;
                    const float p1 = c0 + i + 1 < valid ? ex2f(fmaf(__uint_as_float(r[i + 1]), a.scale_log2, -m_new)) : 0.f;
                    pk[i >> 1] = pack_bf16(p0, p1);
                    sum += p0 + p1;
                }
                tmem_st_x16(tp + (c0 >> 1), pk);
            }
            l = fmaf(l, alpha, sum);
            m = m_new;
            fence_before();
            mbar_arrive(&bars->s_empty);                          // every read of S(j) has completed
            // O holds tiles 0..j-1 once PV(j-1) has completed: scale it to the new maximum
            if (j > 0) {
#pragma unroll 1
                for (int c0 = 0; c0 < 64; c0 += 32) {
                    uint32_t r[32];
                    tmem_ld_x32(tlane + TM_O + c0, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                    tmem_st_x32(tlane + TM_O + c0, r);
                }
                if constexpr (NT == 2) {
                    uint32_t r[16];
                    tmem_ld_x16(tlane + TM_O + 64, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                    tmem_st_x16(tlane + TM_O + 64, r);
                }
            }
            tmem_wait_st();
            fence_before();
            mbar_arrive(&bars->p_full);
        }
        if (ok) {
            ok = WAIT(&bars->o_done, (uint32_t)((n_kv - 1) & 1));
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            fence_after();
            const float inv = 1.f / l;
            const int t = q0 + row;
            auto store8 = [&](__nv_bfloat16 *dst, const uint32_t *r) {
                *reinterpret_cast<uint4 *>(dst) =
                    make_uint4(pack_bf16(__uint_as_float(r[0]) * inv, __uint_as_float(r[1]) * inv), pack_bf16(__uint_as_float(r[2]) * inv, __uint_as_float(r[3]) * inv),
                               pack_bf16(__uint_as_float(r[4]) * inv, __uint_as_float(r[5]) * inv), pack_bf16(__uint_as_float(r[6]) * inv, __uint_as_float(r[7]) * inv));
            };
            __nv_bfloat16 *orow = a.out + ((int64_t)b * a.Lq + t) * a.d + h * DH;
#pragma unroll 1
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t r[32];
                tmem_ld_x32(tlane + TM_O + c0, r);
                tmem_wait_ld();
                if (t < a.Lq) {
#pragma unroll
                    for (int i = 0; i < 32; i += 8) store8(orow + c0 + i, r + i);
                }
            }
            if constexpr (NT == 2) {
                uint32_t r[16];
                tmem_ld_x16(tlane + TM_O + 64, r);
                tmem_wait_ld();
                if (t < a.Lq) { store8(orow + 64, r); store8(orow + 72, r + 8); }
            }
        }
    }
    // ---------------------------------------------------------------- teardown
    fence_before();
    __syncthreads();
    if (warp == 1) {
        fence_after();
        tmem_dealloc(tmem, TM_COLS);
    }
}

// The block's keys and values (columns [d, 3 d) of qkv [B*G, 3 d]) go to rows [len, len + G) of the caches [B, cap, d].
__global__ void kv_append_kernel(const __nv_bfloat16 *__restrict__ qkv, __nv_bfloat16 *__restrict__ kc, __nv_bfloat16 *__restrict__ vc,
                                 int G, int d, int len, int cap) {
    const int t = blockIdx.x, b = blockIdx.y;
    const uint4 *src = reinterpret_cast<const uint4 *>(qkv + ((int64_t)b * G + t) * 3 * d + d);
    uint4 *dk = reinterpret_cast<uint4 *>(kc + ((int64_t)b * cap + len + t) * d), *dv = reinterpret_cast<uint4 *>(vc + ((int64_t)b * cap + len + t) * d);
    const int n = d / 8;                                   // 16-byte pieces per row (d is a multiple of 16)
    for (int i = threadIdx.x; i < n; i += blockDim.x) { dk[i] = src[i]; dv[i] = src[n + i]; }
}

}  // namespace

bool attention_supports(int dtype, int d, int n_heads) {
    return dtype == DM_BF16 && n_heads > 0 && (d == n_heads * 64 || d == n_heads * 80) && encode_fn() != nullptr;
}

// qkv [B*Lq, 3 d] bf16 (columns [Q | K | V], heads contiguous inside each), out [B*Lq, d] bf16.
// k_cache == NULL: keys and values are the K and V columns of qkv (Lk = Lq).  Otherwise the block's keys and values are
// first appended at rows [cache_len, cache_len + Lq) of k_cache, v_cache [B, cache_cap, d], and the queries attend to the
// first cache_len + Lq rows of the caches.
cudaError_t attention_forward(const void *qkv, void *out, int B, int Lq, int d, int n_heads, void *k_cache, void *v_cache,
                              int cache_len, int cache_cap, cudaStream_t s) {
    if (!attention_supports(DM_BF16, d, n_heads) || B <= 0 || Lq <= 0 || B > 65535 || n_heads > 65535) return cudaErrorNotSupported;
    const bool cached = k_cache != nullptr;
    if (cached && (!v_cache || cache_len < 0 || cache_len + Lq > cache_cap)) return cudaErrorInvalidValue;
    const int Lk = cached ? cache_len + Lq : Lq;
    CUtensorMap mq, mk, mv;
    const uint32_t box[3] = {(uint32_t)SUB, (uint32_t)BQ, 1};
    const int dh = d / n_heads;
    {
        const uint64_t dims[3] = {(uint64_t)3 * d, (uint64_t)Lq, (uint64_t)B};
        const uint64_t str[2] = {(uint64_t)3 * d, (uint64_t)Lq * 3 * d};
        if (!make_map_bf16(&mq, qkv, 3, dims, str, box)) return cudaErrorInvalidValue;
    }
    if (cached) {
        // the maps end at the last valid key: the rest of a tile is filled with zeros, whatever the cache holds there
        const uint64_t dims[3] = {(uint64_t)d, (uint64_t)Lk, (uint64_t)B};
        const uint64_t str[2] = {(uint64_t)d, (uint64_t)cache_cap * d};
        if (!make_map_bf16(&mk, k_cache, 3, dims, str, box) || !make_map_bf16(&mv, v_cache, 3, dims, str, box)) return cudaErrorInvalidValue;
        kv_append_kernel<<<dim3(Lq, B), 128, 0, s>>>(static_cast<const __nv_bfloat16 *>(qkv), static_cast<__nv_bfloat16 *>(k_cache),
                                                      static_cast<__nv_bfloat16 *>(v_cache), Lq, d, cache_len, cache_cap);
        count_launch();
        cudaError_t e0 = cudaGetLastError();
        if (e0 != cudaSuccess) return e0;
    } else {
        mk = mq; mv = mq;
    }
    int *status = device_status_ptr();
    if (!status) return cudaErrorUnknown;
    AttnArgs a{B, Lq, Lk, d, n_heads, cached ? 0 : d, cached ? 0 : 2 * d, static_cast<__nv_bfloat16 *>(out), 1.4426950408889634f / sqrtf((float)dh)};
    const dim3 grid((Lq + BQ - 1) / BQ, n_heads, B);
    cudaError_t e;
    if (dh == 64) {
        if ((e = cudaFuncSetAttribute(attention_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes(1))) != cudaSuccess) return e;
        attention_kernel<1><<<grid, NTHREADS, smem_bytes(1), s>>>(mq, mk, mv, a, status);
    } else {
        if ((e = cudaFuncSetAttribute(attention_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes(2))) != cudaSuccess) return e;
        attention_kernel<2><<<grid, NTHREADS, smem_bytes(2), s>>>(mq, mk, mv, a, status);
    }
    count_launch();
    return cudaGetLastError();
}

}  // namespace dm
