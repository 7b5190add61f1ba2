// Fused conv + selective scan + gate for bf16 I/O with d_state = 128 and headdim = 64, in the chunked
// (state-space-duality) form of the same recurrence, with the chunk products on the tensor cores.
//
// Unrolling h_t = a_t h_{t-1} + Delta_t x_t (x) B_t over one chunk of Q = 128 tokens, with
// Lambda_i = sum_{r <= i} Delta_r A (inclusive, in the direction's own time order) gives
//     y_i   = sum_{j <= i} exp(Lambda_i - Lambda_j) (C_i . B_j) Delta_j x_j  +  exp(Lambda_i) C_i . h_in  +  D x_i
//     h_out = exp(Lambda_last) h_in + sum_j exp(Lambda_last - Lambda_j) Delta_j x_j (x) B_j
// Only differences of Lambda with non-positive sign are exponentiated; nothing is divided by a decay.
//
// Launch 1 (ssd_prep): per (direction, batch row, chunk): conv + SiLU of the B and C columns (shared by
// all heads) to bf16, and Delta, Lambda of every head, into scratch.
// Launch 2 (ssd_scan): one CTA per (batch row, direction, head) walks the chunks in the direction's time
// order.  Both directions use the same physical chunk grid [c*Q, (c+1)*Q); the reverse direction visits
// the chunks in descending order and uses the transposed causal mask, so nothing is ever flipped in memory.
// Per chunk:  S = C B^T,  W = S o mask  (bf16, shared memory),  Y = W x' + diag(exp Lambda) C h_in,
// state accumulator = B^T (w o x'), all four products as tcgen05 MMAs with fp32 accumulators in TMEM.
// The running state h [d_state x headdim] stays in fp32 registers (one state row per thread of warps 4-7).
//
// Every mbarrier wait is bounded; on expiry the CTA stores DM_ERR_TIMEOUT in the device status word,
// lets its outstanding TMA loads land (bounded), frees TMEM and returns.
#include "dm_internal.h"
#include "tc_ptx.cuh"

namespace dm {
namespace {

using namespace tc;

constexpr int Q = 128;            // tokens per chunk
constexpr int P = 64;             // headdim
constexpr int N = 128;            // d_state
constexpr int HALO = 8;           // conv look-back rows kept with the x tile (8 keeps the tile 1024-byte aligned)
constexpr int XROWS = Q + HALO;
constexpr uint32_t T16 = Q * 128;           // bytes of a [128 rows][64 bf16] tile
constexpr uint32_t XTILE = XROWS * 128;     // 17408
constexpr int NTHREADS = 256;

// shared-memory map (offsets from a 1024-byte aligned base)
constexpr uint32_t OFF_X = 0;                       // 2 stages of the x tile (raw, then conv'd in place)
constexpr uint32_t OFF_B = OFF_X + 2 * XTILE;       // B' as two [Q][64] tiles (d_state halves)
constexpr uint32_t OFF_C = OFF_B + 2 * T16;
constexpr uint32_t OFF_W = OFF_C + 2 * T16;         // masked S, two [Q][64] tiles (halves of the j axis)
constexpr uint32_t OFF_XS = OFF_W + 2 * T16;        // w_j x'_j
constexpr uint32_t OFF_H = OFF_XS + T16;            // bf16 copy of the incoming state [d_state rows][headdim]
constexpr uint32_t OFF_DL = OFF_H + T16;            // 2 stages x (Delta[Q], Lambda[Q]) fp32
constexpr uint32_t OFF_MISC = OFF_DL + 2 * 2 * Q * 4;
constexpr uint32_t SMEM_BYTES = OFF_MISC + 1024 + 1024;   // + barriers/scalars + alignment slack

// TMEM columns
constexpr uint32_t TM_S = 0, TM_YA = 128, TM_YB = 192, TM_ST = 256, TM_COLS = 512;

struct Misc {
    uint64_t in_full[2], bc_full, mma_done;
    uint32_t tmem_base;
    int abort;
    float norm_w[P];
};

struct SsdArgs {
    int B, L, H, d_inner, d_in_proj, conv_ch, k, flags, nch, Lp;
    const __nv_bfloat16 *zx;
    __nv_bfloat16 *g;
    float *ssq;
    const float *dA;             // [2][B][H][2][Lp]
    const float *ssm_in; float *ssm_out;
    ScanDir dir[2];
};

__device__ __forceinline__ float silu_fast(float v) { return v / (1.f + __expf(-v)); }

// --------------------------------------------------------------------------------------------------
// Launch 1: B', C' (bf16) and Delta, Lambda (fp32) for one physical chunk of one (direction, batch row).
// --------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
ssd_prep_kernel(const SsdArgs a, __nv_bfloat16 *__restrict__ Bp, __nv_bfloat16 *__restrict__ Cp, float *__restrict__ dA, int dir0) {
    const int pc = blockIdx.x, b = blockIdx.y, dir = dir0 + blockIdx.z;
    const bool rev = dir == 1;
    const int L = a.L, k = a.k;
    const ScanDir &w = a.dir[dir];
    const int64_t seq = (int64_t)dir * a.B + b;
    const __nv_bfloat16 *zx = a.zx + seq * L * a.d_in_proj;
    const int r0 = pc * Q;
    const bool has_bias = (a.flags & DM_FLAG_CONV_BIAS) && w.conv_b;
    // B and C channels
    for (int c = threadIdx.x; c < 2 * N; c += blockDim.x) {
        const int cc = a.d_inner + c;                                  // conv channel
        const __nv_bfloat16 *cw = static_cast<const __nv_bfloat16 *>(w.conv_w) + (int64_t)cc * k;
        float wl[4] = {0.f, 0.f, 0.f, 0.f};                            // wl[m]: weight of the row m steps back in time
        for (int m = 0; m < k; ++m) wl[m] = __bfloat162float(cw[k - 1 - m]);
        const float bias = has_bias ? __bfloat162float(static_cast<const __nv_bfloat16 *>(w.conv_b)[cc]) : 0.f;
        const __nv_bfloat16 *col = zx + a.d_inner + cc;
        auto raw = [&](int t) -> float { return (t >= 0 && t < L) ? __bfloat162float(col[(int64_t)t * a.d_in_proj]) : 0.f; };
        __nv_bfloat16 *dst = (c < N ? Bp + c : Cp + (c - N)) + seq * L * N;
        const int step = rev ? -1 : 1;                                 // direction of time in physical rows
        int t = rev ? min(r0 + Q, L) - 1 : r0;
        float h1 = raw(t - step), h2 = raw(t - 2 * step), h3 = raw(t - 3 * step);
        const int rows = min(r0 + Q, L) - r0;
        for (int i = 0; i < rows; ++i, t += step) {
            const float cur = raw(t);
            float v = bias;
            v = fmaf(wl[3], h3, v); v = fmaf(wl[2], h2, v); v = fmaf(wl[1], h1, v); v = fmaf(wl[0], cur, v);
            dst[(int64_t)t * N] = __float2bfloat16_rn(silu_fast(v));
            h3 = h2; h2 = h1; h1 = cur;
        }
    }
    // Delta and the inclusive cumulative log-decay of every head, in the direction's time order
    for (int h = threadIdx.x; h < a.H; h += blockDim.x) {
        const float Ah = -expf(w.A_log[h]), dtb = w.dt_bias[h];
        float *dl = dA + ((seq * a.H + h) * 2) * a.Lp + r0, *lam = dl + a.Lp;
        float cum = 0.f;
        for (int i = 0; i < Q; ++i) {
            const int r = rev ? Q - 1 - i : i, t = r0 + r;
            float d = 0.f;
            if (t < L) {
                const float v = __bfloat162float(zx[(int64_t)t * a.d_in_proj + a.d_inner + a.conv_ch + h]) + dtb;
                d = fmaxf(v, 0.f) + log1pf(expf(-fabsf(v)));
            }
            cum = fmaf(d, Ah, cum);
            dl[r] = d;
            lam[r] = cum;
        }
    }
}

// --------------------------------------------------------------------------------------------------
// Launch 2: the chunked scan.
// --------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(NTHREADS, 1)
ssd_scan_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_b,
                const __grid_constant__ CUtensorMap map_c, const SsdArgs a, int dir0, int *status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    Misc *misc = reinterpret_cast<Misc *>(smem + OFF_MISC);
    volatile int *abort_flag = &misc->abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int h = blockIdx.x, b = blockIdx.z, dir = dir0 + blockIdx.y;
    const bool rev = dir == 1;
    const int L = a.L, nch = a.nch;
    const int seq = dir * a.B + b;
    const ScanDir &w = a.dir[dir];
    const bool norm_on = (a.flags & DM_FLAG_GATED_RMSNORM) != 0;
    const float Dh = (a.flags & DM_FLAG_D_SKIP) ? w.D[h] : 0.f;
    const bool group_a = warp < 4;                  // conv, mask, epilogue: thread <-> token row
    const int row = tid & 127;                      // token row (group A) or state row n (group B)
    const int quarter = warp & 3;                   // TMEM lane quarter this warp may read

    if (tid == 0) {
        mbar_init(&misc->in_full[0], 1); mbar_init(&misc->in_full[1], 1);
        mbar_init(&misc->bc_full, 1); mbar_init(&misc->mma_done, 1);
        misc->abort = 0;
        mbar_fence_init();
    }
    if (tid < P) misc->norm_w[tid] = (norm_on && w.norm_w) ? __bfloat162float(static_cast<const __nv_bfloat16 *>(w.norm_w)[h * P + tid]) : 1.f;
    if (warp == 0) tmem_alloc(&misc->tmem_base, TM_COLS);
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem = misc->tmem_base;

    // conv parameters of this thread's 8 channels (group A): wl[e][m] multiplies the row m steps back in time
    const int cc8 = row & 7, rb = row >> 3;
    float wl[8][4], cbias[8];
    if (group_a) {
        const bool has_bias = (a.flags & DM_FLAG_CONV_BIAS) && w.conv_b;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int ch = h * P + cc8 * 8 + e;
            const __nv_bfloat16 *cw = static_cast<const __nv_bfloat16 *>(w.conv_w) + (int64_t)ch * a.k;
#pragma unroll
            for (int m = 0; m < 4; ++m) wl[e][m] = m < a.k ? __bfloat162float(cw[a.k - 1 - m]) : 0.f;
            cbias[e] = has_bias ? __bfloat162float(static_cast<const __nv_bfloat16 *>(w.conv_b)[ch]) : 0.f;
        }
    }
    // running state of state row n = row (group B): hreg[p], fp32
    float hreg[P];
    if (!group_a) {
        if (!rev && a.ssm_in) {
            const float *h0 = a.ssm_in + (((int64_t)b * a.H + h) * P) * N + row;
#pragma unroll
            for (int p = 0; p < P; ++p) hreg[p] = h0[(int64_t)p * N];
        } else {
#pragma unroll
            for (int p = 0; p < P; ++p) hreg[p] = 0.f;
        }
    }

    const float *dA_head = a.dA + (((int64_t)seq * a.H + h) * 2) * a.Lp;
    auto issue_in = [&](int c, int s) {             // x tile (+halo) and Delta/Lambda of chunk index c into stage s
        const int pc = rev ? nch - 1 - c : c;
        mbar_expect_tx(&misc->in_full[s], XTILE + 2 * Q * 4);
        tma_load_3d(smem + OFF_X + s * XTILE, &map_x, a.d_inner + h * P, rev ? pc * Q : pc * Q - HALO, seq, &misc->in_full[s]);
        bulk_load(smem + OFF_DL + s * 2 * Q * 4, dA_head + pc * Q, Q * 4, &misc->in_full[s]);
        bulk_load(smem + OFF_DL + s * 2 * Q * 4 + Q * 4, dA_head + a.Lp + pc * Q, Q * 4, &misc->in_full[s]);
    };
    auto issue_bc = [&](int c) {
        const int pc = rev ? nch - 1 - c : c;
        mbar_expect_tx(&misc->bc_full, 4 * T16);
        tma_load_3d(smem + OFF_B, &map_b, 0, pc * Q, seq, &misc->bc_full);
        tma_load_3d(smem + OFF_B + T16, &map_b, 64, pc * Q, seq, &misc->bc_full);
        tma_load_3d(smem + OFF_C, &map_c, 0, pc * Q, seq, &misc->bc_full);
        tma_load_3d(smem + OFF_C + T16, &map_c, 64, pc * Q, seq, &misc->bc_full);
    };
    if (tid == 0) { issue_in(0, 0); issue_bc(0); }

    uint32_t mma_phase = 0;
    int in_issued = 1, bc_issued = 1;               // chunks whose loads have been issued (thread 0 bookkeeping)
    bool ok = true;
    for (int c = 0; c < nch; ++c) {
        const int s = c & 1;
        const int pc = rev ? nch - 1 - c : c;
        uint8_t *xt = smem + OFF_X + s * XTILE;
        const float *dl = reinterpret_cast<const float *>(smem + OFF_DL + s * 2 * Q * 4), *lam = dl + Q;
        if (tid == 0 && c + 1 < nch) { issue_in(c + 1, s ^ 1); in_issued = c + 2; }

        ok = mbar_wait(&misc->in_full[s], (c >> 1) & 1, abort_flag, status);
        if (!__syncthreads_and(ok)) { ok = false; break; }

        const float lam_last = lam[rev ? 0 : Q - 1];
        // ---------------- phase A: conv + SiLU in place (group A) | bf16 copy of the incoming state (group B)
        if (group_a) {
            uint4 win[11];
            const int base_row = rev ? rb * 8 : rb * 8 + HALO - 3;
#pragma unroll
            for (int i = 0; i < 11; ++i) {
                const int r = base_row + i;
                win[i] = *reinterpret_cast<const uint4 *>(xt + r * 128 + ((cc8 ^ (r & 7)) << 4));
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");          // all raw rows are read before anyone overwrites
#pragma unroll
            for (int e8 = 0; e8 < 8; ++e8) {
                const int j = rb * 8 + e8;                          // chunk row
                const float wj = __expf(lam_last - lam[j]) * dl[j];
                float o[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    float v = cbias[e];
#pragma unroll
                    for (int m = 3; m >= 0; --m) {
                        const int wi = rev ? e8 + m : e8 + 3 - m;
                        const uint32_t word = reinterpret_cast<const uint32_t *>(&win[wi])[e >> 1];
                        v = fmaf(wl[e][m], (e & 1) ? bf16_hi(word) : bf16_lo(word), v);
                    }
                    o[e] = silu_fast(v);
                }
                const int xr = rev ? j : j + HALO;
                *reinterpret_cast<uint4 *>(xt + xr * 128 + ((cc8 ^ (xr & 7)) << 4)) =
                    make_uint4(pack_bf16(o[0], o[1]), pack_bf16(o[2], o[3]), pack_bf16(o[4], o[5]), pack_bf16(o[6], o[7]));
                *reinterpret_cast<uint4 *>(smem + OFF_XS + j * 128 + ((cc8 ^ (j & 7)) << 4)) =
                    make_uint4(pack_bf16(wj * o[0], wj * o[1]), pack_bf16(wj * o[2], wj * o[3]), pack_bf16(wj * o[4], wj * o[5]),
                               pack_bf16(wj * o[6], wj * o[7]));
            }
        } else {
#pragma unroll
            for (int c8 = 0; c8 < 8; ++c8)
                *reinterpret_cast<uint4 *>(smem + OFF_H + row * 128 + ((c8 ^ (row & 7)) << 4)) =
                    make_uint4(pack_bf16(hreg[c8 * 8], hreg[c8 * 8 + 1]), pack_bf16(hreg[c8 * 8 + 2], hreg[c8 * 8 + 3]),
                               pack_bf16(hreg[c8 * 8 + 4], hreg[c8 * 8 + 5]), pack_bf16(hreg[c8 * 8 + 6], hreg[c8 * 8 + 7]));
        }
        fence_proxy_async();
        ok = mbar_wait(&misc->bc_full, c & 1, abort_flag, status);
        fence_before();
        if (!__syncthreads_and(ok)) { ok = false; break; }
        // ---------------- MMAs: S = C B^T;  Y_b = C h_in;  state accumulator = B^T (w o x')
        if (tid == 0) {
            fence_after();
            const uint32_t sB = smem_u32(smem + OFF_B), sC = smem_u32(smem + OFF_C), sH = smem_u32(smem + OFF_H), sXs = smem_u32(smem + OFF_XS);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const uint64_t dc = desc_k_sw128(sC + (kk >> 2) * T16) + 2 * (kk & 3);
                umma_bf16(tmem + TM_S, dc, desc_k_sw128(sB + (kk >> 2) * T16) + 2 * (kk & 3), idesc_bf16(128, 128, 0, 0), kk != 0);
                umma_bf16(tmem + TM_YB, dc, desc_mn_sw128(sH + kk * 2048, T16, 1024), idesc_bf16(128, 64, 0, 1), kk != 0);
            }
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
                umma_bf16(tmem + TM_ST, desc_mn_sw128(sB + kk * 2048, T16, 1024), desc_mn_sw128(sXs + kk * 2048, T16, 1024),
                          idesc_bf16(128, 64, 1, 1), kk != 0);
            umma_commit(&misc->mma_done);
        }
        ok = mbar_wait(&misc->mma_done, mma_phase, abort_flag, status);
        mma_phase ^= 1;
        if (!__syncthreads_and(ok)) { ok = false; break; }
        fence_after();
        if (tid == 0 && c + 1 < nch) { issue_bc(c + 1); bc_issued = c + 2; }     // B', C' tiles are free again
        // ---------------- phase B: W = S o mask (group A) | state update (group B)
        if (group_a) {
            const float li = lam[row];
#pragma unroll 1
            for (int jb = 0; jb < 4; ++jb) {
                const bool needed = rev ? jb >= quarter : jb <= quarter;
                uint32_t out[16];
                if (needed) {
                    uint32_t r[32];
                    tmem_ld_x32(tmem + ((uint32_t)(quarter * 32) << 16) + TM_S + jb * 32, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int jj = 0; jj < 32; jj += 2) {
                        const int j0 = jb * 32 + jj;
                        const bool v0 = rev ? j0 >= row : j0 <= row, v1 = rev ? j0 + 1 >= row : j0 + 1 <= row;
                        const float m0 = v0 ? __expf(li - lam[j0]) * dl[j0] : 0.f;
                        const float m1 = v1 ? __expf(li - lam[j0 + 1]) * dl[j0 + 1] : 0.f;
                        out[jj >> 1] = pack_bf16(__uint_as_float(r[jj]) * m0, __uint_as_float(r[jj + 1]) * m1);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i) out[i] = 0u;
                }
                uint8_t *wt = smem + OFF_W + (jb >> 1) * T16 + row * 128;
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4) {
                    const int cidx = (jb & 1) * 4 + c4;
                    *reinterpret_cast<uint4 *>(wt + ((cidx ^ (row & 7)) << 4)) = make_uint4(out[c4 * 4], out[c4 * 4 + 1], out[c4 * 4 + 2], out[c4 * 4 + 3]);
                }
            }
        } else {
            const float dec = __expf(lam_last);
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t r[32];
                tmem_ld_x32(tmem + ((uint32_t)(quarter * 32) << 16) + TM_ST + half * 32, r);
                tmem_wait_ld();
#pragma unroll
                for (int p = 0; p < 32; ++p) hreg[half * 32 + p] = fmaf(dec, hreg[half * 32 + p], __uint_as_float(r[p]));
            }
        }
        fence_proxy_async();
        fence_before();
        __syncthreads();
        // ---------------- MMA: Y_a = W x'
        if (tid == 0) {
            fence_after();
            const uint32_t sW = smem_u32(smem + OFF_W), sX = smem_u32(xt) + (rev ? 0 : HALO * 128);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
                umma_bf16(tmem + TM_YA, desc_k_sw128(sW + (kk >> 2) * T16) + 2 * (kk & 3), desc_mn_sw128(sX + kk * 2048, T16, 1024),
                          idesc_bf16(128, 64, 0, 1), kk != 0);
            umma_commit(&misc->mma_done);
        }
        ok = mbar_wait(&misc->mma_done, mma_phase, abort_flag, status);
        mma_phase ^= 1;
        if (!__syncthreads_and(ok)) { ok = false; break; }
        fence_after();
        // ---------------- phase C: y = Y_a + exp(Lambda_i) Y_b + D x';  g = y SiLU(z);  store
        if (group_a) {
            const int t = pc * Q + row;
            const bool valid = t < L;
            const float ei = __expf(lam[row]);
            const int xr = rev ? row : row + HALO;
            const __nv_bfloat16 *zrow = a.zx + ((int64_t)seq * L + (valid ? t : 0)) * a.d_in_proj + h * P;
            __nv_bfloat16 *grow = a.g + ((int64_t)seq * L + (valid ? t : 0)) * a.d_inner + h * P;
            float ss = 0.f;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t ya[32], yb[32];
                tmem_ld_x32(tmem + ((uint32_t)(quarter * 32) << 16) + TM_YA + half * 32, ya);
                tmem_ld_x32(tmem + ((uint32_t)(quarter * 32) << 16) + TM_YB + half * 32, yb);
                tmem_wait_ld();
                if (valid) {
#pragma unroll
                    for (int c4 = 0; c4 < 4; ++c4) {                 // 8 channels per 16-byte chunk
                        const int c8 = half * 4 + c4;
                        const uint4 xv = *reinterpret_cast<const uint4 *>(xt + xr * 128 + ((c8 ^ (xr & 7)) << 4));
                        const uint4 zv = *reinterpret_cast<const uint4 *>(zrow + c8 * 8);
                        const uint32_t xw[4] = {xv.x, xv.y, xv.z, xv.w}, zw[4] = {zv.x, zv.y, zv.z, zv.w};
                        uint32_t ow[4];
#pragma unroll
                        for (int e2 = 0; e2 < 4; ++e2) {
                            const int p = c4 * 8 + e2 * 2;           // within this half
                            const float y0 = fmaf(ei, __uint_as_float(yb[p]), __uint_as_float(ya[p])) + Dh * bf16_lo(xw[e2]);
                            const float y1 = fmaf(ei, __uint_as_float(yb[p + 1]), __uint_as_float(ya[p + 1])) + Dh * bf16_hi(xw[e2]);
                            const float g0 = y0 * silu_fast(bf16_lo(zw[e2])), g1 = y1 * silu_fast(bf16_hi(zw[e2]));
                            ss = fmaf(g0, g0, ss); ss = fmaf(g1, g1, ss);
                            ow[e2] = pack_bf16(g0 * misc->norm_w[half * 32 + p], g1 * misc->norm_w[half * 32 + p + 1]);
                        }
                        *reinterpret_cast<uint4 *>(grow + c8 * 8) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
                    }
                }
            }
            if (valid && a.ssq) a.ssq[((int64_t)seq * L + t) * a.H + h] = ss;
        }
        fence_before();
        __syncthreads();
    }

    // ---------------------------------------------------------------- teardown
    if (!ok && tid == 0) {          // aborting: bounded wait for the loads still in flight
        for (int c = max(0, in_issued - 2); c < in_issued; ++c) mbar_wait_quiet(&misc->in_full[c & 1], (c >> 1) & 1, 100000000ull);
        if (bc_issued > 0) mbar_wait_quiet(&misc->bc_full, (bc_issued - 1) & 1, 100000000ull);
    }
    if (ok && !group_a && !rev && a.ssm_out) {
        float *ho = a.ssm_out + (((int64_t)b * a.H + h) * P) * N + row;
#pragma unroll
        for (int p = 0; p < P; ++p) ho[(int64_t)p * N] = hreg[p];
    }
    fence_before();
    __syncthreads();
    if (warp == 0) {
        fence_after();
        tmem_dealloc(tmem, TM_COLS);
    }
}

struct Scratch {
    size_t bp, cp, da, total;
    int nch, Lp;
};
Scratch scratch_layout(const ScanArgs &a) {
    Scratch s;
    s.nch = (a.L + Q - 1) / Q;
    s.Lp = s.nch * Q;
    size_t off = 0;
    s.bp = off; off += align_up((size_t)2 * a.B * a.L * N * 2);
    s.cp = off; off += align_up((size_t)2 * a.B * a.L * N * 2);
    s.da = off; off += align_up((size_t)2 * a.B * a.H * 2 * s.Lp * 4);
    s.total = off;
    return s;
}

}  // namespace

bool scan_ssd_supports(const ScanArgs &a) {
    if (a.dtype != DM_BF16 || a.N != N || a.P != P || a.k < 2 || a.k > 4) return false;
    if (a.d_in_proj % 8 || a.d_inner % 8) return false;                  // 16-byte rows for TMA and vector access
    if (a.conv_in) return false;                                         // carried conv rows take the sequential kernel
    if (a.L < 64) return false;                                          // short blocks: the sequential kernel is the better fit
    if (a.H > 65535 || a.B > 65535) return false;
    return encode_fn() != nullptr;
}

size_t scan_ssd_workspace_bytes(const ScanArgs &a) {
    if (a.dtype != DM_BF16 || a.N != N || a.P != P) return 0;
    return scratch_layout(a).total;
}

cudaError_t scan_ssd(const ScanArgs &a, void *ws, cudaStream_t s) {
    if (!scan_ssd_supports(a) || !ws) return cudaErrorNotSupported;
    const Scratch l = scratch_layout(a);
    char *base = static_cast<char *>(ws);
    __nv_bfloat16 *Bp = reinterpret_cast<__nv_bfloat16 *>(base + l.bp), *Cp = reinterpret_cast<__nv_bfloat16 *>(base + l.cp);
    float *dA = reinterpret_cast<float *>(base + l.da);
    SsdArgs k{};
    k.B = a.B; k.L = a.L; k.H = a.H; k.d_inner = a.d_inner; k.d_in_proj = a.d_in_proj; k.conv_ch = a.conv_ch; k.k = a.k;
    k.flags = a.flags; k.nch = l.nch; k.Lp = l.Lp;
    k.zx = static_cast<const __nv_bfloat16 *>(a.zx); k.g = static_cast<__nv_bfloat16 *>(a.g); k.ssq = a.ssq; k.dA = dA;
    k.ssm_in = a.ssm_in; k.ssm_out = a.ssm_out;
    k.dir[0] = a.dir[0]; k.dir[1] = a.dir[1];
    const int ndir = a.dir_mask == DM_DIR_BOTH ? 2 : 1, dir0 = a.dir_mask == DM_DIR_REV ? 1 : 0;

    CUtensorMap mx, mb, mc;
    {
        const uint64_t dims[3] = {(uint64_t)a.d_in_proj, (uint64_t)a.L, (uint64_t)2 * a.B};
        const uint64_t str[2] = {(uint64_t)a.d_in_proj, (uint64_t)a.L * a.d_in_proj};
        const uint32_t box[3] = {64, (uint32_t)XROWS, 1};
        if (!make_map_bf16(&mx, a.zx, 3, dims, str, box)) return cudaErrorInvalidValue;
    }
    {
        const uint64_t dims[3] = {(uint64_t)N, (uint64_t)a.L, (uint64_t)2 * a.B};
        const uint64_t str[2] = {(uint64_t)N, (uint64_t)a.L * N};
        const uint32_t box[3] = {64, (uint32_t)Q, 1};
        if (!make_map_bf16(&mb, Bp, 3, dims, str, box) || !make_map_bf16(&mc, Cp, 3, dims, str, box)) return cudaErrorInvalidValue;
    }
    int *status = device_status_ptr();
    if (!status) return cudaErrorUnknown;

    ssd_prep_kernel<<<dim3(l.nch, a.B, ndir), 256, 0, s>>>(k, Bp, Cp, dA, dir0);
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(ssd_scan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
    if (e != cudaSuccess) return e;
    ssd_scan_kernel<<<dim3(a.H, ndir, a.B), NTHREADS, SMEM_BYTES, s>>>(mx, mb, mc, k, dir0, status);
    count_launch();
    return cudaGetLastError();
}

}  // namespace dm
