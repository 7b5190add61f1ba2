// Fused conv + selective scan + gate for bf16 I/O with d_state <= 128 (zero-padded to 128) and headdim 64 or 32, in
// the chunked (state-space-duality) form of the same recurrence.
//
// Unrolling h_t = a_t h_{t-1} + Delta_t x_t (x) B_t over one chunk of Q tokens, with
// Lambda_i = sum_{r <= i} Delta_r A (inclusive, in the direction's own time order) gives
//     y_i   = sum_{j <= i} exp(Lambda_i - Lambda_j) (C_i . B_j) Delta_j x_j  +  exp(Lambda_i) C_i . h_in  +  D x_i
//     h_out = exp(Lambda_last) h_in + sum_j exp(Lambda_last - Lambda_j) Delta_j x_j (x) B_j
// Only differences of Lambda with non-positive sign are kept; nothing is divided by a decay.  Delta_j is
// folded into the exponent (Lambda'_j = Lambda_j - log Delta_j), and D x_i into the diagonal of the masked
// product, so that  y_i = sum_j W_ij x_j + exp(Lambda_i) C_i . h_in  with  W_ij = S_ij exp(Lambda_i - Lambda'_j) [+ D].
//
// Launch 1 (ssd_prep): per (direction, batch row, chunk): conv + SiLU of the B and C columns (shared by
// all heads) to bf16, and Lambda, Lambda' of every head (in log2 units), into scratch.
// Launch 2, long sequences (ssd_scan, Q = 128, chunk products on the tcgen05 tensor cores): one CTA per (batch row,
// direction, head) walks the chunks in the direction's time order.  Both directions use the same physical chunk grid
// [c*Q, (c+1)*Q); the reverse direction visits the chunks in descending order and uses the transposed causal mask, so
// nothing is ever flipped in memory.
// The CTA is a pipeline of specialised warps that work on different chunks at the same time:
//     warp 0      TMA loads of the x tile (+ conv halo) and of Lambda, Lambda'
//     warp 1      issues the four tcgen05 products of a chunk:  S = C B^T,  Yb = C h_in,  Ya = W x',  St = B^T (w o x')
//     warp 2      TMA loads of the z tile        warp 3   TMA loads of the B' and C' tiles
//     warps 4-11   conv groups: state hand-over (the fp32 state stays in TMEM and St accumulates onto it: its bf16 copy for Yb is
//                  taken and it is scaled by exp(Lambda_last) before St is issued); depthwise conv + SiLU of the x tile in place
//                  (8-row blocks); the decay-weighted copy w o x'
//     warps 12-19  mask groups: S (TMEM, fp32) -> W (TMEM, bf16), the 16-column groups split between the two groups
//     warps 20-27  epilogue groups (half of the channels each): y = Ya + exp(Lambda_i) Yb,  g = y SiLU(z) [* norm_w] (the z
//                  tile arrives as SiLU(z): the in_proj epilogue applies it), per-head sum of squares, written over the z tile and stored with TMA
// Every hand-off is an mbarrier; every wait is bounded.  On expiry the CTA stores DM_ERR_TIMEOUT in the
// device status word, all roles leave their loops, outstanding TMA traffic is waited for (bounded), TMEM is
// freed and the CTA returns.
// Launch 2, short blocks (ssd_block, Q = 32, products with mma.sync from registers): the active block of block-autoregressive
// decoding is 32 tokens, a quarter of one tcgen05 tile, and a call has thousands of (batch row, head) items of that size;
// for them the pipeline above is all set-up and tear-down.  ssd_block is a plain CTA of 256 threads per item: it takes the
// 32 x 32 matrix S of each sub-chunk from the prep launch (which computes it once per (batch row, direction)), builds W
// and runs the other three products of the identities above on 16 x 8 x 16 tiles; a state that has to outlive the
// sub-chunk stays in its fp32 accumulators.  It is also what `chunk = 32` selects at any length.
#include <cstddef>

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
constexpr int NX = 3, NZ = 2, NB = 2, NDL = 4;      // pipeline depths: x tile, z tile, B' tile, (Lambda, Lambda')
constexpr int WG = 128;                     // threads of one worker group (four warps = the four TMEM lane quarters)
constexpr int NWG = 2;                      // worker groups per role: conv, mask + state, epilogue (the column splits below assume 2)
constexpr int ROLE = NWG * WG;              // threads of one role
constexpr int NTHREADS = 128 + 3 * ROLE;    // warps 0-3: TMA producers and the MMA issuer

// shared-memory map (offsets from a 1024-byte aligned base; every tile starts on a 1024-byte boundary)
constexpr uint32_t OFF_X = 0;                           // NX stages of the x tile (raw, then conv'd in place)
constexpr uint32_t OFF_Z = OFF_X + NX * XTILE;          // NZ stages of the z tile, overwritten by the gated output
constexpr uint32_t OFF_B = OFF_Z + NZ * T16;            // NB stages of B' as two [Q][64] tiles (d_state halves)
constexpr uint32_t OFF_C = OFF_B + NB * 2 * T16;        // C' in transit to TMEM, two [Q][64] tiles
constexpr uint32_t OFF_XS = OFF_C + 2 * T16;            // w_j x'_j
constexpr uint32_t OFF_H = OFF_XS + T16;                // bf16 copy of the incoming state [d_state rows][headdim]
constexpr uint32_t OFF_DL = OFF_H + T16;                // NDL stages x (Lambda[Q], Lambda'[Q]) fp32
constexpr uint32_t DL_HEAD = 2 * Q * 4;                  // one head's (Lambda, Lambda') of a chunk
constexpr uint32_t OFF_MISC = OFF_DL + NDL * DL_HEAD;    // one head per CTA; two heads per CTA: OFF_MISC + NDL * DL_HEAD
constexpr uint32_t SMEM_BYTES = OFF_MISC + 7168 + 1024;  // + barriers/scalars + alignment slack
constexpr uint32_t SMEM_BYTES_PAIR = SMEM_BYTES + NDL * DL_HEAD;
static_assert(OFF_Z % 1024 == 0 && OFF_B % 1024 == 0 && OFF_C % 1024 == 0 && OFF_XS % 1024 == 0 && OFF_H % 1024 == 0, "tile alignment");
static_assert(SMEM_BYTES_PAIR <= 232448, "shared memory budget");

// TMEM columns (all 512 are allocated)
constexpr uint32_t TM_S = 0, TM_W = 128, TM_YB1 = 192, TM_YA = 256, TM_YB0 = 320, TM_W1 = 384, TM_HS = 448, TM_COLS = 512;    // Yb is double-buffered; W1: the second head's W when a CTA carries two heads

struct Misc {
    uint64_t full_x[NX], empty_x[NX], full_z[NZ], empty_z[NZ], full_b[NB], empty_b[NB], full_c, empty_c, full_dl[NDL], empty_dl[NDL];
    uint64_t xs_full, s_full, s_empty, w_full, st_full, hs_ready, h_full, y_full, ya_empty, yb_empty[2];
    uint32_t tmem_base;
    int abort;
    int ticket;                   // order in which this CTA started (fused prep: the first ones take the prep role)
    alignas(16) float norm_w[P];  // the three arrays below are read as float4
    alignas(16) float wbuf[2][Q];  // [1] only with two heads per CTA
    alignas(16) float cbuf[NWG][4][Q]; // per mask warp: column factors of the off-diagonal blocks
    float ssq_part[Q];            // sum of squares of the second epilogue group's channels
};
static_assert(sizeof(Misc) <= 7168, "Misc must fit its slot");
static_assert(offsetof(Misc, norm_w) % 16 == 0 && offsetof(Misc, wbuf) % 16 == 0 && offsetof(Misc, cbuf) % 16 == 0, "float4 access");

struct SsdArgs {
    int B, L, H, d_inner, d_in_proj, conv_ch, k, flags, nch, Lp;
    int Nr;                      // d_state of the model (<= N); B', C' and the state are zero-padded to N
    int Pr;                      // headdim of the model: P, or P / 2 (the CTA then carries the next head's channels as unused padding)
    int zx_tied;                 // both directions read the in_proj output of direction 0 (shared projections)
    __nv_bfloat16 *g;            // [2][B*L][d_inner] gated output (written with plain stores when Pr < P, else through map_g)
    const __nv_bfloat16 *zx;
    float *ssq;
    const float *dA;             // [2][B][H][2][Lp]: Lambda, Lambda' (log2 units)
    const float *ssm_in; float *ssm_out;
    const __nv_bfloat16 *conv_in;  // [B][k-1][conv_ch] pre-conv rows before the first token (left-to-right layer), or NULL
    ScanDir dir[2];
};

__device__ __forceinline__ float silu_fast(float v) { const float hv = 0.5f * v; return fmaf(hv, tanh_fast(hv), hv); }     // SiLU(v) = v/2 + v/2 tanh(v/2)
// Arithmetic shared by the two forms of the prep work (the launch of its own below and the prep role inside the scan
// launch), so that both give the same bits.
// conv + SiLU of one bf16 channel pair: r[m] = the pre-conv pair m steps back in time, wl[e][m] its weight
__device__ __forceinline__ uint32_t prep_conv_pair(const float (&wl)[2][4], const float (&bias)[2], const uint32_t (&r)[4]) {
    float v0 = bias[0], v1 = bias[1];
#pragma unroll
    for (int m = 3; m >= 0; --m) {
        v0 = fmaf(wl[0][m], bf16_lo(r[m]), v0);
        v1 = fmaf(wl[1][m], bf16_hi(r[m]), v1);
    }
    return pack_bf16(silu_fast(v0), silu_fast(v1));
}
// softplus(dt + bias) = max(v, 0) + log1p(exp(-|v|)) with the fast exponential and logarithm: log1p by its series where 1 + e
// would round e away (e < 2^-7: error below e^4 / 4), by log(1 + e) elsewhere.  Relative error of Delta about 1e-6, far inside
// what the bf16 path needs.
__device__ __forceinline__ float prep_delta(__nv_bfloat16 dt, float dt_bias) {
    const float v = __bfloat162float(dt) + dt_bias;
    const float e = __expf(-fabsf(v));
    const float l = e < 0.0078125f ? e * fmaf(e, fmaf(e, 0.33333334f, -0.5f), 1.f) : __logf(1.f + e);
    return fmaxf(v, 0.f) + l;
}
// One warp, one head, one 128-token chunk: d[r * ld] = Delta of physical chunk row r.  Writes Lambda (inclusive cumulative
// Delta A in the direction's time order, log2 units) to dl[0..Q) and Lambda' = Lambda - log2 Delta to dl[Lp..Lp + Q).
__device__ __forceinline__ void prep_lambda_head(const float *d_col, int ld, float A_log, bool rev, int lane, float *dl, int Lp) {
    const float Ah = -expf(A_log) * 1.4426950408889634f;
    float d[4], cum[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int tau = 4 * lane + e, r = rev ? Q - 1 - tau : tau;
        d[e] = d_col[r * ld];
    }
    cum[0] = d[0] * Ah; cum[1] = fmaf(d[1], Ah, cum[0]); cum[2] = fmaf(d[2], Ah, cum[1]); cum[3] = fmaf(d[3], Ah, cum[2]);
    float run = cum[3];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const float up = __shfl_up_sync(0xffffffffu, run, off);
        if (lane >= off) run += up;
    }
    const float base = run - cum[3];                             // sum over the lanes before this one
    float lam[4], lamp[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) { lam[e] = base + cum[e]; lamp[e] = lam[e] - __log2f(d[e]); }    // Delta = 0 (padding): Lambda' = +inf
    const int rlo = rev ? Q - 4 - 4 * lane : 4 * lane;           // lowest physical row of this lane's four
    const float4 v0 = rev ? make_float4(lam[3], lam[2], lam[1], lam[0]) : make_float4(lam[0], lam[1], lam[2], lam[3]);
    const float4 v1 = rev ? make_float4(lamp[3], lamp[2], lamp[1], lamp[0]) : make_float4(lamp[0], lamp[1], lamp[2], lamp[3]);
    *reinterpret_cast<float4 *>(dl + rlo) = v0;
    *reinterpret_cast<float4 *>(dl + Lp + rlo) = v1;
}

// --------------------------------------------------------------------------------------------------
// Launch 1: B', C' (bf16) and Lambda, Lambda' (fp32, log2 units).  A CTA takes one quarter of one physical chunk of one
// (direction, batch row): 32 of its rows for B' and C', 16 of every 64 heads for the decays.  The work per CTA is a
// chain of dependent memory round trips, so many small CTAs per SM hide it better than few large ones.
// --------------------------------------------------------------------------------------------------
constexpr int PREP_PARTS = 4, PREP_THREADS = 128, PREP_HEADS = 64 / PREP_PARTS;
constexpr int QB = Q / PREP_PARTS;          // tokens per sub-chunk of the short-block kernel = rows of one prep CTA
constexpr int BCT_LD = N / 2 + 4;           // row pitch (32-bit words) of the prep CTA's B' / C' tile: 16-byte rows, conflict-free ldmatrix
static_assert(QB == 32, "one prep CTA covers exactly one sub-chunk");

__device__ __forceinline__ void ldmatrix_x4(uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3, const void *p) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(smem_u32(p)));
}
__device__ __forceinline__ void ldmatrix_x2(uint32_t &r0, uint32_t &r1, const void *p) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0, %1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(smem_u32(p)));
}
// D (16 x 8, fp32) += A (16 x 16, row-major) B (16 x 8, column-major), bf16 operands
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// One unit of prep work, by a group of PREP_THREADS threads (tid = index in the group; `bar` = the group's named barrier): part
// `part` of chunk pc of (direction, batch row): QB rows of B' and C', PREP_HEADS of every 64 heads for the decays.
// dsm: the group's [Q][PREP_HEADS + 1] floats.  Sb != NULL (short-block mode, with bct = the group's [2][QB][BCT_LD] words): the unit
// also writes S[i][j] = C'_i . B'_j over its rows, fp32, to Sb[seq][pc * PREP_PARTS + part][QB][QB].
// what: PREP_BC = the B', C' (and S) half of the unit, PREP_DECAY = its decays, or both.
constexpr int PREP_BC = 1, PREP_DECAY = 2;
__device__ __forceinline__ void prep_unit(const SsdArgs &a, __nv_bfloat16 *__restrict__ Bp, __nv_bfloat16 *__restrict__ Cp, float *__restrict__ dA,
                                          float *__restrict__ Sb, int dir, int b, int pc, int part, int tid, int bar, float *dsm,
                                          uint32_t (*bct)[QB][BCT_LD], int what) {
    const bool rev = dir == 1;
    const int L = a.L, k = a.k;
    const ScanDir &w = a.dir[dir];
    const int64_t seq = (int64_t)dir * a.B + b;
    const __nv_bfloat16 *zx = a.zx + ((int64_t)(a.zx_tied ? 0 : dir) * a.B + b) * L * a.d_in_proj;
    const int r0 = pc * Q;
    const bool has_bias = (a.flags & DM_FLAG_CONV_BIAS) && w.conv_b;

    // ---- B and C channels: thread = channel pair, over this unit's block of 32 rows; the 35-row window is loaded up front
    // (a block past the end of the sequence has nothing to write and nobody reads its S)
    const bool bc_live = (what & PREP_BC) && r0 + part * 32 < L;
    if (bc_live) {
        const int cp = tid, rg = part;
        const bool isC = cp >= N / 2;
        const int pi = cp & (N / 2 - 1);                                 // pair index inside B or C
        const bool valid = 2 * pi < a.Nr;                                // beyond the model's d_state: zero padding
        const int cc = a.d_inner + (isC ? a.Nr : 0) + (valid ? 2 * pi : 0);   // conv channel of the pair's first member
        const __nv_bfloat16 *cw = static_cast<const __nv_bfloat16 *>(w.conv_w) + (int64_t)cc * k;
        float wl[2][4];                                                  // wl[e][m]: weight of the row m steps back in time
#pragma unroll
        for (int e = 0; e < 2; ++e)
#pragma unroll
            for (int m = 0; m < 4; ++m) wl[e][m] = (m < k && valid) ? __bfloat162float(cw[e * k + k - 1 - m]) : 0.f;
        float bias[2] = {0.f, 0.f};
        if (has_bias && valid) {
            bias[0] = __bfloat162float(static_cast<const __nv_bfloat16 *>(w.conv_b)[cc]);
            bias[1] = __bfloat162float(static_cast<const __nv_bfloat16 *>(w.conv_b)[cc + 1]);
        }
        const uint32_t *col = reinterpret_cast<const uint32_t *>(zx + a.d_inner + cc);      // 4-byte aligned: all widths are even
        const int64_t ld32 = a.d_in_proj / 2;
        const int first = rev ? r0 + rg * 32 + 31 : r0 + rg * 32, step = rev ? -1 : 1;        // first-in-time row of the block
        const uint32_t *cin = (!rev && a.conv_in) ? reinterpret_cast<const uint32_t *>(a.conv_in + (int64_t)b * (k - 1) * a.conv_ch + cc) : nullptr;
        uint32_t raw[35];
#pragma unroll
        for (int i = 0; i < 35; ++i) {
            const int t = first + (i - 3) * step;
            raw[i] = (valid && t >= 0 && t < L) ? __ldg(col + (int64_t)t * ld32) : 0u;
            if (valid && cin && t < 0 && k - 1 + t >= 0) raw[i] = __ldg(cin + (int64_t)(k - 1 + t) * (a.conv_ch / 2));    // carried rows
        }
        __nv_bfloat16 *dst = (isC ? Cp : Bp) + 2 * pi + seq * L * N;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const int t = first + i * step;
            const uint32_t win[4] = {raw[i + 3], raw[i + 2], raw[i + 1], raw[i]};
            const uint32_t pk = prep_conv_pair(wl, bias, win);
            if (t < L) *reinterpret_cast<uint32_t *>(dst + (int64_t)t * N) = pk;
            if (Sb) bct[isC ? 1 : 0][rev ? QB - 1 - i : i][pi] = pk;          // row of the tile = physical row inside the block
        }
    }
    if (Sb && bc_live) {
        // S = C' B'^T of this block's 32 rows on the legacy tensor path: warp = 16 rows i x 16 columns j, K = d_state
        named_sync(bar, PREP_THREADS);
        const int warp = tid >> 5, lane = tid & 31;
        const int mt = warp & 1, nh = warp >> 1;
        float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
        for (int k0 = 0; k0 < N; k0 += 16) {
            uint32_t a0, a1, a2, a3;
            ldmatrix_x4(a0, a1, a2, a3, &bct[1][16 * mt + (lane & 15)][(k0 + (lane >> 4) * 8) / 2]);
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
                uint32_t b0, b1;
                ldmatrix_x2(b0, b1, &bct[0][16 * nh + 8 * nt + (lane & 7)][(k0 + ((lane >> 3) & 1) * 8) / 2]);
                mma_bf16_16816(acc[nt], a0, a1, a2, a3, b0, b1);
            }
        }
        float *S = Sb + (seq * (a.nch * PREP_PARTS) + pc * PREP_PARTS + part) * (QB * QB);
        const int gr = lane >> 2, qc = lane & 3;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            const int col = 16 * nh + 8 * nt + 2 * qc, row = 16 * mt + gr;
            *reinterpret_cast<float2 *>(S + row * QB + col) = make_float2(acc[nt][0], acc[nt][1]);
            *reinterpret_cast<float2 *>(S + (row + 8) * QB + col) = make_float2(acc[nt][2], acc[nt][3]);
        }
    }
    // ---- Delta, then the inclusive cumulative log-decay of every head in the direction's time order
    if (!(what & PREP_DECAY)) return;
    for (int h0 = 0; h0 < a.H; h0 += 64) {
        named_sync(bar, PREP_THREADS);
#pragma unroll 4
        for (int i = 0; i < Q * PREP_HEADS / PREP_THREADS; ++i) {
            const int idx = tid + PREP_THREADS * i, hh = idx % PREP_HEADS, r = idx / PREP_HEADS, t = r0 + r, h = h0 + part * PREP_HEADS + hh;
            dsm[r * (PREP_HEADS + 1) + hh] = (t < L && h < a.H) ? prep_delta(zx[(int64_t)t * a.d_in_proj + a.d_inner + a.conv_ch + h], w.dt_bias[h]) : 0.f;
        }
        named_sync(bar, PREP_THREADS);
        const int warp = tid >> 5, lane = tid & 31;
        for (int hh = warp; hh < PREP_HEADS && h0 + part * PREP_HEADS + hh < a.H; hh += PREP_THREADS / 32) {
            const int h = h0 + part * PREP_HEADS + hh;
            prep_lambda_head(dsm + hh, PREP_HEADS + 1, w.A_log[h], rev, lane, dA + ((seq * a.H + h) * 2) * a.Lp + r0, a.Lp);
        }
    }
}

// grid.x covers the chunks the direction visits first: blockIdx.x / PREP_PARTS is the chunk's index in time order.  With split set (short
// blocks, where the launch is a handful of CTAs and its latency is what counts) grid.x is twice that: the first half of the CTAs take the
// B', C', S halves of the units, the second half their decays.
__global__ void __launch_bounds__(PREP_THREADS)
ssd_prep_kernel(const SsdArgs a, __nv_bfloat16 *__restrict__ Bp, __nv_bfloat16 *__restrict__ Cp, float *__restrict__ dA, float *__restrict__ Sb,
                int dir0, int split) {
    __shared__ float dsm[Q * (PREP_HEADS + 1)];
    __shared__ __align__(16) uint32_t bct[2][QB][BCT_LD];     // short-block mode: this CTA's rows of B' ([0]) and C' ([1]) as bf16 pairs
    const int units = split ? gridDim.x / 2 : gridDim.x, u = blockIdx.x % units;
    const int what = !split ? (PREP_BC | PREP_DECAY) : blockIdx.x < units ? PREP_BC : PREP_DECAY;
    const int dir = dir0 + blockIdx.z, c = u / PREP_PARTS;
    prep_unit(a, Bp, Cp, dA, Sb, dir, blockIdx.y, dir == 1 ? a.nch - 1 - c : c, u % PREP_PARTS, threadIdx.x, 0, dsm, bct, what);
}

// --------------------------------------------------------------------------------------------------
// The same prep work as a role inside the scan launch.  When the scan has fewer CTAs than the GPU has SMs (one long
// sequence: 2 H CTAs), the launch is widened by `nprep` CTAs; the CTAs that start first take the prep role (a ticket
// from an atomic counter decides, so the role never waits for a CTA that has not been scheduled), work through the
// (batch row, chunk, direction) items in the order the scan consumes them and release one flag per item; the scan CTAs'
// load warps acquire the flag of a chunk before they fetch its B', C', Lambda through TMA (followed by a proxy fence: the
// data were written through the generic proxy).  All threads of a prep CTA work on one item: its 131 rows of the B and C
// columns and its dt columns are fetched with every load in flight at once -- the next item's while the current one is
// computed -- and staged in shared memory; then every thread filters one channel pair over a run of rows and every warp
// scans heads.  With two directions nprep is even, so that a CTA's items all belong to one direction and its conv
// weights are read once.
// --------------------------------------------------------------------------------------------------
struct PrepJob {
    __nv_bfloat16 *Bp, *Cp;
    float *dA;
    int *sync;          // [0]: ticket counter, [1 + seq * nch + pc]: item flags; zeroed before the launch.  NULL: no fused prep
    int nprep, ndir;
    int c0;             // chunks before this one (in time order) come from a prep launch of their own that ran before the scan launch
};
// 16-byte asynchronous copy global -> shared; src_bytes = 16, or 0 to fill the destination with zeros (src must still be a valid address)
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

constexpr int PREP_SEG = 7, PREP_SEG_ROWS = (Q + PREP_SEG - 1) / PREP_SEG;     // row runs per channel pair
// shared memory of a prep CTA: two stages of { rows [Q + 3][N] words, dt [Q][64] bf16 }, then Delta [Q][65] floats
constexpr uint32_t PREP_RAW_BYTES = (Q + 3) * N * 4, PREP_DT_BYTES = Q * 64 * 2, PREP_STAGE = PREP_RAW_BYTES + PREP_DT_BYTES;
constexpr uint32_t PREP_SMEM = 2 * PREP_STAGE + Q * 65 * 4;

struct PrepItem { int dir, b, pc; };
__device__ __forceinline__ PrepItem prep_item(const SsdArgs &a, const PrepJob &pj, int it, int dir0) {
    PrepItem r;
    r.dir = dir0 + it % pj.ndir;
    const int nc = a.nch - pj.c0, c = pj.c0 + (it / pj.ndir) % nc;
    r.b = it / (pj.ndir * nc);
    r.pc = r.dir == 1 ? a.nch - 1 - c : c;
    return r;
}
// Asynchronous copies of the item's rows (tile row rr = physical row r0 - 3 + rr for ->, history first; r0 + rr for <-,
// history last; rows and columns that do not exist are filled with zeros) and of the dt columns of the first 64 heads.
__device__ __forceinline__ void prep_fetch(const SsdArgs &a, const PrepItem &q, uint8_t *stage, bool dt_vec) {
    const int tid = threadIdx.x, L = a.L, k = a.k, r0 = q.pc * Q;
    const bool rev = q.dir == 1;
    const __nv_bfloat16 *zx = a.zx + ((int64_t)(a.zx_tied ? 0 : q.dir) * a.B + q.b) * L * a.d_in_proj;
    for (int u = tid; u < (Q + 3) * 32; u += NTHREADS) {
        const int rr = u >> 5, c16 = u & 31, ch = (c16 & 15) * 8;
        const int pr = rev ? r0 + rr : r0 - 3 + rr;
        const __nv_bfloat16 *src = zx;
        uint32_t nb = 0;
        if (ch < a.Nr) {                                                       // beyond the model's d_state: zero padding
            const int cc = a.d_inner + ((c16 >> 4) ? a.Nr : 0) + ch;           // conv channel
            if (pr >= 0 && pr < L) { src = zx + (int64_t)pr * a.d_in_proj + a.d_inner + cc; nb = 16; }
            else if (pr < 0 && !rev && a.conv_in && k - 1 + pr >= 0) {         // rows before the sequence: the carried conv state
                src = a.conv_in + ((int64_t)q.b * (k - 1) + (k - 1 + pr)) * a.conv_ch + cc; nb = 16;
            }
        }
        cp_async16(stage + rr * (N * 4) + c16 * 16, src, nb);
    }
    if (dt_vec)
        for (int u = tid; u < Q * 8; u += NTHREADS) {
            const int r = u >> 3, h8 = (u & 7) * 8;
            const bool ok = r0 + r < L && h8 < a.H;
            cp_async16(stage + PREP_RAW_BYTES + u * 16, ok ? zx + (int64_t)(r0 + r) * a.d_in_proj + a.d_inner + a.conv_ch + h8 : zx, ok ? 16 : 0);
        }
}

__device__ __noinline__ void prep_role(const SsdArgs &a, const PrepJob &pj, int first, int dir0, uint8_t *smem) {
    static_assert(PREP_SEG * 128 == NTHREADS && PREP_SMEM <= OFF_MISC, "prep role: thread and shared-memory layout");
    float *dsm = reinterpret_cast<float *>(smem + 2 * PREP_STAGE);              // [Q][65] Delta of one tile of 64 heads
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int L = a.L, k = a.k, n_items = pj.ndir * a.B * (a.nch - pj.c0);
    if (first >= n_items) return;
    // 16-byte copies of eight heads' dt: the dt columns start on a 16-byte boundary and the head count is a multiple of 8
    const bool dt_vec = (a.d_inner + a.conv_ch) % 8 == 0 && a.H % 8 == 0;
    prep_fetch(a, prep_item(a, pj, first, dir0), smem, dt_vec);
    // conv weights of this thread's channel pair: every item of this CTA has the direction of the first one
    const int dirc = dir0 + first % pj.ndir;
    const ScanDir &w = a.dir[dirc];
    const bool rev = dirc == 1;
    const int pi = tid & 127, seg = tid >> 7, pp = pi & 63;
    const bool isC = pi >= 64, valid = 2 * pp < a.Nr;
    float wl[2][4], bias[2] = {0.f, 0.f};
    {
        const int cc = a.d_inner + (isC ? a.Nr : 0) + (valid ? 2 * pp : 0);
        const __nv_bfloat16 *cw = static_cast<const __nv_bfloat16 *>(w.conv_w) + (int64_t)cc * k;
#pragma unroll
        for (int e = 0; e < 2; ++e)
#pragma unroll
            for (int m = 0; m < 4; ++m) wl[e][m] = (m < k && valid) ? __bfloat162float(cw[e * k + k - 1 - m]) : 0.f;
        if ((a.flags & DM_FLAG_CONV_BIAS) && w.conv_b && valid) {
            bias[0] = __bfloat162float(static_cast<const __nv_bfloat16 *>(w.conv_b)[cc]);
            bias[1] = __bfloat162float(static_cast<const __nv_bfloat16 *>(w.conv_b)[cc + 1]);
        }
    }
    int stg = 0;
    for (int it = first; it < n_items; it += pj.nprep, stg ^= 1) {
        const PrepItem q = prep_item(a, pj, it, dir0);
        const int r0 = q.pc * Q;
        const int64_t seq = (int64_t)q.dir * a.B + q.b;
        const __nv_bfloat16 *zx = a.zx + ((int64_t)(a.zx_tied ? 0 : q.dir) * a.B + q.b) * L * a.d_in_proj;
        const uint32_t *rawt = reinterpret_cast<const uint32_t *>(smem + stg * PREP_STAGE);
        const __nv_bfloat16 *dtt = reinterpret_cast<const __nv_bfloat16 *>(smem + stg * PREP_STAGE + PREP_RAW_BYTES);
        cp_async_wait_all();
        __syncthreads();                           // this item's tiles have landed; the previous item's readers are done with the other stage and with dsm
        if (it + pj.nprep < n_items) prep_fetch(a, prep_item(a, pj, it + pj.nprep, dir0), smem + (stg ^ 1) * PREP_STAGE, dt_vec);      // in flight while this item is computed
        // ---- conv + SiLU: thread = (channel pair, run of rows)
        {
            __nv_bfloat16 *dst = (isC ? pj.Cp : pj.Bp) + 2 * pp + seq * L * N;
            const int i0 = seg * PREP_SEG_ROWS, i1 = min(Q, i0 + PREP_SEG_ROWS);
            for (int i = i0; i < i1; ++i) {
                const uint32_t *col = rawt + pi + (rev ? i : i + 3) * N;           // the row itself; m steps back in time = m rows further (<-) or back (->)
                const int st = rev ? N : -N;
                const uint32_t win[4] = {col[0], col[st], col[2 * st], col[3 * st]};
                const uint32_t pk = prep_conv_pair(wl, bias, win);
                if (r0 + i < L) *reinterpret_cast<uint32_t *>(dst + (int64_t)(r0 + i) * N) = pk;
            }
        }
        // ---- Delta and the cumulative log-decay, 64 heads at a time
        for (int h0 = 0; h0 < a.H; h0 += 64) {
            if (h0 > 0) __syncthreads();                                       // the previous head tile's scans are done with dsm
            for (int idx = tid; idx < Q * 64; idx += NTHREADS) {
                const int hh = idx & 63, r = idx >> 6, t = r0 + r, h = h0 + hh;
                float d = 0.f;
                if (t < L && h < a.H)
                    d = prep_delta((h0 == 0 && dt_vec) ? dtt[idx] : zx[(int64_t)t * a.d_in_proj + a.d_inner + a.conv_ch + h], w.dt_bias[h]);
                dsm[r * 65 + hh] = d;
            }
            __syncthreads();
            for (int hh = warp; hh < 64 && h0 + hh < a.H; hh += NTHREADS / 32) {
                const int h = h0 + hh;
                prep_lambda_head(dsm + hh, 65, w.A_log[h], rev, lane, pj.dA + ((seq * a.H + h) * 2) * a.Lp + r0, a.Lp);
            }
        }
        // ---- publish the item
        __threadfence();
        __syncthreads();
        if (tid == 0) atomicExch(pj.sync + 1 + seq * a.nch + q.pc, PREP_PARTS);
    }
}

// --------------------------------------------------------------------------------------------------
// Launch 2: the chunked scan.
// --------------------------------------------------------------------------------------------------
// HM = 0: heads of P = 64 channels, one per CTA.
// HM = 1 (HALFP): the model's headdim is P / 2 and the CTA carries one head.  It still moves 64-channel tiles (the second half is
// padding that never leaves it), but the conv, the state hand-over and the epilogue work on the 32 real channels only, split over
// the same threads; the padded halves of the w o x' tile and of the state copy are zeroed once, so the padded state columns stay zero.
// HM = 2 (PAIR): headdim P / 2 and an even number of heads: the CTA carries two neighbouring heads in its 64 channels.  They share
// the B', C' tiles and S; each has its own Lambda, Lambda' (two per stage), its own mask W (mask group g builds head g's W, the second
// one in the TMEM columns the other modes leave unused) and its own 32-wide Ya = W x' product; Yb, St, the state (two 32-column halves)
// and the tiles are those of a 64-channel head, with the decay factors taken per column half.
template <int HM>
__global__ void __launch_bounds__(NTHREADS, 1)
ssd_scan_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_z,
                const __grid_constant__ CUtensorMap map_b, const __grid_constant__ CUtensorMap map_c,
                const __grid_constant__ CUtensorMap map_g, const __grid_constant__ SsdArgs a, const __grid_constant__ PrepJob pj, int dir0, int *status) {
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte aligned base, derived by offsetting the __shared__ array so that accesses stay shared-space loads and stores
    uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    constexpr bool HALFP = HM == 1, PAIR = HM == 2;
    constexpr int NH = PAIR ? 2 : 1;                               // heads per CTA
    constexpr uint32_t DL_STAGE = NH * DL_HEAD;                    // bytes of one (Lambda, Lambda') stage
    Misc *misc = reinterpret_cast<Misc *>(smem + OFF_DL + NDL * DL_STAGE);
    volatile int *abort_flag = &misc->abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    int item = blockIdx.x;                     // (batch row, direction, head or head pair), heads fastest
    if (pj.sync) {
        if (tid == 0) misc->ticket = atomicAdd(pj.sync, 1);
        __syncthreads();
        const int ticket = misc->ticket;
        if (ticket < pj.nprep) { prep_role(a, pj, ticket, dir0, smem); return; }
        item = ticket - pj.nprep;
    }
    const int HC = a.H / NH;                   // CTAs per (batch row, direction)
    const int h = (item % HC) * NH, b = item / (HC * pj.ndir), dir = dir0 + (item / HC) % pj.ndir;     // h: the CTA's (first) head
    const bool rev = dir == 1;
    const int *ready = pj.sync ? pj.sync + 1 + ((int64_t)dir * a.B + b) * a.nch : nullptr;     // per chunk: units of its B', C', Lambda that are in memory
    const int L = a.L, nch = a.nch;
    const int seq = dir * a.B + b;
    const int zseq = a.zx_tied ? b : seq;          // the sequence's rows in the in_proj output (shared by the directions when the projections are tied)
    const ScanDir &w = a.dir[dir];
    const bool norm_on = (a.flags & DM_FLAG_GATED_RMSNORM) != 0;

    if (tid == 0) {
        for (int i = 0; i < NX; ++i) { mbar_init(&misc->full_x[i], 1); mbar_init(&misc->empty_x[i], 1); }
        for (int i = 0; i < NZ; ++i) { mbar_init(&misc->full_z[i], 1); mbar_init(&misc->empty_z[i], 1); }
        for (int i = 0; i < NB; ++i) { mbar_init(&misc->full_b[i], 1); mbar_init(&misc->empty_b[i], 1); }
        for (int i = 0; i < NDL; ++i) { mbar_init(&misc->full_dl[i], 1); mbar_init(&misc->empty_dl[i], 3 * ROLE); }
        mbar_init(&misc->full_c, 1);   mbar_init(&misc->empty_c, 1);
        mbar_init(&misc->xs_full, ROLE);
        mbar_init(&misc->s_full, 1);   mbar_init(&misc->s_empty, ROLE);
        mbar_init(&misc->w_full, ROLE);
        mbar_init(&misc->st_full, 1);  mbar_init(&misc->hs_ready, ROLE);
        mbar_init(&misc->h_full, ROLE);
        mbar_init(&misc->y_full, 1);   mbar_init(&misc->ya_empty, ROLE);
        mbar_init(&misc->yb_empty[0], ROLE); mbar_init(&misc->yb_empty[1], ROLE);
        misc->abort = 0;
        mbar_fence_init();
    }
    const int Pr = a.Pr;                 // channels of this head; the tile's remaining P - Pr columns are padding and never leave the CTA
    if (tid < P) misc->norm_w[tid] = (norm_on && w.norm_w && tid < NH * Pr) ? __bfloat162float(static_cast<const __nv_bfloat16 *>(w.norm_w)[h * Pr + tid]) : 1.f;
    if (warp == 1) tmem_alloc(&misc->tmem_base, TM_COLS);
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem = misc->tmem_base;
    const uint32_t tlane = tmem + ((uint32_t)((warp & 3) * 32) << 16);     // this warp's TMEM lane quarter
    const float *dA_head = a.dA + (((int64_t)seq * a.H + h) * 2) * a.Lp;
    auto WAIT = [&](uint64_t *bar, uint32_t parity) { return mbar_wait(bar, parity, abort_flag, status); };
    auto WAIT2 = [&](uint64_t *b1, uint32_t p1, uint64_t *b2, uint32_t p2) { return mbar_wait2(b1, p1, b2, p2, abort_flag, status); };
    auto WAIT3 = [&](uint64_t *b1, uint32_t p1, uint64_t *b2, uint32_t p2, uint64_t *b3, uint32_t p3) {
        return mbar_wait3(b1, p1, b2, p2, b3, p3, abort_flag, status);
    };

    if (warp == 0) {
        // ============================================================ TMA: x tile (+halo) and Lambda, Lambda'
        if (lane == 0) {
            int issued = 0;
            for (int c = 0; c < nch; ++c) {
                const int sx = c % NX, sd = c % NDL, pc = rev ? nch - 1 - c : c;
                // the chunk's Lambda are in memory (fused prep): asked first, so that the flag's round trip to L2 hides behind the wait for a free stage
                if (ready && c >= pj.c0 && !flag_wait<PREP_PARTS>(ready + pc, abort_flag, status)) break;
                if (!WAIT2(&misc->empty_x[sx], ((c / NX) & 1) ^ 1, &misc->empty_dl[sd], ((c / NDL) & 1) ^ 1)) break;
                mbar_expect_tx(&misc->full_x[sx], XTILE);
                tma_load_3d(smem + OFF_X + sx * XTILE, &map_x, a.d_inner + h * Pr, rev ? pc * Q : pc * Q - HALO, zseq, &misc->full_x[sx]);
                mbar_expect_tx(&misc->full_dl[sd], DL_STAGE);
#pragma unroll
                for (int hh = 0; hh < NH; ++hh) {                  // stage layout: [head][Lambda | Lambda'][Q]
                    bulk_load(smem + OFF_DL + sd * DL_STAGE + hh * DL_HEAD, dA_head + (int64_t)hh * 2 * a.Lp + pc * Q, Q * 4, &misc->full_dl[sd]);
                    bulk_load(smem + OFF_DL + sd * DL_STAGE + hh * DL_HEAD + Q * 4, dA_head + (int64_t)hh * 2 * a.Lp + a.Lp + pc * Q, Q * 4, &misc->full_dl[sd]);
                }
                issued = c + 1;
            }
            if (*abort_flag)            // aborting: bounded wait for the loads still in flight
                for (int c = max(0, issued - NDL); c < issued; ++c) {
                    if (c >= issued - NX) mbar_wait_quiet(&misc->full_x[c % NX], (c / NX) & 1, 100000000ull);
                    mbar_wait_quiet(&misc->full_dl[c % NDL], (c / NDL) & 1, 100000000ull);
                }
        }
    } else if (warp == 2) {
        // ============================================================ TMA: z tile
        if (lane == 0) {
            int issued = 0;
            for (int c = 0; c < nch; ++c) {
                const int sz = c % NZ, pc = rev ? nch - 1 - c : c;
                if (!WAIT(&misc->empty_z[sz], ((c / NZ) & 1) ^ 1)) break;
                mbar_expect_tx(&misc->full_z[sz], T16);
                tma_load_3d(smem + OFF_Z + sz * T16, &map_z, h * Pr, pc * Q, zseq, &misc->full_z[sz]);
                issued = c + 1;
            }
            if (*abort_flag)
                for (int c = max(0, issued - NZ); c < issued; ++c) mbar_wait_quiet(&misc->full_z[c % NZ], (c / NZ) & 1, 100000000ull);
        }
    } else if (warp == 3) {
        // ============================================================ TMA: B' and C' tiles
        if (lane == 0) {
            int issued_b = 0, issued_c = 0;
            for (int c = 0; c < nch; ++c) {
                const int sb = c % NB, pc = rev ? nch - 1 - c : c;
                if (ready && c >= pj.c0 && !flag_wait<PREP_PARTS>(ready + pc, abort_flag, status)) break;          // the chunk's B', C' are in memory
                if (!WAIT(&misc->empty_b[sb], ((c / NB) & 1) ^ 1)) break;
                mbar_expect_tx(&misc->full_b[sb], 2 * T16);
                tma_load_3d(smem + OFF_B + sb * 2 * T16, &map_b, 0, pc * Q, seq, &misc->full_b[sb]);
                tma_load_3d(smem + OFF_B + sb * 2 * T16 + T16, &map_b, 64, pc * Q, seq, &misc->full_b[sb]);
                issued_b = c + 1;
                if (!WAIT(&misc->empty_c, (c & 1) ^ 1)) break;
                mbar_expect_tx(&misc->full_c, 2 * T16);
                tma_load_3d(smem + OFF_C, &map_c, 0, pc * Q, seq, &misc->full_c);
                tma_load_3d(smem + OFF_C + T16, &map_c, 64, pc * Q, seq, &misc->full_c);
                issued_c = c + 1;
            }
            if (*abort_flag) {
                for (int c = max(0, issued_b - NB); c < issued_b; ++c) mbar_wait_quiet(&misc->full_b[c % NB], (c / NB) & 1, 100000000ull);
                if (issued_c > 0) mbar_wait_quiet(&misc->full_c, (issued_c - 1) & 1, 100000000ull);
            }
        }
    } else if (warp == 1) {
        // ============================================================ MMA issuer
        // Order per iteration: S(c), Yb(c), Ya(c-1), St(c).  S(c) goes out as soon as the mask of chunk c-1 has read
        // S(c-1); Yb(c) follows at once (its accumulator is double-buffered, so it does not wait for the epilogue of
        // chunk c-1), which frees the single C' buffer early enough for the next chunk's load.
        // Half-width heads: the whole warp walks the loop and waits, one elected lane issues the products and their
        // commits (the operand descriptors then live in uniform registers and a product takes a third of the time to
        // issue), and Ya(c-1) goes out before Yb(c) so that the mask of chunk c starts earlier.  With full-width heads
        // the conv groups are the longer chain and both changes only take issue slots from them at the wrong time
        // (measured 5 % slower), so there one lane runs the loop and Ya(c-1) follows Yb(c).
        auto mma_role = [&](const bool leader) {
            // low halves of the operand descriptors; a K step of 16 advances a K-major operand by 32 bytes inside its
            // 64-wide tile (+2) or to the next tile (+T16/16), an MN-major operand by 16 rows (+2048/16)
            const uint32_t dH = desc_lo_mn(smem_u32(smem + OFF_H), T16), dXs = desc_lo_mn(smem_u32(smem + OFF_XS), T16);
            const uint32_t dC = desc_lo_k(smem_u32(smem + OFF_C));
            const uint32_t dBk0 = desc_lo_k(smem_u32(smem + OFF_B)), dBm0 = desc_lo_mn(smem_u32(smem + OFF_B), T16);
            const uint32_t dX0 = desc_lo_mn(smem_u32(smem + OFF_X) + (rev ? 0 : HALO * 128), T16);
            constexpr uint32_t I128 = idesc_bf16(128, 128, 0, 0), I64 = idesc_bf16(128, 64, 0, 1), I64T = idesc_bf16(128, 64, 1, 1);
            constexpr uint32_t I32 = idesc_bf16(128, 32, 0, 1);
            auto issue_ya = [&](int c) -> bool {       // Ya = W x'  (A = W from TMEM, B = x' [j][p] MN-major)
                const int sx = c % NX;
                if (!WAIT2(&misc->w_full, c & 1, &misc->ya_empty, (c & 1) ^ 1)) return false;
                fence_after();
                const uint32_t dX = dX0 + (uint32_t)sx * (XTILE >> 4);
                if constexpr (PAIR) {
                    // two products of 32 channels: head 0 = W x'[:, 0:32], head 1 = W1 x'[:, 32:64] (the operand starts 64 bytes into the 128-byte rows)
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        if (kk == 0) { if (leader) umma_ts<0>(tmem + TM_YA, tmem + TM_W, dX, I32); }
                        else if (leader) umma_ts<1>(tmem + TM_YA, tmem + TM_W + 8 * kk, dX + kk * 128, I32);
                    }
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        if (kk == 0) { if (leader) umma_ts<0>(tmem + TM_YA + 32, tmem + TM_W1, dX + 4, I32); }
                        else if (leader) umma_ts<1>(tmem + TM_YA + 32, tmem + TM_W1 + 8 * kk, dX + kk * 128 + 4, I32);
                    }
                } else {
                    if (leader) umma_ts<0>(tmem + TM_YA, tmem + TM_W, dX, I64);
#pragma unroll
                    for (int kk = 1; kk < 8; ++kk) if (leader) umma_ts<1>(tmem + TM_YA, tmem + TM_W + 8 * kk, dX + kk * 128, I64);
                }
                if (leader) umma_commit(&misc->y_full);              // Yb of the same chunk was issued earlier: it has completed as well; also frees W
                if (leader) umma_commit(&misc->empty_x[sx]);
                return true;
            };
            bool ok = true;
            for (int c = 0; c < nch && ok; ++c) {
                const int sb = c % NB;
                const uint32_t par = c & 1;
                const uint32_t dBk = dBk0 + (uint32_t)sb * (2 * T16 >> 4), dBm = dBm0 + (uint32_t)sb * (2 * T16 >> 4);
                // S = C' B'^T  (both K-major in shared memory)
                if (!WAIT3(&misc->full_c, par, &misc->full_b[sb], (c / NB) & 1, &misc->s_empty, par ^ 1)) break;
                fence_after();
                if (leader) umma_ss<0>(tmem + TM_S, dC, dBk, I128);
#pragma unroll
                for (int kk = 1; kk < 8; ++kk) {
                    const uint32_t o = (kk >> 2) * (T16 >> 4) + 2 * (kk & 3);
                    if (leader) umma_ss<1>(tmem + TM_S, dC + o, dBk + o, I128);
                }
                if (leader) umma_commit(&misc->s_full);
                if constexpr (HALFP) { if (c > 0 && !issue_ya(c - 1)) break; }
                // Yb = C' h_in  (A = C' K-major, B = bf16 state [n][p] MN-major) into the buffer the epilogue of chunk c-2 has drained;
                // its completion releases C' (S was issued before it) and the state copy
                const uint32_t tyb = tmem + (par ? TM_YB1 : TM_YB0);
                if (!WAIT2(&misc->h_full, par, &misc->yb_empty[par], ((c >> 1) & 1) ^ 1)) break;
                fence_after();
                if (leader) umma_ss<0>(tyb, dC, dH, I64);
#pragma unroll
                for (int kk = 1; kk < 8; ++kk) if (leader) umma_ss<1>(tyb, dC + (kk >> 2) * (T16 >> 4) + 2 * (kk & 3), dH + kk * 128, I64);
                if (leader) umma_commit(&misc->empty_c);             // also releases the bf16 state copy
                if constexpr (!HALFP) { if (c > 0 && !issue_ya(c - 1)) break; }
                // h += B'^T (w o x')  (A = B' [j][n] MN-major, B = w o x' [j][p] MN-major), onto the state the conv groups have scaled
                if (!WAIT2(&misc->xs_full, par, &misc->hs_ready, par)) break;
                fence_after();
                if (leader) umma_ss<1>(tmem + TM_HS, dBm, dXs, I64T);
#pragma unroll
                for (int kk = 1; kk < 8; ++kk) if (leader) umma_ss<1>(tmem + TM_HS, dBm + kk * 128, dXs + kk * 128, I64T);
                if (leader) umma_commit(&misc->st_full);             // also frees the w o x' buffer
                if (leader) umma_commit(&misc->empty_b[sb]);
                if (c == nch - 1) ok = issue_ya(c);
            }
        };
        if constexpr (HALFP) mma_role(elect_one());
        else if (lane == 0) mma_role(true);
    } else if (warp < 4 + 4 * NWG) {
        // ============================================================ state update; conv + SiLU of the x tile; w o x'
        constexpr int CG = HALFP ? 8 : 16;              // 8-byte column groups (4 channels each) that carry real channels
        constexpr int RB = Q * CG / ROLE;               // rows per thread
        const int t = tid - 4 * 32;                     // 0..ROLE-1
        const int cg = t & (CG - 1), rb = t / CG;       // column group x block of RB rows
        const uint32_t colx = cg >> 1, sub = (cg & 1) * 8;
        f32x2 wl2[2][4], cb2[2];                        // per channel pair; wl2[.][m] multiplies the row m steps back in time
        {
            const bool has_bias = (a.flags & DM_FLAG_CONV_BIAS) && w.conv_b;
            float wl[4][4], cbias[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int ch = min(h * Pr + cg * 4 + e, a.conv_ch - 1);      // padding columns read some valid weight: their results are unused
                const __nv_bfloat16 *cw = static_cast<const __nv_bfloat16 *>(w.conv_w) + (int64_t)ch * a.k;
#pragma unroll
                for (int m = 0; m < 4; ++m) wl[e][m] = m < a.k ? 0.5f * __bfloat162float(cw[a.k - 1 - m]) : 0.f;      // halved: the loop wants v/2
                cbias[e] = has_bias ? 0.5f * __bfloat162float(static_cast<const __nv_bfloat16 *>(w.conv_b)[ch]) : 0.f;
            }
#pragma unroll
            for (int e2 = 0; e2 < 2; ++e2) {
                cb2[e2] = pk2(cbias[2 * e2], cbias[2 * e2 + 1]);
#pragma unroll
                for (int m = 0; m < 4; ++m) wl2[e2][m] = pk2(wl[2 * e2][m], wl[2 * e2 + 1][m]);
            }
        }
        const int first = rev ? rb * RB + RB - 1 : rb * RB, step = rev ? -1 : 1;   // first-in-time chunk row of the block
        const int toff = rev ? 0 : HALO;                                          // tile row = chunk row + toff
        const int srow = t & (WG - 1), sh = t >> 7;      // state row and column half of this thread
        constexpr int SC8 = HALFP ? 2 : 4;              // 8-column groups of the state per thread
        if (HALFP) {                                     // padded halves of w o x' and of the bf16 state copy
            for (int i = t; i < Q * 4; i += ROLE) {
                const int r = i >> 2, c16 = 4 + (i & 3);
                const uint32_t o = r * 128 + ((c16 ^ (r & 7)) << 4);
                *reinterpret_cast<uint4 *>(smem + OFF_XS + o) = make_uint4(0u, 0u, 0u, 0u);
                *reinterpret_cast<uint4 *>(smem + OFF_H + o) = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        // incoming state -> TMEM (fp32)
        {
            const float *h0 = (!rev && a.ssm_in && srow < a.Nr && sh * 32 < NH * Pr) ? a.ssm_in + (((int64_t)b * a.H + h) * Pr) * a.Nr + srow : nullptr;
            uint32_t hs[32];
#pragma unroll
            for (int p = 0; p < 32; ++p) hs[p] = h0 ? __float_as_uint(h0[(int64_t)(sh * 32 + p) * a.Nr]) : 0u;
            tmem_st_x32(tlane + TM_HS + sh * 32, hs);
            tmem_wait_st();
            fence_before();                              // the hand-over (after the group barrier) may read columns another warp stored
        }
        // The fp32 state lives in TMEM and St accumulates onto it: before chunk c's St is issued, the state entering the
        // chunk is copied to shared memory as bf16 (B operand of Yb) and scaled in place by the chunk's total decay, so
        // that after St it reads h <- 2^(Lambda_last) h + B'^T (w o x').  Thread = state row, half of the columns.
        auto state_prepare = [&](float dec) {
            fence_after();
            const f32x2 dec2 = pk2(dec, dec);
#pragma unroll 1
            for (int c8 = sh * SC8; c8 < sh * SC8 + SC8; ++c8) {   // 8 state columns (one 16-byte chunk of the bf16 copy) at a time
                uint32_t hs[8];
                tmem_ld_x8(tlane + TM_HS + c8 * 8, hs);
                tmem_wait_ld();
                uint32_t hb[4];
#pragma unroll
                for (int e2 = 0; e2 < 4; ++e2) {
                    const f32x2 hv = pk2(__uint_as_float(hs[2 * e2]), __uint_as_float(hs[2 * e2 + 1]));
                    hb[e2] = f2_to_bf2(hv);
                    float lo, hi;
                    upk2(mul2(dec2, hv), lo, hi);
                    hs[2 * e2] = __float_as_uint(lo); hs[2 * e2 + 1] = __float_as_uint(hi);
                }
                tmem_st_x8(tlane + TM_HS + c8 * 8, hs);
                *reinterpret_cast<uint4 *>(smem + OFF_H + srow * 128 + ((c8 ^ (srow & 7)) << 4)) = make_uint4(hb[0], hb[1], hb[2], hb[3]);
            }
            fence_proxy_async();
            tmem_wait_st();
            fence_before();
            mbar_arrive(&misc->hs_ready);
            mbar_arrive(&misc->h_full);
        };
        bool ok = true;
        for (int c = 0; c < nch; ++c) {
            const int sx = c % NX, sd = c % NDL;
            const uint32_t par = c & 1;
            if (ok) ok = WAIT3(&misc->full_x[sx], (c / NX) & 1, &misc->full_dl[sd], (c / NDL) & 1, &misc->st_full, par ^ 1);
            if (!named_all(1, ROLE, ok)) { ok = false; break; }
            // (Lambda, Lambda') of the head whose state columns this thread hands over (two heads per CTA: the column half sh)
            const float *lam = reinterpret_cast<const float *>(smem + OFF_DL + sd * DL_STAGE + (PAIR ? sh : 0) * DL_HEAD), *lamp = lam + Q;
            // St of the previous chunk has completed (so has its Yb, issued before it): hand the state over first, Yb and St wait for it
            state_prepare(ex2f(lam[rev ? 0 : Q - 1]));
            // ---- conv.  The three rows before the block (in time) belong to a neighbour, who overwrites them in
            // place: they are read before the group barrier; the block's own rows are read just before being replaced.
            uint8_t *xt = smem + OFF_X + sx * XTILE;
            f32x2 h1[2], h2[2], h3[2];
            {
                uint2 hr[3];
#pragma unroll
                for (int m = 1; m <= 3; ++m) {
                    const int r = first - m * step + toff;
                    hr[m - 1] = *reinterpret_cast<const uint2 *>(xt + r * 128 + ((colx ^ (r & 7)) << 4) + sub);
                    if (c == 0 && rb == 0 && !rev && a.conv_in)      // rows before the sequence: the carried conv state (zeros beyond it)
                        hr[m - 1] = a.k - 1 - m >= 0
                            ? __ldg(reinterpret_cast<const uint2 *>(a.conv_in + ((int64_t)b * (a.k - 1) + (a.k - 1 - m)) * a.conv_ch + h * Pr + cg * 4))
                            : make_uint2(0u, 0u);
                }
                h1[0] = bf2_to_f2(hr[0].x); h1[1] = bf2_to_f2(hr[0].y);
                h2[0] = bf2_to_f2(hr[1].x); h2[1] = bf2_to_f2(hr[1].y);
                h3[0] = bf2_to_f2(hr[2].x); h3[1] = bf2_to_f2(hr[2].y);
            }
            if (t < NH * Q) {                              // w_j of every head: thread t = (head t / Q, row t % Q); with two heads t / Q == sh
                const int tr = t & (Q - 1);
                misc->wbuf[PAIR ? sh : 0][tr] = ex2f(lam[rev ? 0 : Q - 1] - lamp[tr]);
            }
            mbar_arrive(&misc->empty_dl[sd]);
            named_sync(1, ROLE);                           // halo rows are in registers; wbuf is visible
            // Row j of the block sits at j * 128 + ((colx ^ (j & 7)) << 4) in both tiles; with j & 7 = jx this is
            // ((9 jx) ^ colx) << 4, so one running counter k = 144 jx and one exclusive-or give the offset of every row.
            constexpr int R8 = 8 / RB;                          // blocks per group of eight rows
            const int r8 = (rb / R8) * 8, rlo = (rb % R8) * RB;  // the block starts rlo rows into the eight rows at r8
            uint8_t *bx = xt + (toff + r8) * 128 + sub, *bs = smem + OFF_XS + r8 * 128 + sub;
            const uint8_t *wp = reinterpret_cast<const uint8_t *>(misc->wbuf[PAIR ? cg >> 3 : 0] + rb * RB + (rev ? RB - 1 : 0));      // the head of this thread's channels
            uint32_t k = (uint32_t)(rlo + (rev ? RB - 1 : 0)) * 144u;
#pragma unroll 2
            for (int tau = 0; tau < RB; ++tau) {
                const uint32_t off = k ^ (colx << 4);
                uint2 *xp = reinterpret_cast<uint2 *>(bx + off);
                const uint2 rw = *xp;
                const f32x2 cur[2] = {bf2_to_f2(rw.x), bf2_to_f2(rw.y)};
                const float wj = *reinterpret_cast<const float *>(wp);
                const f32x2 w2 = pk2(wj, wj);
                uint32_t ox[2], os[2];
#pragma unroll
                for (int e2 = 0; e2 < 2; ++e2) {
                    f32x2 hh = fma2(wl2[e2][3], h3[e2], cb2[e2]);          // half of the conv output (weights and bias are halved)
                    hh = fma2(wl2[e2][2], h2[e2], hh); hh = fma2(wl2[e2][1], h1[e2], hh); hh = fma2(wl2[e2][0], cur[e2], hh);
                    // SiLU(v) = v/2 + v/2 tanh(v/2)
                    float ha, hb;
                    upk2(hh, ha, hb);
                    const f32x2 o = fma2(hh, pk2(tanh_fast(ha), tanh_fast(hb)), hh);
                    ox[e2] = f2_to_bf2(o);
                    os[e2] = f2_to_bf2(mul2(o, w2));
                    h3[e2] = h2[e2]; h2[e2] = h1[e2]; h1[e2] = cur[e2];
                }
                *xp = make_uint2(ox[0], ox[1]);
                *reinterpret_cast<uint2 *>(bs + off) = make_uint2(os[0], os[1]);
                k += rev ? -144u : 144u;
                wp += rev ? -4 : 4;
            }
            fence_proxy_async();
            mbar_arrive(&misc->xs_full);
        }
        if (!(ok && WAIT(&misc->st_full, (nch - 1) & 1))) ok = false;     // the last St has landed: TMEM holds the outgoing state
        fence_after();
        if (ok && !rev && a.ssm_out) {
            float *ho = a.ssm_out + (((int64_t)b * a.H + h) * Pr) * a.Nr + srow;
            const int half = sh;
            uint32_t hs[32];
            tmem_ld_x32(tlane + TM_HS + half * 32, hs);          // warp-wide: every lane takes part
            tmem_wait_ld();
            if (srow < a.Nr && half * 32 < NH * Pr) {            // rows beyond the model's d_state and columns beyond the CTA's channels are padding
#pragma unroll
                for (int p = 0; p < 32; ++p) ho[(int64_t)(half * 32 + p) * a.Nr] = __uint_as_float(hs[p]);
            }
        }
    } else if (warp < 4 + 8 * NWG) {
        // ============================================================ mask S -> W
        // The NWG groups share every row: group g takes the 16-column groups gi = g, g + NWG, ... of the mask and the
        // state columns [g, g+1) * P / NWG, so the triangular mask is split evenly between them.
        const int mg = (warp - 4 - 4 * NWG) >> 2;       // group index
        const int row = (tid - (4 + 4 * NWG) * 32) & (WG - 1);      // token row i (mask) / state row n (state)
        const int q = warp & 3;
        // two heads per CTA: group mg builds the whole mask of head h + mg (its own Lambda, D and W columns) instead of half of one mask
        const float Dh = (a.flags & DM_FLAG_D_SKIP) ? w.D[h + (PAIR ? mg : 0)] : 0.f;
        const uint32_t tm_w = (PAIR && mg) ? TM_W1 : TM_W;
        float *cbuf = misc->cbuf[mg][q];
        bool ok = true;
        for (int c = 0; c < nch; ++c) {
            const int sd = c % NDL;
            const uint32_t par = c & 1;
            // the decay factors depend on Lambda only: they are prepared while S of this chunk is still being computed
            if (ok) ok = WAIT(&misc->full_dl[sd], (c / NDL) & 1);
            if (!named_all(3 + mg, WG, ok)) { ok = false; break; }
            const float *lam = reinterpret_cast<const float *>(smem + OFF_DL + sd * DL_STAGE + (PAIR ? mg : 0) * DL_HEAD), *lamp = lam + Q;
            const float li = lam[row];
            // ---- W_ij = S_ij 2^(Lambda_i - Lambda'_j) for j not after i in time, + D on the diagonal; 0 elsewhere.
            // Blocks of 32 x 32: the block on the diagonal takes one exponential per entry; a block before it (in
            // time) uses 2^(Lambda_i - Lambda_ref) * 2^(Lambda_ref - Lambda'_j) with Lambda_ref the last row before this
            // warp's rows -- both exponents are non-positive -- so it costs one exponential per row and per column.
            const int n_off = rev ? 3 - q : q;
            float ri = 1.f;
            if (n_off > 0) {
                const float ref = lam[rev ? 32 * (q + 1) : 32 * q - 1];
                ri = ex2f(li - ref);
                for (int i = 0; i < n_off; ++i) {
                    const int j = (rev ? 32 * (q + 1) : 0) + 32 * i + lane;
                    cbuf[j] = ex2f(ref - lamp[j]);
                }
                __syncwarp();
            }
            const f32x2 ri2 = pk2(ri, ri);
            // validity of the diagonal block's entries as integers: entry jj (0..31) of the block counts iff key(jj) >= 0,
            // and carries the D skip iff key(jj) == 0
            const int ksign = rev ? 1 : -1, kbase = rev ? -(row & 31) : (row & 31);
            if (!WAIT2(&misc->s_full, par, &misc->y_full, par ^ 1)) { ok = false; continue; }
            fence_after();
#pragma unroll 1
            for (int gi = PAIR ? 0 : mg; gi < 8; gi += PAIR ? 1 : NWG) {        // this group's share of the 8 groups of 16 columns
                const int jb = gi >> 1, j0 = gi * 16;
                uint32_t out[8];
                if (rev ? jb > q : jb < q) {
                    uint32_t r[16];
                    tmem_ld_x16(tlane + TM_S + j0, r);
                    tmem_wait_ld();
                    const float4 *cp = reinterpret_cast<const float4 *>(cbuf + j0);
#pragma unroll
                    for (int v4 = 0; v4 < 4; ++v4) {
                        const float4 cv = cp[v4];
                        out[2 * v4] = f2_to_bf2(mul2(mul2(pk2(__uint_as_float(r[4 * v4]), __uint_as_float(r[4 * v4 + 1])), pk2(cv.x, cv.y)), ri2));
                        out[2 * v4 + 1] = f2_to_bf2(mul2(mul2(pk2(__uint_as_float(r[4 * v4 + 2]), __uint_as_float(r[4 * v4 + 3])), pk2(cv.z, cv.w)), ri2));
                    }
                } else if (jb == q) {
                    uint32_t r[16];
                    tmem_ld_x16(tlane + TM_S + j0, r);
                    tmem_wait_ld();
                    const float4 *lp4 = reinterpret_cast<const float4 *>(lamp + j0);
#pragma unroll
                    for (int v4 = 0; v4 < 4; ++v4) {
                        const float4 lp = lp4[v4];
                        const float lpv[4] = {lp.x, lp.y, lp.z, lp.w};
                        float v[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int key = ksign * ((j0 & 31) + 4 * v4 + e) + kbase;
                            const float m = ex2f(key >= 0 ? li - lpv[e] : -INFINITY);      // 2^-inf = 0: no branch around the exponential
                            v[e] = fmaf(__uint_as_float(r[4 * v4 + e]), m, key == 0 ? Dh : 0.f);
                        }
                        out[2 * v4] = pack_bf16(v[0], v[1]);
                        out[2 * v4 + 1] = pack_bf16(v[2], v[3]);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 8; ++i) out[i] = 0u;
                }
                tmem_st_x8(tlane + tm_w + gi * 8, out);
            }
            fence_before();
            mbar_arrive(&misc->s_empty);                 // every read of S has completed (wait::ld above)
            tmem_wait_st();
            fence_before();
            mbar_arrive(&misc->w_full);
            mbar_arrive(&misc->empty_dl[sd]);
        }
    } else {
        // ============================================================ epilogue
        const int eg = (warp - 4 - 8 * NWG) >> 2;       // group index: channels [eg, eg+1) * P / NWG
        const int row = (tid - (4 + 8 * NWG) * 32) & (WG - 1);
        constexpr int EC8 = HALFP ? 2 : 4;              // 8-channel groups per thread
        bool ok = true;
        for (int c = 0; c < nch; ++c) {
            const int sz = c % NZ, sd = c % NDL, pc = rev ? nch - 1 - c : c;
            const uint32_t par = c & 1;
            if (ok) ok = WAIT3(&misc->full_z[sz], (c / NZ) & 1, &misc->full_dl[sd], (c / NDL) & 1, &misc->y_full, par);
            if (!named_all(2, ROLE, ok)) { ok = false; break; }
            fence_after();
            const float *lam = reinterpret_cast<const float *>(smem + OFF_DL + sd * DL_STAGE + (PAIR ? eg : 0) * DL_HEAD);      // two heads per CTA: group eg = head h + eg
            const float ei = ex2f(lam[row]);
            mbar_arrive(&misc->empty_dl[sd]);
            const int t = pc * Q + row;
            uint8_t *zt = smem + OFF_Z + sz * T16;
            const f32x2 ei2 = pk2(ei, ei);
            f32x2 ss2 = pk2(0.f, 0.f);
#pragma unroll 1
            for (int c8 = eg * EC8; c8 < eg * EC8 + EC8; ++c8) {   // 8 channels (one 16-byte chunk of z) at a time
                uint32_t ya[8], yb[8];
                tmem_ld_x8(tlane + TM_YA + c8 * 8, ya);
                tmem_ld_x8(tlane + (par ? TM_YB1 : TM_YB0) + c8 * 8, yb);
                tmem_wait_ld();
                if (c8 == eg * EC8 + EC8 - 1) { fence_before(); mbar_arrive(&misc->ya_empty); mbar_arrive(&misc->yb_empty[par]); }
                uint4 *zp = reinterpret_cast<uint4 *>(zt + row * 128 + ((c8 ^ (row & 7)) << 4));
                const uint4 zv = *zp;
                const uint32_t zw[4] = {zv.x, zv.y, zv.z, zv.w};
                const float4 n0 = *reinterpret_cast<const float4 *>(misc->norm_w + c8 * 8), n1 = *reinterpret_cast<const float4 *>(misc->norm_w + c8 * 8 + 4);
                const f32x2 nw[4] = {pk2(n0.x, n0.y), pk2(n0.z, n0.w), pk2(n1.x, n1.y), pk2(n1.z, n1.w)};
                uint32_t ow[4];
#pragma unroll
                for (int e2 = 0; e2 < 4; ++e2) {
                    const f32x2 y = fma2(ei2, pk2(__uint_as_float(yb[2 * e2]), __uint_as_float(yb[2 * e2 + 1])),
                                         pk2(__uint_as_float(ya[2 * e2]), __uint_as_float(ya[2 * e2 + 1])));
                    const f32x2 g = mul2(y, bf2_to_f2(zw[e2]));          // the z tile holds SiLU(z): the in_proj epilogue applied it
                    ss2 = fma2(g, g, ss2);
                    ow[e2] = f2_to_bf2(mul2(g, nw[e2]));
                }
                if (!HALFP) *zp = make_uint4(ow[0], ow[1], ow[2], ow[3]);
                else if (t < L)                 // half-width head: its 32 channels go out with plain stores, 64 bytes per token
                    *reinterpret_cast<uint4 *>(a.g + ((int64_t)seq * L + t) * a.d_inner + h * Pr + c8 * 8) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
            }
            float ss, ss_hi;
            upk2(ss2, ss, ss_hi);
            ss += ss_hi;
            if (!PAIR && eg == 1) misc->ssq_part[row] = ss;
            fence_proxy_async();
            named_sync(2, ROLE);
            if (PAIR) {                                    // each group's channels are one head
                if (t < L && a.ssq) a.ssq[((int64_t)seq * L + t) * a.H + h + eg] = ss;
            } else if (eg == 0 && t < L && a.ssq) a.ssq[((int64_t)seq * L + t) * a.H + h] = ss + misc->ssq_part[row];
            if (eg == 0 && row == 0) {
                if (!HALFP) {
                    tma_store_3d(&map_g, zt, h * Pr, pc * Q, seq);   // rows past the end of the sequence are clipped
                    bulk_commit();
                    bulk_wait_read0();
                }
                mbar_arrive(&misc->empty_z[sz]);
            }
        }
        if (eg == 0 && row == 0) bulk_wait0();
    }

    // ---------------------------------------------------------------- teardown
    fence_before();
    __syncthreads();
    if (warp == 1) {
        fence_after();
        tmem_dealloc(tmem, TM_COLS);
    }
}

// --------------------------------------------------------------------------------------------------
// Launch 2 for short blocks: sub-chunks of QB = 32 tokens; the four products of a sub-chunk on the legacy tensor path
// (mma.sync m16n8k16, bf16 operands from shared memory through ldmatrix, fp32 accumulators in registers).
// One CTA of 4 * PP threads per (batch row, direction, head of PP channels); per sub-chunk:
//   load    x rows (+3 rows of conv history), C' and B' rows as they are (bf16), S (fp32, from the prep launch): asynchronous
//           16-byte copies, all in flight together; Lambda, Lambda';
//           the incoming state as a bf16 copy [p][n] (from ssm_in, or from the accumulators of the previous sub-chunk)
//   conv    x' = SiLU(conv(x)) and w_j x'_j as bf16 [j][p];   W_ij = S_ij 2^(Lambda_i - Lambda'_j) [+ D on the diagonal] for j not after i, else 0
//   y       Yb = C' h^T (K = d_state), rows scaled by 2^(Lambda_i - Lambda_0), then += W x' (K = 32) into the same accumulators:
//           warp = 16 tokens x 16 channels
//   gate    through shared memory to a (token, 8 channels) layout: g = y SiLU(z), sum of squares, * norm_w, 16-byte stores
//   state   (only if someone will read it) h <- 2^(Lambda_last - Lambda_0) h + (w o x')^T B': warp = 16 channels x 64 states, the
//           fp32 state stays in the accumulators from one sub-chunk to the next
// Lambda_0 is Lambda of the token before the sub-chunk inside the same 128-token chunk of the prep launch (0 at its start).
// --------------------------------------------------------------------------------------------------
constexpr int NLD = N + 8;             // row pitch (bf16) of the C', B' and state tiles: 16-byte rows, conflict-free ldmatrix
constexpr int SLD = QB + 4;            // row pitch (fp32) of S
constexpr int WTL = QB + 8;            // row pitch (bf16) of W
// The tiles only the state update reads (B', w o x') come last: a launch that carries no state out of its single sub-chunk
// (KEEP = false: the denoising passes of block decoding) asks for the bytes before them only.  The fp32 y tile reuses the
// bytes of S and of the raw x rows, both dead once the conv and mask phase is over.
template <int PP> struct BlockSmem {
    static constexpr int XLD = PP + 8;             // row pitch (bf16) of x' and w o x'
    static constexpr size_t ct = 0, ht = ct + QB * NLD * 2, xt = ht + PP * NLD * 2, wt = xt + QB * XLD * 2, ss = wt + QB * WTL * 2,
                            xr = ss + QB * SLD * 4, lam = xr + (QB + 4) * PP * 2, total_nokeep = lam + (2 * QB + 4) * 4,
                            bt = total_nokeep, wxt = bt + QB * NLD * 2, total = wxt + QB * XLD * 2, ys = ss;
    static_assert(ht % 16 == 0 && xt % 16 == 0 && wt % 16 == 0 && ss % 16 == 0 && xr % 16 == 0 && lam % 16 == 0 && bt % 16 == 0 && wxt % 16 == 0, "16-byte tiles");
    static_assert(QB * PP * 4 <= lam - ss, "the y tile fits the bytes of S and the raw x rows");
};
__device__ __forceinline__ void ldmatrix_x4_t(uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3, const void *p) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(smem_u32(p)));
}
__device__ __forceinline__ void ldmatrix_x2_t(uint32_t &r0, uint32_t &r1, const void *p) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(smem_u32(p)));
}

// KEEP: the fp32 state lives in the accumulators (several sub-chunks, or a state to write out); without it the launch is a
// single sub-chunk whose state nobody reads, the accumulators and the update's tiles are gone and more CTAs fit an SM.
template <int PP, bool KEEP>
__global__ void __launch_bounds__(4 * PP, (KEEP ? 192 : 256) / PP)
ssd_block_kernel(const SsdArgs a, const __nv_bfloat16 *__restrict__ Bp, const __nv_bfloat16 *__restrict__ Cp, const float *__restrict__ Sb, int dir0) {
    constexpr int NT = 4 * PP, U8 = PP / 8, MT = PP / 16, XLD = BlockSmem<PP>::XLD, CP2 = PP / 2;
    extern __shared__ __align__(16) uint8_t bsm[];
    __nv_bfloat16 (*Ct)[NLD] = reinterpret_cast<__nv_bfloat16 (*)[NLD]>(bsm + BlockSmem<PP>::ct);      // C' rows [i][n]
    __nv_bfloat16 (*Bt)[NLD] = reinterpret_cast<__nv_bfloat16 (*)[NLD]>(bsm + BlockSmem<PP>::bt);      // B' rows [j][n]               (KEEP only)
    __nv_bfloat16 (*Ht)[NLD] = reinterpret_cast<__nv_bfloat16 (*)[NLD]>(bsm + BlockSmem<PP>::ht);      // incoming state [p][n]
    __nv_bfloat16 (*Xt)[XLD] = reinterpret_cast<__nv_bfloat16 (*)[XLD]>(bsm + BlockSmem<PP>::xt);      // x' [j][p]
    __nv_bfloat16 (*WXt)[XLD] = reinterpret_cast<__nv_bfloat16 (*)[XLD]>(bsm + BlockSmem<PP>::wxt);    // w_j x'_j [j][p]              (KEEP only)
    __nv_bfloat16 (*Wt)[WTL] = reinterpret_cast<__nv_bfloat16 (*)[WTL]>(bsm + BlockSmem<PP>::wt);      // W [i][j]
    __nv_bfloat16 (*xr)[PP] = reinterpret_cast<__nv_bfloat16 (*)[PP]>(bsm + BlockSmem<PP>::xr);        // raw x rows and conv history
    float (*ys)[PP] = reinterpret_cast<float (*)[PP]>(bsm + BlockSmem<PP>::ys);                        // the sub-chunk's y (over S and the raw rows)
    float (*Ss)[SLD] = reinterpret_cast<float (*)[SLD]>(bsm + BlockSmem<PP>::ss);
    float *lam = reinterpret_cast<float *>(bsm + BlockSmem<PP>::lam), *lamp = lam + QB, *sc = lamp + QB;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, gr = lane >> 2, qc = lane & 3;
    const int h = blockIdx.x, b = blockIdx.z, dir = dir0 + blockIdx.y;
    const bool rev = dir == 1;
    const int L = a.L, k = a.k;
    const int64_t seq = (int64_t)dir * a.B + b;
    const ScanDir &w = a.dir[dir];
    const __nv_bfloat16 *zx = a.zx + ((int64_t)(a.zx_tied ? 0 : dir) * a.B + b) * L * a.d_in_proj;
    const float *dA_head = a.dA + ((seq * a.H + h) * 2) * a.Lp;
    const int nsub = KEEP ? (L + QB - 1) / QB : 1, nsub_all = a.nch * PREP_PARTS;
    const float Dh = (a.flags & DM_FLAG_D_SKIP) ? w.D[h] : 0.f;
    const bool norm_on = (a.flags & DM_FLAG_GATED_RMSNORM) != 0;

    // per-thread constants: conv taps of the channel pair 2 cp2, 2 cp2 + 1 (wl2[m] multiplies the row m steps back in time; halved, the
    // SiLU below wants v / 2), norm weights of the epilogue's 8 channels
    const int cp2 = tid % CP2, rg = tid / CP2;         // conv: channel pair, group of four rows
    f32x2 wl2[4], cb2;
    {
        const __nv_bfloat16 *cw = static_cast<const __nv_bfloat16 *>(w.conv_w) + (int64_t)(h * PP + 2 * cp2) * k;
        float w0[4], w1[4];
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            w0[m] = m < k ? 0.5f * __bfloat162float(cw[k - 1 - m]) : 0.f;
            w1[m] = m < k ? 0.5f * __bfloat162float(cw[k + k - 1 - m]) : 0.f;
            wl2[m] = pk2(w0[m], w1[m]);
        }
        const bool has_bias = (a.flags & DM_FLAG_CONV_BIAS) && w.conv_b;
        const __nv_bfloat16 *cb = static_cast<const __nv_bfloat16 *>(w.conv_b) + h * PP + 2 * cp2;
        cb2 = has_bias ? pk2(0.5f * __bfloat162float(cb[0]), 0.5f * __bfloat162float(cb[1])) : pk2(0.f, 0.f);
    }
    const int ei = tid / U8, ec = (tid % U8) * 8;      // epilogue: token row of the sub-chunk, first of 8 channels
    uint4 nwp = make_uint4(0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u);      // norm weights of those channels as bf16 pairs (ones when the norm is off)
    if (norm_on && w.norm_w) nwp = __ldg(reinterpret_cast<const uint4 *>(static_cast<const __nv_bfloat16 *>(w.norm_w) + h * PP + ec));

    // state accumulators: warp = channels [16 smt, +16) x states [64 snh, +64): tile t covers states 64 snh + 8 t .. + 7;
    // a thread holds rows p = 16 smt + gr (+8), columns n = 64 snh + 8 t + 2 qc (+1)
    const int smt = warp % MT, snh = warp / MT;
    float hacc[KEEP ? 8 : 1][4];
    const float *h_in = (!rev && a.ssm_in) ? a.ssm_in + ((int64_t)b * a.H + h) * PP * a.Nr : nullptr;
    if constexpr (KEEP) {
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            const int n = 64 * snh + 8 * t + 2 * qc, p0 = 16 * smt + gr;
            float2 v0 = make_float2(0.f, 0.f), v1 = v0;
            if (h_in && n < a.Nr) {                        // columns beyond the model's d_state are padding
                v0 = *reinterpret_cast<const float2 *>(h_in + (int64_t)p0 * a.Nr + n);
                v1 = *reinterpret_cast<const float2 *>(h_in + (int64_t)(p0 + 8) * a.Nr + n);
            }
            hacc[t][0] = v0.x; hacc[t][1] = v0.y; hacc[t][2] = v1.x; hacc[t][3] = v1.y;
        }
    }

    for (int si = 0; si < nsub; ++si) {
        const int sub = rev ? nsub - 1 - si : si, r0 = sub * QB;
        const bool have_state = si > 0 || h_in != nullptr;
        const bool need_update = KEEP && (si + 1 < nsub || (!rev && a.ssm_out != nullptr));
        const int nvalid = min(QB, L - r0);                // tokens of the sub-chunk inside the sequence
        if (KEEP) __syncthreads();                         // the previous sub-chunk's readers are done with the tiles
        // ---- load
        if (tid < QB) {
            lam[tid] = dA_head[r0 + tid];
            lamp[tid] = dA_head[a.Lp + r0 + tid];
        } else if (tid == QB) {
            const int rb = rev ? r0 + QB : r0 - 1;         // the token before the sub-chunk in time
            sc[0] = (rev ? (r0 + QB) % Q != 0 : r0 % Q != 0) ? dA_head[rb] : 0.f;
        }
        // tiles that need no conversion go straight to shared memory with 16-byte asynchronous copies, all in flight at once
        // (a copy of zero source bytes fills its 16 bytes with zeros: rows outside the sequence)
        for (int u = tid; u < (QB + 3) * U8; u += NT) {
            const int rr = u / U8, c = (u % U8) * 8;
            const int pr = rev ? r0 + rr : r0 - 3 + rr;    // physical row; the history sits before the chunk (->) or after it (<-)
            const __nv_bfloat16 *src = zx;
            uint32_t nb = 0;
            if (pr >= 0 && pr < L) { src = zx + (int64_t)pr * a.d_in_proj + a.d_inner + h * PP + c; nb = 16; }
            else if (pr < 0 && !rev && a.conv_in && k - 1 + pr >= 0) {            // rows before the sequence: the carried conv state
                src = a.conv_in + ((int64_t)b * (k - 1) + (k - 1 + pr)) * a.conv_ch + h * PP + c; nb = 16;
            }
            cp_async16(&xr[rr][c], src, nb);
        }
        if (have_state || need_update) {
            const __nv_bfloat16 *Cs = Cp + (seq * L + r0) * N, *Bs = Bp + (seq * L + r0) * N;
            for (int u = tid; u < QB * (N / 8); u += NT) {
                const int i = u / (N / 8), c = (u % (N / 8)) * 8;
                const int off = min(i, nvalid - 1) * N + c;
                const uint32_t nb = i < nvalid ? 16 : 0;
                if (have_state) cp_async16(&Ct[i][c], Cs + off, nb);
                if (need_update) cp_async16(&Bt[i][c], Bs + off, nb);
            }
        }
        {
            const float *S = Sb + (seq * nsub_all + sub) * (QB * QB);
            for (int e = tid; e < QB * QB / 4; e += NT) cp_async16(&Ss[e / (QB / 4)][(e % (QB / 4)) * 4], S + 4 * e, 16);
        }
        if (have_state) {
            if (si == 0) {
                // bf16 copy of the carried state: thread = (channel, 32 of its states in four runs of 8)
                const int p = tid >> 2, s4 = tid & 3;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    const int n0 = 8 * (4 * kk + s4);
                    float4 v0 = make_float4(0.f, 0.f, 0.f, 0.f), v1 = v0;
                    if (n0 < a.Nr) {
                        v0 = *reinterpret_cast<const float4 *>(h_in + (int64_t)p * a.Nr + n0);
                        v1 = *reinterpret_cast<const float4 *>(h_in + (int64_t)p * a.Nr + n0 + 4);
                    }
                    *reinterpret_cast<uint4 *>(&Ht[p][n0]) = make_uint4(pack_bf16(v0.x, v0.y), pack_bf16(v0.z, v0.w), pack_bf16(v1.x, v1.y), pack_bf16(v1.z, v1.w));
                }
            } else if constexpr (KEEP) {
#pragma unroll
                for (int t = 0; t < 8; ++t) {              // from the accumulators of the previous sub-chunk
                    const int n = 64 * snh + 8 * t + 2 * qc, p0 = 16 * smt + gr;
                    *reinterpret_cast<uint32_t *>(&Ht[p0][n]) = pack_bf16(hacc[t][0], hacc[t][1]);
                    *reinterpret_cast<uint32_t *>(&Ht[p0 + 8][n]) = pack_bf16(hacc[t][2], hacc[t][3]);
                }
            }
        }
        // the gate's z (it holds SiLU(z): the in_proj epilogue applied it), fetched now so that its latency hides behind the products
        uint4 zv = make_uint4(0u, 0u, 0u, 0u);
        if (ei < nvalid) zv = __ldg(reinterpret_cast<const uint4 *>(zx + (int64_t)(r0 + ei) * a.d_in_proj + h * PP + ec));
        cp_async_wait_all();
        __syncthreads();
        // ---- conv + SiLU: thread = channel pair cp2, four rows in time order with the three rows before them carried in registers
        const float lam_last = lam[rev ? 0 : QB - 1], lam0 = sc[0];      // rows past the end of the sequence have Delta = 0: Lambda stays put there
        {
            auto raw = [&](int rr) { return bf2_to_f2(*reinterpret_cast<const uint32_t *>(&xr[rr][2 * cp2])); };
            const int i0 = 4 * rg;
            // the raw row of chunk row i sits at xr[i + 3] (->) or xr[i] (<-); one step back in time is one row down (->) or up (<-)
            f32x2 h1 = raw(rev ? i0 + 4 : i0 + 2), h2 = raw(rev ? i0 + 5 : i0 + 1), h3 = raw(rev ? i0 + 6 : i0);
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int i = rev ? i0 + 3 - t : i0 + t;
                const f32x2 cur = raw(rev ? i : i + 3);
                f32x2 hh = fma2(wl2[3], h3, cb2);                   // half of the conv output
                hh = fma2(wl2[2], h2, hh); hh = fma2(wl2[1], h1, hh); hh = fma2(wl2[0], cur, hh);
                float ha, hb;
                upk2(hh, ha, hb);
                const f32x2 o = fma2(hh, pk2(tanh_fast(ha), tanh_fast(hb)), hh);      // SiLU(v) = v/2 + v/2 tanh(v/2)
                *reinterpret_cast<uint32_t *>(&Xt[i][2 * cp2]) = f2_to_bf2(o);
                if (need_update) {
                    const float wj = i < nvalid ? ex2f(lam_last - lamp[i]) : 0.f;
                    *reinterpret_cast<uint32_t *>(&WXt[i][2 * cp2]) = f2_to_bf2(mul2(o, pk2(wj, wj)));
                }
                h3 = h2; h2 = h1; h1 = cur;
            }
        }
        // ---- mask: W_ij = S_ij 2^(Lambda_i - Lambda'_j) [+ D on the diagonal] for j not after i in time and inside the sequence, else 0;
        // thread = (row i, four columns)
        for (int u = tid; u < QB * QB / 4; u += NT) {
            const int i = u >> 3, j0 = (u & 7) * 4;
            const float li = lam[i];
            const float4 s4 = *reinterpret_cast<const float4 *>(&Ss[i][j0]), lp4 = *reinterpret_cast<const float4 *>(lamp + j0);
            const float sv[4] = {s4.x, s4.y, s4.z, s4.w}, lpv[4] = {lp4.x, lp4.y, lp4.z, lp4.w};
            float wv[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int jj = j0 + q;
                const bool ok = (rev ? jj >= i : jj <= i) && jj < nvalid;
                wv[q] = fmaf(sv[q], ex2f(ok ? li - lpv[q] : -INFINITY), (ok && i == jj) ? Dh : 0.f);      // 2^-inf = 0: no branch around the exponential
            }
            *reinterpret_cast<uint2 *>(&Wt[i][j0]) = make_uint2(pack_bf16(wv[0], wv[1]), pack_bf16(wv[2], wv[3]));
        }
        __syncthreads();
        // ---- y: warp = tokens [16 ymt, +16) x channels [16 ynh, +16)
        {
            const int ymt = warp & 1, ynh = warp >> 1;
            float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
            if (have_state) {
#pragma unroll
                for (int k0 = 0; k0 < N; k0 += 16) {
                    uint32_t a0, a1, a2, a3;
                    ldmatrix_x4(a0, a1, a2, a3, &Ct[16 * ymt + (lane & 15)][k0 + (lane >> 4) * 8]);
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt) {
                        uint32_t b0, b1;
                        ldmatrix_x2(b0, b1, &Ht[16 * ynh + 8 * nt + (lane & 7)][k0 + ((lane >> 3) & 1) * 8]);
                        mma_bf16_16816(acc[nt], a0, a1, a2, a3, b0, b1);
                    }
                }
                const float e0 = ex2f(lam[16 * ymt + gr] - lam0), e1 = ex2f(lam[16 * ymt + gr + 8] - lam0);
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) { acc[nt][0] *= e0; acc[nt][1] *= e0; acc[nt][2] *= e1; acc[nt][3] *= e1; }
            }
#pragma unroll
            for (int k0 = 0; k0 < QB; k0 += 16) {
                uint32_t a0, a1, a2, a3;
                ldmatrix_x4(a0, a1, a2, a3, &Wt[16 * ymt + (lane & 15)][k0 + (lane >> 4) * 8]);
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    uint32_t b0, b1;
                    ldmatrix_x2_t(b0, b1, &Xt[k0 + (lane & 15)][16 * ynh + 8 * nt]);
                    mma_bf16_16816(acc[nt], a0, a1, a2, a3, b0, b1);
                }
            }
            // S and the raw rows were last read before the barrier above: their bytes take y
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
                const int col = 16 * ynh + 8 * nt + 2 * qc, row = 16 * ymt + gr;
                *reinterpret_cast<float2 *>(&ys[row][col]) = make_float2(acc[nt][0], acc[nt][1]);
                *reinterpret_cast<float2 *>(&ys[row + 8][col]) = make_float2(acc[nt][2], acc[nt][3]);
            }
        }
        // ---- state after the sub-chunk: h <- dec h + (w o x')^T B'
        if constexpr (KEEP) {
            if (need_update) {
                const float dec = ex2f(lam_last - lam0);
#pragma unroll
                for (int t = 0; t < 8; ++t) { hacc[t][0] *= dec; hacc[t][1] *= dec; hacc[t][2] *= dec; hacc[t][3] *= dec; }
#pragma unroll
                for (int k0 = 0; k0 < QB; k0 += 16) {
                    uint32_t a0, a1, a2, a3;                    // A = (w o x')^T [p][j] read transposed from [j][p]
                    ldmatrix_x4_t(a0, a1, a2, a3, &WXt[k0 + (lane & 7) + ((lane >> 4) & 1) * 8][16 * smt + ((lane >> 3) & 1) * 8]);
#pragma unroll
                    for (int t = 0; t < 8; ++t) {
                        uint32_t b0, b1;                        // B = B' [j][n] read transposed
                        ldmatrix_x2_t(b0, b1, &Bt[k0 + (lane & 15)][64 * snh + 8 * t]);
                        mma_bf16_16816(hacc[t], a0, a1, a2, a3, b0, b1);
                    }
                }
            }
        }
        __syncthreads();
        // ---- gate: thread = (token ei, channels ec .. ec + 7)
        {
            const float zf[8] = {bf16_lo(zv.x), bf16_hi(zv.x), bf16_lo(zv.y), bf16_hi(zv.y), bf16_lo(zv.z), bf16_hi(zv.z), bf16_lo(zv.w), bf16_hi(zv.w)};
            const float nw[8] = {bf16_lo(nwp.x), bf16_hi(nwp.x), bf16_lo(nwp.y), bf16_hi(nwp.y), bf16_lo(nwp.z), bf16_hi(nwp.z), bf16_lo(nwp.w), bf16_hi(nwp.w)};
            const float4 y0 = *reinterpret_cast<const float4 *>(&ys[ei][ec]), y1 = *reinterpret_cast<const float4 *>(&ys[ei][ec + 4]);
            const float yv[8] = {y0.x, y0.y, y0.z, y0.w, y1.x, y1.y, y1.z, y1.w};
            float g[8], ss = 0.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) { g[e] = yv[e] * zf[e]; ss = fmaf(g[e], g[e], ss); g[e] *= nw[e]; }
#pragma unroll
            for (int off = 1; off < U8; off <<= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
            if (ei < nvalid) {
                *reinterpret_cast<uint4 *>(a.g + (seq * L + r0 + ei) * a.d_inner + h * PP + ec) =
                    make_uint4(pack_bf16(g[0], g[1]), pack_bf16(g[2], g[3]), pack_bf16(g[4], g[5]), pack_bf16(g[6], g[7]));
                if (a.ssq && ec == 0) a.ssq[(seq * L + r0 + ei) * a.H + h] = ss;
            }
        }
    }
    if constexpr (KEEP) {
        if (!rev && a.ssm_out) {
            float *ho = a.ssm_out + ((int64_t)b * a.H + h) * PP * a.Nr;
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                const int n = 64 * snh + 8 * t + 2 * qc, p0 = 16 * smt + gr;
                if (n < a.Nr) {
                    *reinterpret_cast<float2 *>(ho + (int64_t)p0 * a.Nr + n) = make_float2(hacc[t][0], hacc[t][1]);
                    *reinterpret_cast<float2 *>(ho + (int64_t)(p0 + 8) * a.Nr + n) = make_float2(hacc[t][2], hacc[t][3]);
                }
            }
        }
    }
}

constexpr int BLOCK_MAX_L = 2 * QB;       // sequences up to this length take the short-block kernel by default

bool block_mode(const ScanArgs &a) { return a.chunk == QB || (a.chunk == 0 && a.L <= BLOCK_MAX_L); }

struct Scratch {
    size_t bp, cp, da, sb, sy, total;
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
    s.sb = off;
    if (block_mode(a)) off += align_up((size_t)2 * a.B * s.nch * PREP_PARTS * QB * QB * 4);
    s.sy = off; off += align_up(((size_t)2 * a.B * s.nch + 1) * sizeof(int));      // ticket counter and item flags of the fused prep
    s.total = off;
    return s;
}

bool shape_ok(const ScanArgs &a) {
    if (a.dtype != DM_BF16 || a.N < 4 || a.N > N || a.N % 4 || (a.P != P && a.P != P / 2)) return false;
    if (a.chunk != 0 && a.chunk != QB && a.chunk != Q) return false;
    return true;
}

}  // namespace

// Self-test switch: the scan launch keeps its prep role's flags but gets no prep CTA, so the load warps' bounded waits for the
// ninth chunk run out and every role of every CTA leaves through the abort path (dm_selftest_withhold_prep).
static int g_withhold_prep = 0;
void scan_ssd_selftest_withhold(int on) { g_withhold_prep = on ? 1 : 0; }

bool scan_ssd_chunk_ok(int dtype, int d_state, int chunk) {
    return !(dtype == DM_BF16 && d_state <= N) || chunk == 0 || chunk == QB || chunk == Q;
}

bool scan_ssd_supports(const ScanArgs &a) {
    if (!shape_ok(a) || a.k < 2 || a.k > 4) return false;
    if (a.P != P && 2 * a.N < P / 2) return false;                        // a half-width head's tile reaches P/2 columns past the last head: they must exist in the row
    if (!a.z_gated) return false;                                         // the gate's SiLU is the in_proj epilogue's job on this path
    if (a.d_in_proj % 8 || a.d_inner % 8 || a.conv_ch % 8) return false;  // 16-byte rows for TMA and vector access
    if (a.H > 65535 || a.B > 65535) return false;
    return encode_fn() != nullptr;
}

size_t scan_ssd_workspace_bytes(const ScanArgs &a) {
    if (!shape_ok(a)) return 0;
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
    k.flags = a.flags; k.nch = l.nch; k.Lp = l.Lp; k.Nr = a.N; k.Pr = a.P; k.zx_tied = a.zx_tied; k.g = static_cast<__nv_bfloat16 *>(a.g);
    k.zx = static_cast<const __nv_bfloat16 *>(a.zx); k.ssq = a.ssq; k.dA = dA;
    k.ssm_in = a.ssm_in; k.ssm_out = a.ssm_out; k.conv_in = static_cast<const __nv_bfloat16 *>(a.conv_in);
    k.dir[0] = a.dir[0]; k.dir[1] = a.dir[1];
    const int ndir = a.dir_mask == DM_DIR_BOTH ? 2 : 1, dir0 = a.dir_mask == DM_DIR_REV ? 1 : 0;
    const bool blk = block_mode(a);
    float *Sb = blk ? reinterpret_cast<float *>(base + l.sb) : nullptr;

    // One long sequence leaves SMs without a scan CTA: they take the prep work inside the scan launch (see prep_role), except for
    // the first PRE_CHUNKS chunks of every sequence and direction, which a small prep launch of their own has ready by the time the
    // scan starts (a prep CTA inside the scan launch needs about 20 us for its first chunk; the scan would stand idle that long).
    constexpr int PRE_CHUNKS = 8;
    const bool pair = a.P == P / 2 && a.H % 2 == 0;        // two half-width heads per scan CTA
    const int nscan = (pair ? a.H / 2 : a.H) * ndir * a.B;
    PrepJob pj{Bp, Cp, dA, nullptr, 0, ndir, 0};
    int n_pre = l.nch;                              // chunks (in time order) done by the prep launch
    if (!blk && nscan < sm_count() && a.N % 8 == 0 && l.nch > PRE_CHUNKS) {
        const int n_items = ndir * a.B * (l.nch - PRE_CHUNKS);
        pj.nprep = n_items < sm_count() - nscan ? n_items : sm_count() - nscan;
        if (ndir == 2) pj.nprep &= ~1;                             // even: every prep CTA then stays with one direction
        if (pj.nprep > 0) {
            pj.sync = reinterpret_cast<int *>(base + l.sy);
            pj.c0 = n_pre = PRE_CHUNKS;
        }
    }
    if (pj.sync && g_withhold_prep) pj.nprep = 0;
    cudaError_t e;
    if (pj.sync && (e = cudaMemsetAsync(pj.sync, 0, ((size_t)2 * a.B * l.nch + 1) * sizeof(int), s)) != cudaSuccess) return e;
    ssd_prep_kernel<<<dim3(n_pre * PREP_PARTS * (blk ? 2 : 1), a.B, ndir), PREP_THREADS, 0, s>>>(k, Bp, Cp, dA, Sb, dir0, blk ? 1 : 0);
    count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (blk) {
        // the state is carried in registers when there are several sub-chunks or someone reads it afterwards
        const bool keep = a.L > QB || a.ssm_out != nullptr;
        auto kern = a.P == P ? (keep ? ssd_block_kernel<P, true> : ssd_block_kernel<P, false>)
                             : (keep ? ssd_block_kernel<P / 2, true> : ssd_block_kernel<P / 2, false>);
        const size_t smem = a.P == P ? (keep ? BlockSmem<P>::total : BlockSmem<P>::total_nokeep)
                                     : (keep ? BlockSmem<P / 2>::total : BlockSmem<P / 2>::total_nokeep);
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kern<<<dim3(a.H, ndir, a.B), 4 * a.P, smem, s>>>(k, Bp, Cp, Sb, dir0);
        count_launch();
        return cudaGetLastError();
    }

    CUtensorMap mx, mz, mb, mc, mg;
    {
        const uint64_t dims[3] = {(uint64_t)a.d_in_proj, (uint64_t)a.L, (uint64_t)2 * a.B};
        const uint64_t str[2] = {(uint64_t)a.d_in_proj, (uint64_t)a.L * a.d_in_proj};
        const uint32_t box_x[3] = {64, (uint32_t)XROWS, 1}, box_z[3] = {64, (uint32_t)Q, 1};
        if (!make_map_bf16(&mx, a.zx, 3, dims, str, box_x) || !make_map_bf16(&mz, a.zx, 3, dims, str, box_z)) return cudaErrorInvalidValue;
    }
    {
        const uint64_t dims[3] = {(uint64_t)N, (uint64_t)a.L, (uint64_t)2 * a.B};
        const uint64_t str[2] = {(uint64_t)N, (uint64_t)a.L * N};
        const uint32_t box[3] = {64, (uint32_t)Q, 1};
        if (!make_map_bf16(&mb, Bp, 3, dims, str, box) || !make_map_bf16(&mc, Cp, 3, dims, str, box)) return cudaErrorInvalidValue;
    }
    {
        const uint64_t dims[3] = {(uint64_t)a.d_inner, (uint64_t)a.L, (uint64_t)2 * a.B};
        const uint64_t str[2] = {(uint64_t)a.d_inner, (uint64_t)a.L * a.d_inner};
        const uint32_t box[3] = {64, (uint32_t)Q, 1};
        if (!make_map_bf16(&mg, a.g, 3, dims, str, box)) return cudaErrorInvalidValue;
    }
    int *status = device_status_ptr();
    if (!status) return cudaErrorUnknown;
    auto kern = a.P == P ? ssd_scan_kernel<0> : pair ? ssd_scan_kernel<2> : ssd_scan_kernel<1>;
    const uint32_t smem_bytes = pair ? SMEM_BYTES_PAIR : SMEM_BYTES;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
    if (e != cudaSuccess) return e;
    kern<<<nscan + pj.nprep, NTHREADS, smem_bytes, s>>>(mx, mz, mb, mc, mg, k, pj, dir0, status);
    count_launch();
    return cudaGetLastError();
}

}  // namespace dm
