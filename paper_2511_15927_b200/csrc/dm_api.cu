// C-ABI entry points: argument checks, workspace layout, and the launch sequence of each call.
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <vector>

#include "dm_internal.h"

namespace dm {

static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

__device__ int g_device_status;   // 0 = fine; kernels store a dm_status when a bounded wait gives up

int *device_status_ptr() {
    static int *cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!cached[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_device_status) != cudaSuccess) return nullptr;
        cached[dev] = static_cast<int *>(p);
    }
    return cached[dev];
}

static thread_local char g_err[512] = "";

// Optional per-stage timing: CUDA event pairs recorded on the caller's stream around in_proj, the fused
// scan and out_proj of every mixer call; summed and released by dm_profile_read().
struct StageSpan { int stage; cudaEvent_t a, b; };
static std::mutex g_prof_mu;
static bool g_prof_on = false;
static std::vector<StageSpan> g_spans;

struct StageTimer {
    bool on; int stage; cudaStream_t s; cudaEvent_t a = nullptr;
    StageTimer(int stage_, cudaStream_t s_) : on(g_prof_on), stage(stage_), s(s_) {
        if (on && (cudaEventCreate(&a) != cudaSuccess || cudaEventRecord(a, s) != cudaSuccess)) on = false;
    }
    ~StageTimer() {
        if (!on) return;
        cudaEvent_t b = nullptr;
        if (cudaEventCreate(&b) == cudaSuccess && cudaEventRecord(b, s) == cudaSuccess) {
            std::lock_guard<std::mutex> lk(g_prof_mu);
            g_spans.push_back({stage, a, b});
        }
    }
};

static int fail(int status, const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return status;
}

static int cuda_fail(cudaError_t e, const char *what) {
    if (e == cudaErrorNotSupported) return fail(DM_ERR_UNSUPPORTED, "%s: shape not supported by the kernel", what);
    return fail(DM_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

struct Dims {
    int B, L, d, d_inner, H, P, N, k, G, conv_ch, d_in_proj;
    int ldz;          // row pitch of the in_proj output in the workspace: d_in_proj rounded up to 8 elements (16-byte rows for TMA and vector loads)
    int64_t T;
    size_t es;
};

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int check_cfg(const dm_mixer_cfg *c, Dims *o) {
    if (!c) return fail(DM_ERR_INVALID_ARG, "cfg is NULL");
    if (c->batch <= 0 || c->seqlen <= 0 || c->d_model <= 0 || c->expand <= 0 || c->d_state <= 0 || c->n_heads <= 0)
        return fail(DM_ERR_INVALID_ARG, "batch, seqlen, d_model, expand, d_state and n_heads must be positive");
    if (c->dtype != DM_F32 && c->dtype != DM_BF16) return fail(DM_ERR_INVALID_ARG, "dtype must be DM_F32 or DM_BF16");
    if (c->dir_mask < DM_DIR_FWD || c->dir_mask > DM_DIR_BOTH) return fail(DM_ERR_INVALID_ARG, "dir_mask must be 1, 2 or 3");
    if (c->flags & ~(DM_FLAG_GATED_RMSNORM | DM_FLAG_CONV_BIAS | DM_FLAG_D_SKIP | DM_FLAG_TIED_PROJ)) return fail(DM_ERR_INVALID_ARG, "unknown flag bits");
    if (c->chunk < 0) return fail(DM_ERR_INVALID_ARG, "chunk must be >= 0");
    if (!(c->norm_eps >= 0.f)) return fail(DM_ERR_INVALID_ARG, "norm_eps must be >= 0");
    if (c->n_groups != 1) return fail(DM_ERR_UNSUPPORTED, "n_groups must be 1");
    if (c->d_conv < 2 || c->d_conv > 4) return fail(DM_ERR_UNSUPPORTED, "d_conv must be in [2,4]");
    const int64_t d_inner = (int64_t)c->expand * c->d_model;
    if (d_inner % c->n_heads) return fail(DM_ERR_INVALID_ARG, "expand*d_model must be divisible by n_heads");
    const int P = (int)(d_inner / c->n_heads);
    if (P != 32 && P != 64) return fail(DM_ERR_UNSUPPORTED, "headdim must be 32 or 64 (got %d)", P);
    const int N = c->d_state;
    if (N != 16 && N != 32 && N != 64 && N != 128 && N != 256) return fail(DM_ERR_UNSUPPORTED, "d_state must be 16, 32, 64, 128 or 256");
    if ((int64_t)P * (N / 16) > 1024) return fail(DM_ERR_UNSUPPORTED, "headdim * d_state / 16 must not exceed 1024");
    if ((int64_t)c->batch * c->seqlen > (int64_t)1 << 30) return fail(DM_ERR_UNSUPPORTED, "batch*seqlen too large");
    if (!scan_ssd_chunk_ok(c->dtype, N, c->chunk))
        return fail(DM_ERR_UNSUPPORTED, "bf16 with d_state <= 128 runs the chunked scan: chunk must be 0, 32 or 128 (got %d)", c->chunk);
    o->B = c->batch; o->L = c->seqlen; o->d = c->d_model; o->d_inner = (int)d_inner; o->H = c->n_heads; o->P = P;
    o->N = N; o->k = c->d_conv; o->G = 1;
    o->conv_ch = o->d_inner + 2 * N;
    o->d_in_proj = 2 * o->d_inner + 2 * N + o->H;
    o->ldz = (o->d_in_proj + 7) / 8 * 8;
    o->T = (int64_t)c->batch * c->seqlen;
    o->es = dtype_size(c->dtype);
    return DM_OK;
}

static int check_weights(const dm_mixer_cfg *c, const dm_dir_weights w[2]) {
    if (!w) return fail(DM_ERR_INVALID_ARG, "weights are NULL");
    for (int dir = 0; dir < 2; ++dir) {
        if (!(c->dir_mask & (1 << dir))) continue;
        const dm_dir_weights &q = w[dir];
        const dm_dir_weights &pw = w[(c->flags & DM_FLAG_TIED_PROJ) ? 0 : dir];       // whose projections this direction uses
        if (!pw.w_in || !q.conv_w || !q.dt_bias || !q.A_log || !pw.w_out) return fail(DM_ERR_INVALID_ARG, "direction %d: NULL weight pointer", dir);
        if ((c->flags & DM_FLAG_CONV_BIAS) && !q.conv_b) return fail(DM_ERR_INVALID_ARG, "direction %d: conv_b is NULL but DM_FLAG_CONV_BIAS is set", dir);
        if ((c->flags & DM_FLAG_D_SKIP) && !q.D) return fail(DM_ERR_INVALID_ARG, "direction %d: D is NULL but DM_FLAG_D_SKIP is set", dir);
        if ((c->flags & DM_FLAG_GATED_RMSNORM) && !q.norm_w) return fail(DM_ERR_INVALID_ARG, "direction %d: norm_w is NULL but DM_FLAG_GATED_RMSNORM is set", dir);
        if (!aligned16(pw.w_in) || !aligned16(pw.w_out)) return fail(DM_ERR_INVALID_ARG, "direction %d: matrices must be 16-byte aligned", dir);
    }
    return DM_OK;
}

// Up to this many tokens the two directions' out_proj run as one launch that writes an fp32 partial each (summed by a small
// kernel); above it they are chained, the second adding the first in its epilogue, which moves less memory.
constexpr int64_t PAIR_OUT_MAX_T = 2048;
// Up to this many tokens the two directions' in_proj share one launch.  Beyond it two launches are faster: both weight matrices
// together (70 MB at d_model 2048) no longer stay in L2 while the rows of x stream past them (measured at 16 384 tokens: 1.00 ms
// for the pair against 0.84 ms for two launches; level at 8192, 15-25 % faster for the 512 tokens of a decoding step).
constexpr int64_t PAIR_IN_MAX_T = 4096;

// Workspace layout of one mixer call.
struct MixerWs {
    size_t zx, g, ssq, rstd, ytmp, scan, total;
};

static MixerWs mixer_ws(const dm_mixer_cfg *c, const Dims &m) {
    MixerWs w;
    size_t off = 0;
    w.zx = off;   off += align_up((size_t)2 * m.T * m.ldz * m.es);
    w.g = off;    off += align_up((size_t)2 * m.T * m.d_inner * m.es);
    w.ssq = off;  off += align_up((size_t)2 * m.T * m.H * sizeof(float));
    w.rstd = off; off += align_up((size_t)2 * m.T * sizeof(float));
    w.ytmp = off; off += align_up((size_t)(m.T <= PAIR_OUT_MAX_T ? 4 : 1) * m.T * m.d * sizeof(float));      // short inputs: up to two fp32 partials per direction
    ScanArgs sa{};
    sa.B = m.B; sa.L = m.L; sa.d_inner = m.d_inner; sa.H = m.H; sa.P = m.P; sa.N = m.N; sa.k = m.k;
    sa.d_in_proj = m.ldz; sa.conv_ch = m.conv_ch; sa.dtype = c->dtype; sa.flags = c->flags; sa.dir_mask = c->dir_mask; sa.chunk = c->chunk;
    {
        const size_t a_ssd = scan_ssd_workspace_bytes(sa), a_seq = scan_seq_workspace_bytes(sa);
        w.scan = off; off += align_up(a_ssd > a_seq ? a_ssd : a_seq);
    }
    w.total = off;
    return w;
}

static cudaError_t gemm(const GemmArgs &a, cudaStream_t s) {
    if (gemm_tcgen05_supports(a)) return gemm_tcgen05(a, s);
    return gemm_simple(a, s);
}

struct MixerOut {
    void *y; int y_dtype; const float *addend; int64_t ld_add;
    const float *col_scale = nullptr; int cs_rows = 0; int64_t ld_cs = 0;   // per-sequence gate on the mixer's output (App. A.1), or NULL
    // The caller's next step is u = RMSNorm(y; next_norm_w): a mixer that sums its directions in a pass of its own applies it there and sets *next_done
    const void *next_norm_w = nullptr; void *next_u = nullptr; float next_eps = 0.f; bool *next_done = nullptr;
};

// in_proj -> fused conv/scan/gate -> out_proj of both directions, summed (Sec. 3.2).
static int run_mixer(const dm_mixer_cfg *c, const Dims &m, const dm_dir_weights w[2], const void *x, const MixerOut &out,
                     const float *ssm_in, const void *conv_in, float *ssm_out, void *conv_out,
                     char *ws, cudaStream_t s) {
    const MixerWs l = mixer_ws(c, m);
    char *zx = ws + l.zx, *g = ws + l.g;
    float *ssq = reinterpret_cast<float *>(ws + l.ssq), *rstd = reinterpret_cast<float *>(ws + l.rstd);
    float *ytmp = reinterpret_cast<float *>(ws + l.ytmp);
    const bool norm_on = (c->flags & DM_FLAG_GATED_RMSNORM) != 0;
    cudaError_t e;

    ScanArgs sa{};
    sa.B = m.B; sa.L = m.L; sa.d_inner = m.d_inner; sa.H = m.H; sa.P = m.P; sa.N = m.N; sa.k = m.k;
    sa.d_in_proj = m.ldz; sa.conv_ch = m.conv_ch;          // the kernels use it as the row pitch only
    sa.dtype = c->dtype; sa.flags = c->flags; sa.dir_mask = c->dir_mask; sa.chunk = c->chunk;
    sa.zx = zx; sa.g = g; sa.ssq = norm_on ? ssq : nullptr;
    for (int dir = 0; dir < 2; ++dir) {
        sa.dir[dir].conv_w = w[dir].conv_w; sa.dir[dir].conv_b = w[dir].conv_b; sa.dir[dir].norm_w = w[dir].norm_w;
        sa.dir[dir].dt_bias = w[dir].dt_bias; sa.dir[dir].A_log = w[dir].A_log; sa.dir[dir].D = w[dir].D;
    }
    sa.ssm_in = ssm_in; sa.conv_in = conv_in; sa.ssm_out = ssm_out;
    const bool tied = (c->flags & DM_FLAG_TIED_PROJ) != 0;
    sa.zx_tied = tied ? 1 : 0;
    // The tensor-core scan is bound by instruction issue while the GEMM's epilogue warps mostly wait: on that path the
    // gate's SiLU(z) (Sec. 3.2) is applied to the z columns by the in_proj epilogue.
    sa.z_gated = 1;
    const bool ssd = scan_ssd_supports(sa);
    sa.z_gated = ssd ? 1 : 0;

    {
        GemmArgs ga[2];
        int n = 0;
        for (int dir = 0; dir < 2; ++dir) {
            if (!(c->dir_mask & (1 << dir))) continue;
            if (tied && dir == 1 && (c->dir_mask & DM_DIR_FWD)) continue;     // tied projections: one in_proj serves both directions
            GemmArgs a{};
            a.A = x; a.lda = m.d; a.B = w[tied ? 0 : dir].w_in; a.ldb = m.d;
            a.C = zx + (size_t)(tied ? 0 : dir) * m.T * m.ldz * m.es; a.ldc = m.ldz;
            a.in_dtype = c->dtype; a.c_dtype = c->dtype; a.M = (int)m.T; a.N = m.d_in_proj; a.K = m.d;
            a.silu_cols = ssd ? m.d_inner : 0;
            ga[n++] = a;
        }
        StageTimer tm(DM_STAGE_IN_PROJ, s);
        if (n == 2 && m.T <= PAIR_IN_MAX_T && gemm_tcgen05_pair_supports(ga[0], ga[1])) {
            // both directions in one launch: x is fetched once for the two, and there is one tail round instead of two
            if ((e = gemm_tcgen05_pair(ga[0], ga[1], s)) != cudaSuccess) return cuda_fail(e, "in_proj");
        } else {
            for (int i = 0; i < n; ++i)
                if ((e = gemm(ga[i], s)) != cudaSuccess) return cuda_fail(e, "in_proj");
        }
    }
    {
        StageTimer tm(DM_STAGE_SCAN, s);
        if (ssd) e = scan_ssd(sa, ws + l.scan, s);
        else e = scan_sequential(sa, ws + l.scan, s);
    }
    if (e != cudaSuccess) return cuda_fail(e, "scan");

    if (conv_out && (c->dir_mask & DM_DIR_FWD)) {
        e = conv_state_update(zx, conv_in, conv_out, c->dtype, m.B, m.L, m.k, m.d_inner, m.conv_ch, m.ldz, s);
        if (e != cudaSuccess) return cuda_fail(e, "conv_state_update");
    }
    if (!tied && c->dir_mask == DM_DIR_BOTH && m.T <= PAIR_OUT_MAX_T && sum_partials_norm_supports(m.d)) {
        // short inputs (block decoding): both out_proj in one launch, each into its own fp32 partial (gated by col_scale, not yet scaled by the
        // gated norm); one pass then scales, sums, adds the residual and applies the caller's next norm
        GemmArgs ga[2];
        for (int dir = 0; dir < 2; ++dir) {
            GemmArgs a{};
            a.A = g + (size_t)dir * m.T * m.d_inner * m.es; a.lda = m.d_inner;
            a.B = w[dir].w_out; a.ldb = m.d_inner;
            a.in_dtype = c->dtype; a.M = (int)m.T; a.N = m.d; a.K = m.d_inner;
            a.col_scale = out.col_scale; a.cs_rows = out.cs_rows; a.ld_cs = out.ld_cs;
            a.C = ytmp + (size_t)dir * m.T * m.d; a.ldc = m.d; a.c_dtype = DM_F32;
            ga[dir] = a;
        }
        if (gemm_tcgen05_pair_supports(ga[0], ga[1])) {
            {
                StageTimer tm(DM_STAGE_OUT_PROJ, s);
                const size_t part = (size_t)m.T * m.d;
                const bool split = gemm_tcgen05_pair_splitk_pays(ga[0], ga[1]);
                e = split ? gemm_tcgen05_pair_splitk(ga[0], ga[1], ytmp + 2 * part, ytmp + 3 * part, s) : gemm_tcgen05_pair(ga[0], ga[1], s);
                if (e != cudaSuccess) return cuda_fail(e, "out_proj");
                const bool next = out.next_norm_w && out.next_u;
                e = sum_partials_norm(ytmp, ytmp + part, split ? ytmp + 2 * part : nullptr, split ? ytmp + 3 * part : nullptr, norm_on ? ssq : nullptr, norm_on ? ssq + (size_t)m.T * m.H : nullptr, m.H, m.d_inner,
                                      c->norm_eps, out.addend, out.ld_add, out.y, out.y_dtype, next ? out.next_norm_w : nullptr, next ? out.next_u : nullptr,
                                      c->dtype, m.T, m.d, out.next_eps, s);
                if (next && out.next_done) *out.next_done = true;
            }
            if (e != cudaSuccess) return cuda_fail(e, "out_proj sum");
            return DM_OK;
        }
    }
    if (norm_on) {
        e = rstd_from_ssq(ssq, rstd, (int)(2 * m.T), m.H, m.d_inner, c->norm_eps, s);
        if (e != cudaSuccess) return cuda_fail(e, "rstd");
    }
    if (tied && c->dir_mask == DM_DIR_BOTH) {
        // shared out_proj: W_out (s-> g-> + s<- g<-) with s the gated-norm scale of each direction (1 without the norm); one GEMM
        e = combine_directions(g, g + (size_t)m.T * m.d_inner * m.es, norm_on ? rstd : nullptr, norm_on ? rstd + m.T : nullptr, c->dtype, m.T,
                               m.d_inner, s);
        if (e != cudaSuccess) return cuda_fail(e, "combine_directions");
        StageTimer tm(DM_STAGE_OUT_PROJ, s);
        GemmArgs a{};
        a.A = g; a.lda = m.d_inner; a.B = w[0].w_out; a.ldb = m.d_inner;
        a.in_dtype = c->dtype; a.M = (int)m.T; a.N = m.d; a.K = m.d_inner;
        a.addend = out.addend; a.ld_add = out.ld_add;
        a.col_scale = out.col_scale; a.cs_rows = out.cs_rows; a.ld_cs = out.ld_cs;
        a.C = out.y; a.ldc = m.d; a.c_dtype = out.y_dtype;
        if ((e = gemm(a, s)) != cudaSuccess) return cuda_fail(e, "out_proj");
        return DM_OK;
    }
    // out_proj of each direction; the second one adds the first (Mamba(x) = h-> + h<-)
    const float *carry = out.addend;
    int64_t ld_carry = out.ld_add;
    const int last_dir = (c->dir_mask & DM_DIR_REV) ? 1 : 0;
    for (int dir = 0; dir < 2; ++dir) {
        if (!(c->dir_mask & (1 << dir))) continue;
        const bool last = dir == last_dir;
        StageTimer tm(DM_STAGE_OUT_PROJ, s);
        GemmArgs a{};
        a.A = g + (size_t)dir * m.T * m.d_inner * m.es; a.lda = m.d_inner;
        a.B = w[tied ? 0 : dir].w_out; a.ldb = m.d_inner;
        a.in_dtype = c->dtype; a.M = (int)m.T; a.N = m.d; a.K = m.d_inner;
        a.row_scale = norm_on ? rstd + (size_t)dir * m.T : nullptr;
        a.addend = carry; a.ld_add = ld_carry;
        a.col_scale = out.col_scale; a.cs_rows = out.cs_rows; a.ld_cs = out.ld_cs;   // the gate distributes over the sum of the directions
        if (last) { a.C = out.y; a.ldc = m.d; a.c_dtype = out.y_dtype; }
        else { a.C = ytmp; a.ldc = m.d; a.c_dtype = DM_F32; carry = ytmp; ld_carry = m.d; }
        if ((e = gemm(a, s)) != cudaSuccess) return cuda_fail(e, "out_proj");
    }
    return DM_OK;
}

static int check_ws(const void *ws, size_t have, size_t need) {
    if (!ws) return fail(DM_ERR_WORKSPACE, "workspace is NULL");
    if (reinterpret_cast<uintptr_t>(ws) & 255u) return fail(DM_ERR_WORKSPACE, "workspace must be 256-byte aligned");
    if (have < need) return fail(DM_ERR_WORKSPACE, "workspace too small: %zu bytes given, %zu needed", have, need);
    return DM_OK;
}

struct StackWs {
    size_t r, u, logits, mixer, mod, hmid, idx, count, ug, qkv, att, total;
    int logits_rows;
};

static StackWs stack_ws(const dm_stack_cfg *c, const Dims &m, const dm_block_cfg *blk = nullptr, bool sampler = false, bool hybrid = false) {
    StackWs w;
    size_t off = 0;
    w.r = off; off += align_up((size_t)m.T * m.d * sizeof(float));
    w.u = off; off += align_up((size_t)m.T * m.d * m.es);
    w.logits_rows = (int)(m.T < 2048 ? m.T : 2048);
    w.logits = off; off += align_up((size_t)w.logits_rows * c->vocab * m.es);
    w.mixer = off; off += mixer_ws(&c->mixer, m).total;
    w.mod = w.hmid = off;
    if (blk) {
        w.mod = off; off += align_up((size_t)m.B * 6 * m.d * sizeof(float));
        w.hmid = off; off += align_up((size_t)m.T * blk->d_ff * m.es);
    }
    w.idx = w.count = w.ug = off;
    if (sampler) {
        w.idx = off; off += align_up((size_t)m.T * sizeof(int32_t));
        w.count = off; off += align_up(sizeof(int));
        w.ug = off; off += align_up((size_t)m.T * m.d * m.es);
    }
    w.qkv = w.att = off;
    if (hybrid) {
        w.qkv = off; off += align_up((size_t)m.T * 3 * m.d * m.es);
        w.att = off; off += align_up((size_t)m.T * m.d * m.es);
    }
    w.total = off;
    return w;
}

// Fixed scratch for dm_bimamba_forward_static.  In host code the symbol below is only a handle: the device
// address has to be asked for, once per device, with that device current.
static __device__ __align__(256) unsigned char g_static_ws[DM_STATIC_WORKSPACE_BYTES];

static int static_ws_ptr(char **out) {
    static char *cached[64] = {};
    static std::mutex mu;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "dm_bimamba_forward_static: cudaGetDevice");
    if (dev < 0 || dev >= 64) return fail(DM_ERR_UNSUPPORTED, "dm_bimamba_forward_static: device index %d out of range", dev);
    std::lock_guard<std::mutex> lk(mu);
    if (!cached[dev]) {
        void *p = nullptr;
        if ((e = cudaGetSymbolAddress(&p, g_static_ws)) != cudaSuccess)
            return cuda_fail(e, "dm_bimamba_forward_static: cudaGetSymbolAddress");
        cached[dev] = static_cast<char *>(p);
    }
    *out = cached[dev];
    return DM_OK;
}

}  // namespace dm

using namespace dm;

extern "C" {

const char *dm_status_string(int status) {
    switch (status) {
        case DM_OK: return "ok";
        case DM_ERR_INVALID_ARG: return "invalid argument";
        case DM_ERR_UNSUPPORTED: return "unsupported shape or option";
        case DM_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case DM_ERR_CUDA: return "CUDA runtime error";
        case DM_ERR_TIMEOUT: return "a bounded device-side wait expired";
        default: return "unknown status";
    }
}

const char *dm_last_error_message(void) { return g_err; }

uint64_t dm_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int dm_profile_enable(int on) {
    std::lock_guard<std::mutex> lk(g_prof_mu);
    g_prof_on = on != 0;
    return DM_OK;
}

int dm_profile_read(float *ms, uint64_t *spans) {
    if (!ms || !spans) return fail(DM_ERR_INVALID_ARG, "ms or spans is NULL");
    std::vector<StageSpan> v;
    {
        std::lock_guard<std::mutex> lk(g_prof_mu);
        v.swap(g_spans);
    }
    for (int i = 0; i < DM_STAGE_COUNT; ++i) { ms[i] = 0.f; spans[i] = 0; }
    int st = DM_OK;
    for (const StageSpan &sp : v) {
        float t = 0.f;
        cudaError_t e = cudaEventSynchronize(sp.b);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&t, sp.a, sp.b);
        if (e == cudaSuccess && sp.stage >= 0 && sp.stage < DM_STAGE_COUNT) { ms[sp.stage] += t; spans[sp.stage] += 1; }
        else if (e != cudaSuccess) st = cuda_fail(e, "dm_profile_read");
        cudaEventDestroy(sp.a);
        cudaEventDestroy(sp.b);
    }
    return st;
}

int dm_bimamba_workspace_bytes(const dm_mixer_cfg *cfg, size_t *bytes) {
    Dims m;
    if (!bytes) return fail(DM_ERR_INVALID_ARG, "bytes is NULL");
    int st = check_cfg(cfg, &m);
    if (st != DM_OK) return st;
    *bytes = mixer_ws(cfg, m).total;
    return DM_OK;
}

int dm_denoise_workspace_bytes(const dm_stack_cfg *cfg, size_t *bytes) {
    Dims m;
    if (!bytes || !cfg) return fail(DM_ERR_INVALID_ARG, "NULL argument");
    int st = check_cfg(&cfg->mixer, &m);
    if (st != DM_OK) return st;
    if (cfg->n_layers <= 0 || cfg->vocab <= 0) return fail(DM_ERR_INVALID_ARG, "n_layers and vocab must be positive");
    *bytes = stack_ws(cfg, m).total;
    return DM_OK;
}

int dm_check(void *cuda_stream) {
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(e, "dm_check: synchronize");
    int *p = device_status_ptr();
    if (!p) return fail(DM_ERR_CUDA, "dm_check: no status word");
    int v = 0;
    if ((e = cudaMemcpy(&v, p, sizeof(int), cudaMemcpyDeviceToHost)) != cudaSuccess) return cuda_fail(e, "dm_check: read status");
    if (v != 0) {
        int zero = 0;
        cudaMemcpy(p, &zero, sizeof(int), cudaMemcpyHostToDevice);
        return fail(v, "a kernel reported status %d (%s)", v, dm_status_string(v));
    }
    return DM_OK;
}

int dm_bimamba_forward(const dm_mixer_cfg *cfg, const dm_dir_weights w[2], const void *x, void *y,
                       void *workspace, size_t workspace_bytes, void *cuda_stream) {
    Dims m;
    int st = check_cfg(cfg, &m);
    if (st != DM_OK) return st;
    if ((st = check_weights(cfg, w)) != DM_OK) return st;
    if (!x || !y) return fail(DM_ERR_INVALID_ARG, "x or y is NULL");
    if (x == y) return fail(DM_ERR_INVALID_ARG, "y must not alias x");
    if (!aligned16(x) || !aligned16(y)) return fail(DM_ERR_INVALID_ARG, "x and y must be 16-byte aligned");
    if ((st = check_ws(workspace, workspace_bytes, mixer_ws(cfg, m).total)) != DM_OK) return st;
    MixerOut out{y, cfg->dtype, nullptr, 0};
    return run_mixer(cfg, m, w, x, out, nullptr, nullptr, nullptr, nullptr, static_cast<char *>(workspace),
                     static_cast<cudaStream_t>(cuda_stream));
}

int dm_bimamba_forward_static(const dm_mixer_cfg *cfg, const dm_dir_weights w[2], const void *x, void *y, void *cuda_stream) {
    Dims m;
    int st = check_cfg(cfg, &m);
    if (st != DM_OK) return st;
    if ((st = check_weights(cfg, w)) != DM_OK) return st;
    if (!x || !y) return fail(DM_ERR_INVALID_ARG, "x or y is NULL");
    if (x == y) return fail(DM_ERR_INVALID_ARG, "y must not alias x");
    if (!aligned16(x) || !aligned16(y)) return fail(DM_ERR_INVALID_ARG, "x and y must be 16-byte aligned");
    const size_t need = mixer_ws(cfg, m).total;
    if (need > DM_STATIC_WORKSPACE_BYTES)
        return fail(DM_ERR_WORKSPACE, "this configuration needs %zu bytes of scratch, the built-in array holds %zu: "
                    "call dm_bimamba_forward with a workspace of your own", need, (size_t)DM_STATIC_WORKSPACE_BYTES);
    char *ws = nullptr;
    if ((st = static_ws_ptr(&ws)) != DM_OK) return st;
    MixerOut out{y, cfg->dtype, nullptr, 0};
    return run_mixer(cfg, m, w, x, out, nullptr, nullptr, nullptr, nullptr, ws, static_cast<cudaStream_t>(cuda_stream));
}

int dm_bimamba_block_step(const dm_mixer_cfg *cfg, const dm_dir_weights w[2], const void *x_blk,
                          const float *ssm_state_in, const void *conv_state_in,
                          float *ssm_state_out, void *conv_state_out, void *y_blk,
                          void *workspace, size_t workspace_bytes, void *cuda_stream) {
    Dims m;
    int st = check_cfg(cfg, &m);
    if (st != DM_OK) return st;
    if ((st = check_weights(cfg, w)) != DM_OK) return st;
    if (!x_blk || !y_blk) return fail(DM_ERR_INVALID_ARG, "x_blk or y_blk is NULL");
    if (x_blk == y_blk) return fail(DM_ERR_INVALID_ARG, "y_blk must not alias x_blk");
    if (!aligned16(x_blk) || !aligned16(y_blk) || !aligned16(ssm_state_in) || !aligned16(ssm_state_out) ||
        !aligned16(conv_state_in) || !aligned16(conv_state_out))
        return fail(DM_ERR_INVALID_ARG, "tensors must be 16-byte aligned");
    if ((ssm_state_in && ssm_state_in == ssm_state_out) || (conv_state_in && conv_state_in == conv_state_out))
        return fail(DM_ERR_INVALID_ARG, "state_in and state_out must be different buffers");
    if ((ssm_state_out || conv_state_out) && !(cfg->dir_mask & DM_DIR_FWD))
        return fail(DM_ERR_INVALID_ARG, "state_out needs the left-to-right direction");
    if ((st = check_ws(workspace, workspace_bytes, mixer_ws(cfg, m).total)) != DM_OK) return st;
    MixerOut out{y_blk, cfg->dtype, nullptr, 0};
    return run_mixer(cfg, m, w, x_blk, out, ssm_state_in, conv_state_in, ssm_state_out, conv_state_out,
                     static_cast<char *>(workspace), static_cast<cudaStream_t>(cuda_stream));
}

}  // extern "C"

// One denoiser evaluation.  blk == NULL: RMSNorm pre-norm + mixer per layer; otherwise the timestep-conditioned block of
// App. A.1 (AdaLN -> mixer -> gated residual, AdaLN -> MLP -> gated residual) with the modulation of each layer from tau.
struct SampleArgs {
    const dm_sample_cfg *cfg; const float *u_keep, *u_cat; int32_t *tokens_out;
};
struct HybridArgs {
    const dm_hybrid_cfg *cfg; const dm_attn_weights *aw;      // aw: HOST array of n_layers entries (used where the layer is attention)
    const dm_attn_state *ast = nullptr;                       // block mode: key/value caches of the attention layers (HOST array), or NULL
};

static int denoise_impl(const dm_stack_cfg *cfg, const dm_block_cfg *blk, const dm_stack_weights *weights, const dm_block_weights *bw,
                        const int32_t *tokens, const float *tau, void *logits,
                        int32_t *argmax_out, const dm_layer_state *states, void *workspace, size_t workspace_bytes,
                        void *cuda_stream, const SampleArgs *smp = nullptr, const HybridArgs *hyb = nullptr) {
    Dims m;
    if (!cfg || !weights) return fail(DM_ERR_INVALID_ARG, "cfg or weights is NULL");
    int st = check_cfg(&cfg->mixer, &m);
    if (st != DM_OK) return st;
    if (cfg->n_layers <= 0 || cfg->vocab <= 0) return fail(DM_ERR_INVALID_ARG, "n_layers and vocab must be positive");
    if (!(cfg->rms_eps >= 0.f)) return fail(DM_ERR_INVALID_ARG, "rms_eps must be >= 0");
    if (!tokens) return fail(DM_ERR_INVALID_ARG, "tokens is NULL");
    if (!logits && !argmax_out && !smp) return fail(DM_ERR_INVALID_ARG, "logits and argmax_out are both NULL");
    if (smp) {
        if (!smp->cfg || !smp->u_keep || !smp->u_cat || !smp->tokens_out) return fail(DM_ERR_INVALID_ARG, "NULL pointer in the sampling arguments");
        if (smp->tokens_out == tokens) return fail(DM_ERR_INVALID_ARG, "tokens_out must not be tokens_in");
        const dm_sample_cfg &q = *smp->cfg;
        if (q.vocab_real <= 0 || q.vocab_real > cfg->vocab || q.mask_id < 0 || q.mask_id >= cfg->vocab)
            return fail(DM_ERR_INVALID_ARG, "vocab_real must be in (0, vocab], mask_id in [0, vocab)");
        if (q.vocab_real == 1 && q.mask_id == 0) return fail(DM_ERR_INVALID_ARG, "no token left to draw");
        if (!(q.keep_prob >= 0.f && q.keep_prob <= 1.f)) return fail(DM_ERR_INVALID_ARG, "keep_prob must be in [0, 1]");
    }
    if (!weights->embed || !weights->layers || !weights->final_norm_w || !weights->w_vocab)
        return fail(DM_ERR_INVALID_ARG, "NULL pointer in stack weights");
    if (!aligned16(weights->embed) || !aligned16(weights->w_vocab) || !aligned16(logits))
        return fail(DM_ERR_INVALID_ARG, "embed, w_vocab and logits must be 16-byte aligned");
    if (logits && (((size_t)cfg->vocab * m.es) % 16)) return fail(DM_ERR_UNSUPPORTED, "vocab*sizeof(dtype) must be a multiple of 16");
    if (blk) {
        if (!bw || !tau) return fail(DM_ERR_INVALID_ARG, "block weights or tau is NULL");
        if (blk->d_ff <= 0 || blk->d_cond <= 0 || !(blk->ln_eps >= 0.f)) return fail(DM_ERR_INVALID_ARG, "d_ff and d_cond must be positive, ln_eps >= 0");
        if (m.d % 4) return fail(DM_ERR_UNSUPPORTED, "the conditioned block needs d_model to be a multiple of 4");
        if (!aligned16(tau)) return fail(DM_ERR_INVALID_ARG, "tau must be 16-byte aligned");
        for (int i = 0; i < cfg->n_layers; ++i) {
            const dm_block_weights &q = bw[i];
            if (!q.w_cond || !q.w_up || !q.w_down) return fail(DM_ERR_INVALID_ARG, "layer %d: NULL pointer in block weights", i);
            if (!aligned16(q.w_cond) || !aligned16(q.w_up) || !aligned16(q.w_down) || !aligned16(q.b_cond) || !aligned16(q.b_up) || !aligned16(q.b_down))
                return fail(DM_ERR_INVALID_ARG, "layer %d: block weights must be 16-byte aligned", i);
        }
    }
    const int period = hyb ? hyb->cfg->attn_period : 0;
    if (hyb) {
        if (!hyb->cfg || !hyb->aw) return fail(DM_ERR_INVALID_ARG, "hybrid configuration or attention weights are NULL");
        if (period < 0) return fail(DM_ERR_INVALID_ARG, "attn_period must be >= 0");
        if (period > 0) {
            if (states && !hyb->ast) return fail(DM_ERR_INVALID_ARG, "block mode needs the key/value caches of the attention layers");
            if (hyb->ast)
                for (int i = 0; i < cfg->n_layers; i += period) {
                    const dm_attn_state &q = hyb->ast[i];
                    if (!q.k_cache || !q.v_cache || !aligned16(q.k_cache) || !aligned16(q.v_cache))
                        return fail(DM_ERR_INVALID_ARG, "layer %d: key/value caches must be non-NULL and 16-byte aligned", i);
                    if (q.len < 0 || q.len + m.L > q.cap) return fail(DM_ERR_INVALID_ARG, "layer %d: cache length + block length exceeds its capacity", i);
                }
            if (hyb->cfg->attn_heads <= 0 || !attention_supports(cfg->mixer.dtype, m.d, hyb->cfg->attn_heads))
                return fail(DM_ERR_UNSUPPORTED, "attention layers need bf16 and heads of width 64 or 80 (d_model = 64 or 80 * attn_heads)");
            for (int i = 0; i < cfg->n_layers; i += period)
                if (!hyb->aw[i].w_qkv || !hyb->aw[i].w_o || !aligned16(hyb->aw[i].w_qkv) || !aligned16(hyb->aw[i].w_o))
                    return fail(DM_ERR_INVALID_ARG, "layer %d: attention weights must be non-NULL and 16-byte aligned", i);
        }
    }
    for (int i = 0; i < cfg->n_layers; ++i) {
        if (!blk && !weights->layers[i].norm_w) return fail(DM_ERR_INVALID_ARG, "layer %d: norm_w is NULL", i);
        if (period > 0 && i % period == 0) continue;          // an attention layer: its Mamba weights are not read
        if ((st = check_weights(&cfg->mixer, weights->layers[i].dir)) != DM_OK) return st;
        if (states) {
            const dm_layer_state &q = states[i];
            if ((q.ssm_in && q.ssm_in == q.ssm_out) || (q.conv_in && q.conv_in == q.conv_out))
                return fail(DM_ERR_INVALID_ARG, "layer %d: state_in and state_out must be different buffers", i);
            if (!aligned16(q.ssm_in) || !aligned16(q.ssm_out) || !aligned16(q.conv_in) || !aligned16(q.conv_out))
                return fail(DM_ERR_INVALID_ARG, "layer %d: states must be 16-byte aligned", i);
            if ((q.ssm_out || q.conv_out) && !(cfg->mixer.dir_mask & DM_DIR_FWD))
                return fail(DM_ERR_INVALID_ARG, "state_out needs the left-to-right direction");
        }
    }
    const StackWs l = stack_ws(cfg, m, blk, smp != nullptr, period > 0);
    if ((st = check_ws(workspace, workspace_bytes, l.total)) != DM_OK) return st;
    char *ws = static_cast<char *>(workspace);
    float *r = reinterpret_cast<float *>(ws + l.r);
    float *mod = reinterpret_cast<float *>(ws + l.mod);
    void *u = ws + l.u;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const int dtype = cfg->mixer.dtype;
    cudaError_t e;

    if ((e = embed_gather(weights->embed, dtype, tokens, r, (int)m.T, m.d, cfg->vocab, s)) != cudaSuccess) return cuda_fail(e, "embed");
    bool u_ready = false;                         // u already holds the norm of r (applied by the previous layer's last pass)
    for (int i = 0; i < cfg->n_layers; ++i) {
        const dm_layer_weights &lw = weights->layers[i];
        MixerOut out{r, DM_F32, r, m.d};          // r <- r + Mamba(u): the residual add rides in the out_proj epilogue
        const int64_t ldm = 6 * (int64_t)m.d;     // modulation row: [beta1 | gamma1 | gate1 | beta2 | gamma2 | gate2]
        if (blk) {
            if ((e = modulation_rows(tau, bw[i].w_cond, bw[i].b_cond, mod, dtype, m.B, 6 * m.d, blk->d_cond, s)) != cudaSuccess) return cuda_fail(e, "modulation");
            if ((e = adaln_rows(r, mod + m.d, mod, ldm, u, dtype, (int)m.T, m.L, m.d, blk->ln_eps, s)) != cudaSuccess) return cuda_fail(e, "adaln");
            out.col_scale = mod + 2 * m.d; out.cs_rows = m.L; out.ld_cs = ldm;
        } else {
            if (!u_ready && (e = rmsnorm_rows(r, lw.norm_w, u, dtype, (int)m.T, m.d, cfg->rms_eps, s)) != cudaSuccess) return cuda_fail(e, "rmsnorm");
            // what follows this layer's mixer is the next layer's (or the final) RMSNorm of r
            out.next_norm_w = i + 1 < cfg->n_layers ? weights->layers[i + 1].norm_w : weights->final_norm_w;
            out.next_u = u; out.next_eps = cfg->rms_eps; out.next_done = &u_ready;
        }
        u_ready = false;
        if (period > 0 && i % period == 0) {
            // attention mixer (Sec. 3.3): r <- r + [gate *] Attn(u); gate and residual ride in the output projection's epilogue
            void *qkv = ws + l.qkv, *att = ws + l.att;
            GemmArgs a{};
            a.A = u; a.lda = m.d; a.B = hyb->aw[i].w_qkv; a.ldb = m.d; a.C = qkv; a.ldc = 3 * m.d;
            a.in_dtype = dtype; a.c_dtype = dtype; a.M = (int)m.T; a.N = 3 * m.d; a.K = m.d;
            if ((e = gemm(a, s)) != cudaSuccess) return cuda_fail(e, "qkv projection");
            if ((e = attention_forward(qkv, att, m.B, m.L, m.d, hyb->cfg->attn_heads, hyb->ast ? hyb->ast[i].k_cache : nullptr,
                                       hyb->ast ? hyb->ast[i].v_cache : nullptr, hyb->ast ? hyb->ast[i].len : 0, hyb->ast ? hyb->ast[i].cap : 0, s)) != cudaSuccess) return cuda_fail(e, "attention");
            GemmArgs o{};
            o.A = att; o.lda = m.d; o.B = hyb->aw[i].w_o; o.ldb = m.d; o.C = r; o.ldc = m.d;
            o.in_dtype = dtype; o.c_dtype = DM_F32; o.M = (int)m.T; o.N = m.d; o.K = m.d;
            o.addend = r; o.ld_add = m.d; o.col_scale = out.col_scale; o.cs_rows = out.cs_rows; o.ld_cs = out.ld_cs;
            if ((e = gemm(o, s)) != cudaSuccess) return cuda_fail(e, "attention output projection");
        } else {
            const dm_layer_state *q = states ? &states[i] : nullptr;
            st = run_mixer(&cfg->mixer, m, lw.dir, u, out, q ? q->ssm_in : nullptr, q ? q->conv_in : nullptr,
                           q ? q->ssm_out : nullptr, q ? q->conv_out : nullptr, ws + l.mixer, s);
            if (st != DM_OK) return st;
        }
        if (blk) {
            // r <- r + gate2 * (W_down GELU(W_up AdaLN(r) + b_up) + b_down): activation, bias, gate and residual ride in the epilogues
            if ((e = adaln_rows(r, mod + 4 * m.d, mod + 3 * m.d, ldm, u, dtype, (int)m.T, m.L, m.d, blk->ln_eps, s)) != cudaSuccess) return cuda_fail(e, "adaln");
            void *hmid = ws + l.hmid;
            GemmArgs up{};
            up.A = u; up.lda = m.d; up.B = bw[i].w_up; up.ldb = m.d; up.C = hmid; up.ldc = blk->d_ff;
            up.in_dtype = dtype; up.c_dtype = dtype; up.M = (int)m.T; up.N = blk->d_ff; up.K = m.d;
            up.col_bias = bw[i].b_up; up.gelu = 1;
            if ((e = gemm(up, s)) != cudaSuccess) return cuda_fail(e, "mlp up");
            GemmArgs dn{};
            dn.A = hmid; dn.lda = blk->d_ff; dn.B = bw[i].w_down; dn.ldb = blk->d_ff; dn.C = r; dn.ldc = m.d;
            dn.in_dtype = dtype; dn.c_dtype = DM_F32; dn.M = (int)m.T; dn.N = m.d; dn.K = blk->d_ff;
            dn.col_bias = bw[i].b_down; dn.col_scale = mod + 5 * m.d; dn.cs_rows = m.L; dn.ld_cs = ldm;
            dn.addend = r; dn.ld_add = m.d;
            if ((e = gemm(dn, s)) != cudaSuccess) return cuda_fail(e, "mlp down");
        }
    }
    if (!u_ready && (e = rmsnorm_rows(r, weights->final_norm_w, u, dtype, (int)m.T, m.d, cfg->rms_eps, s)) != cudaSuccess) return cuda_fail(e, "final norm");
    if (smp) {
        // Eq. 3: only the positions drawn this step go through the vocabulary projection; how many there are stays on the device
        int32_t *idx = reinterpret_cast<int32_t *>(ws + l.idx);
        int *count = reinterpret_cast<int *>(ws + l.count);
        void *ug = ws + l.ug;
        const dm_sample_cfg &q = *smp->cfg;
        if ((e = select_drawn(tokens, smp->u_keep, q.keep_prob, q.mask_id, smp->tokens_out, idx, count, (int)m.T, s)) != cudaSuccess) return cuda_fail(e, "select");
        if ((e = gather_rows(u, idx, count, ug, dtype, (int)m.T, m.d, s)) != cudaSuccess) return cuda_fail(e, "gather");
        for (int64_t t0 = 0; t0 < m.T; t0 += l.logits_rows) {
            const int rows = (int)((m.T - t0) < l.logits_rows ? (m.T - t0) : l.logits_rows);
            GemmArgs a{};
            a.A = static_cast<char *>(ug) + (size_t)t0 * m.d * m.es; a.lda = m.d;
            a.B = weights->w_vocab; a.ldb = m.d;
            a.C = ws + l.logits; a.ldc = cfg->vocab;
            a.in_dtype = dtype; a.c_dtype = dtype; a.M = rows; a.N = cfg->vocab; a.K = m.d;
            a.m_dev = count; a.m_off = (int)t0;
            if ((e = gemm(a, s)) != cudaSuccess) return cuda_fail(e, "vocab projection");
            if ((e = draw_rows(a.C, cfg->vocab, dtype, idx, count, (int)t0, rows, smp->u_cat, q.mask_id, q.vocab_real, smp->tokens_out, s)) != cudaSuccess)
                return cuda_fail(e, "draw");
        }
        return DM_OK;
    }
    const int64_t rows_per = logits ? m.T : l.logits_rows;
    for (int64_t t0 = 0; t0 < m.T; t0 += rows_per) {
        const int rows = (int)((m.T - t0) < rows_per ? (m.T - t0) : rows_per);
        GemmArgs a{};
        a.A = static_cast<char *>(u) + (size_t)t0 * m.d * m.es; a.lda = m.d;
        a.B = weights->w_vocab; a.ldb = m.d;
        a.C = logits ? static_cast<char *>(logits) + (size_t)t0 * cfg->vocab * m.es : ws + l.logits; a.ldc = cfg->vocab;
        a.in_dtype = dtype; a.c_dtype = dtype; a.M = rows; a.N = cfg->vocab; a.K = m.d;
        if ((e = gemm(a, s)) != cudaSuccess) return cuda_fail(e, "vocab projection");
        if (argmax_out && (e = argmax_rows(a.C, dtype, argmax_out + t0, rows, cfg->vocab, s)) != cudaSuccess) return cuda_fail(e, "argmax");
    }
    return DM_OK;
}

extern "C" {

int dm_denoise_step(const dm_stack_cfg *cfg, const dm_stack_weights *weights, const int32_t *tokens, void *logits,
                    int32_t *argmax_out, const dm_layer_state *states, void *workspace, size_t workspace_bytes,
                    void *cuda_stream) {
    return denoise_impl(cfg, nullptr, weights, nullptr, tokens, nullptr, logits, argmax_out, states, workspace, workspace_bytes, cuda_stream);
}

int dm_denoise_cond_workspace_bytes(const dm_stack_cfg *cfg, const dm_block_cfg *blk, size_t *bytes) {
    Dims m;
    if (!cfg || !blk || !bytes) return fail(DM_ERR_INVALID_ARG, "NULL argument");
    int st = check_cfg(&cfg->mixer, &m);
    if (st != DM_OK) return st;
    if (cfg->vocab <= 0 || blk->d_ff <= 0) return fail(DM_ERR_INVALID_ARG, "vocab and d_ff must be positive");
    *bytes = stack_ws(cfg, m, blk).total;
    return DM_OK;
}

int dm_denoise_step_cond(const dm_stack_cfg *cfg, const dm_block_cfg *blk, const dm_stack_weights *weights,
                         const dm_block_weights *block_weights, const int32_t *tokens, const float *tau, void *logits,
                         int32_t *argmax_out, const dm_layer_state *states, void *workspace, size_t workspace_bytes,
                         void *cuda_stream) {
    if (!blk) return fail(DM_ERR_INVALID_ARG, "block configuration is NULL");
    return denoise_impl(cfg, blk, weights, block_weights, tokens, tau, logits, argmax_out, states, workspace, workspace_bytes, cuda_stream);
}

int dm_denoise_sample_workspace_bytes(const dm_stack_cfg *cfg, const dm_block_cfg *blk, size_t *bytes) {
    Dims m;
    if (!cfg || !bytes) return fail(DM_ERR_INVALID_ARG, "NULL argument");
    int st = check_cfg(&cfg->mixer, &m);
    if (st != DM_OK) return st;
    if (cfg->vocab <= 0 || (blk && blk->d_ff <= 0)) return fail(DM_ERR_INVALID_ARG, "vocab and d_ff must be positive");
    *bytes = stack_ws(cfg, m, blk, true).total;
    return DM_OK;
}

int dm_denoise_sample_step(const dm_stack_cfg *cfg, const dm_block_cfg *blk, const dm_stack_weights *weights,
                           const dm_block_weights *block_weights, const int32_t *tokens_in, const float *tau,
                           const dm_sample_cfg *sample, const float *u_keep, const float *u_cat, int32_t *tokens_out,
                           const dm_layer_state *states, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    const SampleArgs smp{sample, u_keep, u_cat, tokens_out};
    return denoise_impl(cfg, blk, weights, block_weights, tokens_in, tau, nullptr, nullptr, states, workspace, workspace_bytes, cuda_stream, &smp);
}

int dm_generate_workspace_bytes(const dm_stack_cfg *cfg, const dm_block_cfg *blk, size_t *bytes) {
    size_t n = 0;
    if (!bytes) return fail(DM_ERR_INVALID_ARG, "NULL argument");
    int st = dm_denoise_sample_workspace_bytes(cfg, blk, &n);
    if (st != DM_OK) return st;
    *bytes = n + align_up((size_t)cfg->mixer.batch * cfg->mixer.seqlen * sizeof(int32_t));       // + the second token buffer of the ping-pong
    return DM_OK;
}

int dm_generate(const dm_stack_cfg *cfg, const dm_block_cfg *blk, const dm_stack_weights *weights,
                const dm_block_weights *block_weights, const dm_generate_cfg *gen, const int32_t *tokens_in,
                const float *tau, const float *u_keep, const float *u_cat, int32_t *tokens_out, int32_t *trace,
                void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!cfg || !gen) return fail(DM_ERR_INVALID_ARG, "cfg or gen is NULL");
    if (gen->steps < 1 || !(gen->t_eps > 0.f && gen->t_eps < 1.f)) return fail(DM_ERR_INVALID_ARG, "steps must be >= 1 and t_eps in (0, 1)");
    if (!tokens_in || !tokens_out || !u_keep || !u_cat) return fail(DM_ERR_INVALID_ARG, "NULL pointer in the generation arguments");
    if (tokens_in == tokens_out) return fail(DM_ERR_INVALID_ARG, "tokens_out must not be tokens_in");
    size_t need = 0, step_ws = 0;
    int st = dm_generate_workspace_bytes(cfg, blk, &need);
    if (st != DM_OK) return st;
    if ((st = dm_denoise_sample_workspace_bytes(cfg, blk, &step_ws)) != DM_OK) return st;
    if ((st = check_ws(workspace, workspace_bytes, need)) != DM_OK) return st;
    const int64_t T = (int64_t)cfg->mixer.batch * cfg->mixer.seqlen;
    int32_t *spare = reinterpret_cast<int32_t *>(static_cast<char *>(workspace) + step_ws);
    const int K = gen->steps, n_calls = K + 1;
    const int32_t *cur = tokens_in;
    for (int k = 0; k < n_calls; ++k) {
        // noise levels in double, the ratio rounded once to the float the decision u_keep < s/t is taken with
        const double tk = 1.0 - (1.0 - (double)gen->t_eps) * k / K, tk1 = 1.0 - (1.0 - (double)gen->t_eps) * (k + 1) / K;
        const dm_sample_cfg sc{gen->mask_id, gen->vocab_real, k < K ? (float)(tk1 / tk) : 0.f};
        // destinations alternate so that the last step writes tokens_out (or follow the trace, copied out at the end)
        int32_t *dst = trace ? trace + (int64_t)k * T : (((n_calls - 1 - k) & 1) ? spare : tokens_out);
        const SampleArgs smp{&sc, u_keep + (int64_t)k * T, u_cat + (int64_t)k * T, dst};
        st = denoise_impl(cfg, blk, weights, block_weights, cur, (blk && tau) ? tau + (int64_t)k * cfg->mixer.batch * blk->d_cond : tau,
                          nullptr, nullptr, nullptr, workspace, step_ws, cuda_stream, &smp);
        if (st != DM_OK) return st;
        cur = dst;
    }
    if (trace) {
        cudaError_t e = cudaMemcpyAsync(tokens_out, cur, (size_t)T * sizeof(int32_t), cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(cuda_stream));
        if (e != cudaSuccess) return cuda_fail(e, "dm_generate: copy of the result");
    }
    return DM_OK;
}

int dm_denoise_hybrid_workspace_bytes(const dm_stack_cfg *cfg, const dm_block_cfg *blk, size_t *bytes) {
    Dims m;
    if (!cfg || !bytes) return fail(DM_ERR_INVALID_ARG, "NULL argument");
    int st = check_cfg(&cfg->mixer, &m);
    if (st != DM_OK) return st;
    if (cfg->vocab <= 0 || (blk && blk->d_ff <= 0)) return fail(DM_ERR_INVALID_ARG, "vocab and d_ff must be positive");
    *bytes = stack_ws(cfg, m, blk, false, true).total;
    return DM_OK;
}

int dm_denoise_step_hybrid(const dm_stack_cfg *cfg, const dm_block_cfg *blk, const dm_hybrid_cfg *hybrid,
                           const dm_stack_weights *weights, const dm_block_weights *block_weights,
                           const dm_attn_weights *attn_weights, const int32_t *tokens, const float *tau, void *logits,
                           int32_t *argmax_out, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!hybrid) return fail(DM_ERR_INVALID_ARG, "hybrid configuration is NULL");
    const HybridArgs hyb{hybrid, attn_weights};
    return denoise_impl(cfg, blk, weights, block_weights, tokens, tau, logits, argmax_out, nullptr, workspace, workspace_bytes, cuda_stream,
                        nullptr, &hyb);
}

int dm_denoise_step_hybrid_block(const dm_stack_cfg *cfg, const dm_block_cfg *blk, const dm_hybrid_cfg *hybrid,
                                 const dm_stack_weights *weights, const dm_block_weights *block_weights,
                                 const dm_attn_weights *attn_weights, const int32_t *tokens, const float *tau, void *logits,
                                 int32_t *argmax_out, const dm_layer_state *states, const dm_attn_state *attn_states,
                                 void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!hybrid) return fail(DM_ERR_INVALID_ARG, "hybrid configuration is NULL");
    HybridArgs hyb{hybrid, attn_weights};
    hyb.ast = attn_states;
    return denoise_impl(cfg, blk, weights, block_weights, tokens, tau, logits, argmax_out, states, workspace, workspace_bytes, cuda_stream,
                        nullptr, &hyb);
}

int dm_attention_block_step(int32_t batch, int32_t block_len, int32_t d_model, int32_t n_heads, int32_t dtype, const void *w_qkv,
                            const void *w_o, const void *x_blk, void *k_cache, void *v_cache, int32_t cache_len, int32_t cache_cap,
                            void *y_blk, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    size_t need = 0;
    int st = dm_attention_workspace_bytes(batch, block_len, d_model, dtype, &need);
    if (st != DM_OK) return st;
    if (!w_qkv || !w_o || !x_blk || !y_blk || !k_cache || !v_cache) return fail(DM_ERR_INVALID_ARG, "NULL pointer");
    if (x_blk == y_blk) return fail(DM_ERR_INVALID_ARG, "y must not alias x");
    if (!aligned16(w_qkv) || !aligned16(w_o) || !aligned16(x_blk) || !aligned16(y_blk) || !aligned16(k_cache) || !aligned16(v_cache))
        return fail(DM_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    if (n_heads <= 0 || (d_model != n_heads * 64 && d_model != n_heads * 80))
        return fail(DM_ERR_UNSUPPORTED, "the attention mixer needs heads of width 64 or 80 (d_model = 64 or 80 * n_heads)");
    if (batch > 65535 || n_heads > 65535) return fail(DM_ERR_UNSUPPORTED, "batch and n_heads must be below 65536");
    if (cache_len < 0 || cache_len + block_len > cache_cap) return fail(DM_ERR_INVALID_ARG, "cache length + block length exceeds the cache's capacity");
    if (!attention_supports(dtype, d_model, n_heads)) return fail(DM_ERR_UNSUPPORTED, "the attention mixer is not available for this configuration");
    if ((st = check_ws(workspace, workspace_bytes, need)) != DM_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const int64_t T = (int64_t)batch * block_len;
    char *ws = static_cast<char *>(workspace);
    void *qkv = ws, *att = ws + align_up((size_t)T * 3 * d_model * 2);
    GemmArgs a{};
    a.A = x_blk; a.lda = d_model; a.B = w_qkv; a.ldb = d_model; a.C = qkv; a.ldc = 3 * d_model;
    a.in_dtype = dtype; a.c_dtype = dtype; a.M = (int)T; a.N = 3 * d_model; a.K = d_model;
    cudaError_t e;
    if ((e = gemm(a, s)) != cudaSuccess) return cuda_fail(e, "qkv projection");
    if ((e = attention_forward(qkv, att, batch, block_len, d_model, n_heads, k_cache, v_cache, cache_len, cache_cap, s)) != cudaSuccess)
        return cuda_fail(e, "attention");
    GemmArgs o{};
    o.A = att; o.lda = d_model; o.B = w_o; o.ldb = d_model; o.C = y_blk; o.ldc = d_model;
    o.in_dtype = dtype; o.c_dtype = dtype; o.M = (int)T; o.N = d_model; o.K = d_model;
    if ((e = gemm(o, s)) != cudaSuccess) return cuda_fail(e, "attention output projection");
    return DM_OK;
}

int dm_attention_workspace_bytes(int32_t batch, int32_t seqlen, int32_t d_model, int32_t dtype, size_t *bytes) {
    if (!bytes || batch <= 0 || seqlen <= 0 || d_model <= 0) return fail(DM_ERR_INVALID_ARG, "sizes must be positive");
    if (dtype != DM_BF16) return fail(DM_ERR_UNSUPPORTED, "the attention mixer takes bf16 only");
    *bytes = align_up((size_t)batch * seqlen * 3 * d_model * 2) + align_up((size_t)batch * seqlen * d_model * 2);
    return DM_OK;
}

int dm_attention_forward(int32_t batch, int32_t seqlen, int32_t d_model, int32_t n_heads, int32_t dtype, const void *w_qkv,
                         const void *w_o, const void *x, void *y, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    size_t need = 0;
    int st = dm_attention_workspace_bytes(batch, seqlen, d_model, dtype, &need);
    if (st != DM_OK) return st;
    if (!w_qkv || !w_o || !x || !y) return fail(DM_ERR_INVALID_ARG, "NULL pointer");
    if (x == y) return fail(DM_ERR_INVALID_ARG, "y must not alias x");
    if (!aligned16(w_qkv) || !aligned16(w_o) || !aligned16(x) || !aligned16(y)) return fail(DM_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    if (n_heads <= 0 || (d_model != n_heads * 64 && d_model != n_heads * 80))
        return fail(DM_ERR_UNSUPPORTED, "the attention mixer needs heads of width 64 or 80 (d_model = 64 or 80 * n_heads)");
    if (batch > 65535 || n_heads > 65535) return fail(DM_ERR_UNSUPPORTED, "batch and n_heads must be below 65536");
    if (!attention_supports(dtype, d_model, n_heads)) return fail(DM_ERR_UNSUPPORTED, "the attention mixer is not available for this configuration");
    if ((st = check_ws(workspace, workspace_bytes, need)) != DM_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const int64_t T = (int64_t)batch * seqlen;
    char *ws = static_cast<char *>(workspace);
    void *qkv = ws, *att = ws + align_up((size_t)T * 3 * d_model * 2);
    GemmArgs a{};
    a.A = x; a.lda = d_model; a.B = w_qkv; a.ldb = d_model; a.C = qkv; a.ldc = 3 * d_model;
    a.in_dtype = dtype; a.c_dtype = dtype; a.M = (int)T; a.N = 3 * d_model; a.K = d_model;
    cudaError_t e;
    if ((e = gemm(a, s)) != cudaSuccess) return cuda_fail(e, "qkv projection");
    if ((e = attention_forward(qkv, att, batch, seqlen, d_model, n_heads, nullptr, nullptr, 0, 0, s)) != cudaSuccess) return cuda_fail(e, "attention");
    GemmArgs o{};
    o.A = att; o.lda = d_model; o.B = w_o; o.ldb = d_model; o.C = y; o.ldc = d_model;
    o.in_dtype = dtype; o.c_dtype = dtype; o.M = (int)T; o.N = d_model; o.K = d_model;
    if ((e = gemm(o, s)) != cudaSuccess) return cuda_fail(e, "attention output projection");
    return DM_OK;
}

int dm_selftest_withhold_prep(int on) {
    scan_ssd_selftest_withhold(on);
    return DM_OK;
}

int dm_selftest_wait_timeout(uint32_t limit_us, uint64_t *out, void *cuda_stream) {
    if (!out) return fail(DM_ERR_INVALID_ARG, "out is NULL");
    if (limit_us == 0 || limit_us > 1000000u) return fail(DM_ERR_INVALID_ARG, "limit_us must be in [1, 1000000]");
    if (reinterpret_cast<uintptr_t>(out) & 7u) return fail(DM_ERR_INVALID_ARG, "out must be 8-byte aligned");
    cudaError_t e = selftest_wait_timeout((unsigned long long)limit_us * 1000ull, reinterpret_cast<unsigned long long *>(out),
                                          static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(e, "dm_selftest_wait_timeout");
    return DM_OK;
}

int dm_linear(int dtype, const void *x, const void *w, void *y, int y_dtype, int64_t rows, int32_t in_features,
              int32_t out_features, const float *row_scale, const float *addend, void *cuda_stream) {
    if ((dtype != DM_F32 && dtype != DM_BF16) || (y_dtype != DM_F32 && y_dtype != DM_BF16)) return fail(DM_ERR_INVALID_ARG, "bad dtype");
    if (!x || !w || !y) return fail(DM_ERR_INVALID_ARG, "x, w or y is NULL");
    if (rows <= 0 || rows > (int64_t)1 << 30 || in_features <= 0 || out_features <= 0) return fail(DM_ERR_INVALID_ARG, "sizes must be positive");
    if (x == y) return fail(DM_ERR_INVALID_ARG, "y must not alias x");
    if (addend && static_cast<const void *>(addend) == y && y_dtype != DM_F32) return fail(DM_ERR_INVALID_ARG, "addend may alias y only for fp32 y");
    GemmArgs a{};
    a.A = x; a.lda = in_features; a.B = w; a.ldb = in_features; a.C = y; a.ldc = out_features;
    a.in_dtype = dtype; a.c_dtype = y_dtype; a.M = (int)rows; a.N = out_features; a.K = in_features;
    a.row_scale = row_scale; a.addend = addend; a.ld_add = out_features;
    cudaError_t e = gemm(a, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(e, "dm_linear");
    return DM_OK;
}

// Copy streams and events of the host-buffer entry point, one set per device, created on first use.
namespace {
constexpr int HOST_PIECES = 8, MAX_DEVICES = 64;
struct HostPipe {
    bool ready = false;
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t start = nullptr, done = nullptr, copied[HOST_PIECES] = {}, computed[HOST_PIECES] = {};
};
HostPipe *host_pipe() {
    static HostPipe pipes[MAX_DEVICES];
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return nullptr;
    std::lock_guard<std::mutex> lk(mu);
    HostPipe &p = pipes[dev];
    if (p.ready) return &p;
    bool ok = cudaStreamCreateWithFlags(&p.in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&p.out, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&p.done, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < HOST_PIECES && ok; ++i)
        ok = cudaEventCreateWithFlags(&p.copied[i], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&p.computed[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) return nullptr;
    p.ready = true;
    return &p;
}
}  // namespace

int dm_bimamba_forward_host(const dm_mixer_cfg *cfg, const dm_dir_weights w[2], const void *x_host, void *y_host,
                            void *workspace, size_t workspace_bytes, void *cuda_stream) {
    Dims m;
    int st = check_cfg(cfg, &m);
    if (st != DM_OK) return st;
    if ((st = check_weights(cfg, w)) != DM_OK) return st;        // everything the per-piece calls would reject is rejected here, before the first copy
    if (!x_host || !y_host) return fail(DM_ERR_INVALID_ARG, "x_host or y_host is NULL");
    if (x_host == y_host) return fail(DM_ERR_INVALID_ARG, "y_host must not alias x_host");
    const size_t act = align_up((size_t)m.T * m.d * m.es);
    const size_t need = mixer_ws(cfg, m).total + 2 * act;
    if ((st = check_ws(workspace, workspace_bytes, need)) != DM_OK) return st;
    char *ws = static_cast<char *>(workspace);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    char *xd = ws, *yd = ws + act;
    HostPipe *hp = host_pipe();
    if (!hp) return fail(DM_ERR_CUDA, "could not create the copy streams");
    // Batch rows are independent (Sec. 3.2: the mixer acts on each sequence separately), so the batch is cut into
    // pieces of whole rows: while piece i is computed on the caller's stream, piece i+1 is on its way in and piece
    // i-1 on its way out.  The pieces share the mixer workspace (they run one after the other on `cuda_stream`).
    // at least ~4096 tokens per piece (smaller pieces run the kernels below their full-size efficiency), at most HOST_PIECES pieces
    int rows = (int)((4096 + m.L - 1) / m.L);
    if (rows < (m.B + HOST_PIECES - 1) / HOST_PIECES) rows = (m.B + HOST_PIECES - 1) / HOST_PIECES;
    if (rows > m.B) rows = m.B;
    const int pieces = (m.B + rows - 1) / rows;
    const size_t row_bytes = (size_t)m.L * m.d * m.es;
    cudaError_t e;
    if ((e = cudaEventRecord(hp->start, s)) != cudaSuccess) return cuda_fail(e, "record");
    if ((e = cudaStreamWaitEvent(hp->in, hp->start, 0)) != cudaSuccess) return cuda_fail(e, "wait");      // after the caller's earlier work
    if ((e = cudaStreamWaitEvent(hp->out, hp->start, 0)) != cudaSuccess) return cuda_fail(e, "wait");
    dm_mixer_cfg piece_cfg = *cfg;
    // A failure after the first copy was enqueued: let the copy streams drain (their copies still read and write the
    // caller's buffers) and rejoin the caller's stream before reporting it.
    auto bail = [&](int status) {
        cudaStreamSynchronize(hp->in);
        cudaStreamSynchronize(hp->out);
        cudaStreamSynchronize(s);
        return status;
    };
    for (int i = 0; i < pieces; ++i) {
        const int r0 = i * rows, nr = (r0 + rows <= m.B) ? rows : m.B - r0;
        const size_t off = (size_t)r0 * row_bytes, bytes = (size_t)nr * row_bytes;
        if ((e = cudaMemcpyAsync(xd + off, static_cast<const char *>(x_host) + off, bytes, cudaMemcpyHostToDevice, hp->in)) != cudaSuccess)
            return bail(cuda_fail(e, "copy x to the device"));
        if ((e = cudaEventRecord(hp->copied[i], hp->in)) != cudaSuccess) return bail(cuda_fail(e, "record"));
        if ((e = cudaStreamWaitEvent(s, hp->copied[i], 0)) != cudaSuccess) return bail(cuda_fail(e, "wait"));
        piece_cfg.batch = nr;
        st = dm_bimamba_forward(&piece_cfg, w, xd + off, yd + off, ws + 2 * act, workspace_bytes - 2 * act, cuda_stream);
        if (st != DM_OK) return bail(st);
        if ((e = cudaEventRecord(hp->computed[i], s)) != cudaSuccess) return bail(cuda_fail(e, "record"));
        if ((e = cudaStreamWaitEvent(hp->out, hp->computed[i], 0)) != cudaSuccess) return bail(cuda_fail(e, "wait"));
        if ((e = cudaMemcpyAsync(static_cast<char *>(y_host) + off, yd + off, bytes, cudaMemcpyDeviceToHost, hp->out)) != cudaSuccess)
            return bail(cuda_fail(e, "copy y to the host"));
    }
    if ((e = cudaEventRecord(hp->done, hp->out)) != cudaSuccess) return bail(cuda_fail(e, "record"));
    if ((e = cudaStreamWaitEvent(s, hp->done, 0)) != cudaSuccess) return bail(cuda_fail(e, "wait"));
    if ((e = cudaStreamSynchronize(s)) != cudaSuccess) return bail(cuda_fail(e, "synchronize"));
    return DM_OK;
}

}  // extern "C"
