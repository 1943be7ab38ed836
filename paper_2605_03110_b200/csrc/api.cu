// C ABI of libada.so: argument checks, workspace, kernel sequencing.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <new>

#include "common.cuh"

using namespace ada;

namespace {

const char* const kKernelNames[K_COUNT] = {
    "norm_gather",     "gram_ffma_tri",    "gram_ffma_cross",
    "gram_tc_tri",     "gram_tc_cross",    "gram_tc_cascade", "split_bf16x3",  "compact_full",
    "compact_cascade", "nearest_finish",
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

ada_status check_common(ada_ctx* ctx, const void* X, int64_t B, int64_t T, int64_t d, int64_t ldx,
                        ada_dtype dt) {
    if (ctx == nullptr || X == nullptr) return ADA_ERR_INVALID_ARG;
    if (B < 1 || T < 1 || d < 1 || ldx < d) return ADA_ERR_INVALID_ARG;
    if (dt != ADA_F32 && dt != ADA_BF16) return ADA_ERR_INVALID_ARG;
    if (dt != ctx->dt) return ADA_ERR_UNSUPPORTED;
    if (B > ctx->maxB || T > ctx->maxT || d > ctx->maxd) return ADA_ERR_WORKSPACE;
    const int64_t es = dt == ADA_F32 ? 4 : 2;
    if (!aligned16(X) || (ldx * es) % 16 != 0 || (d * es) % 16 != 0) return ADA_ERR_UNSUPPORTED;
    return ADA_OK;
}

inline bool tau_ok(double tau) { return tau > 0.0 && tau < 1.0; }  // also rejects NaN

struct DeviceGuard {
    int prev = -1;
    explicit DeviceGuard(int dev) {
        cudaGetDevice(&prev);
        if (prev != dev) cudaSetDevice(dev);
        else prev = -1;
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

bool use_tc(const ada_ctx* ctx, ada_dtype dt) {
    if (dt != ADA_BF16) return false;
    if (ctx->engine == ADA_ENGINE_FFMA) return false;
    return gram_tc_available();
}

// fp32 storage on the bf16 tensor cores through the three-term split
bool use_split(const ada_ctx* ctx, ada_dtype dt) {
    return dt == ADA_F32 && ctx->engine != ADA_ENGINE_FFMA && ctx->splitXA != nullptr &&
           gram_tc_available();
}

// the pair-CTA form of the tensor-core kernel, or the one-CTA form?
bool use_pair(const ada_ctx* ctx, int64_t B, int64_t T, int64_t d) {
    if (ctx->engine == ADA_ENGINE_TCGEN05_PAIR) return true;
    // The pair kernel pays off from a few thousand rows and a long contraction on (measured on
    // the crossover sweep: at T = 4096, d = 4096 both calls are faster on it, at T = 2048 they
    // are not); small problems are covered better by the finer one-CTA tiles.
    return ctx->engine == ADA_ENGINE_AUTO && B * T >= 4096 && d >= 2048;
}

// tensor-core launch of one or two segments, in the one-CTA or the pair-CTA form
cudaError_t launch_tc(ada_ctx* ctx, const GramProblem* tri, const GramProblem* cross,
                      const NormJob* norms, cudaStream_t s) {
    const GramProblem* p = cross != nullptr ? cross : tri;
    if (use_pair(ctx, p->B, p->rows, p->d)) return launch_gram_tc2(ctx, tri, cross, norms, nullptr, s);
    return launch_gram_tc(ctx, tri, cross, norms, s);
}

cudaError_t run_gram(ada_ctx* ctx, const GramProblem& p, ada_dtype dt, cudaStream_t s) {
    if (use_tc(ctx, dt)) return p.tri ? launch_tc(ctx, &p, nullptr, nullptr, s) : launch_tc(ctx, nullptr, &p, nullptr, s);
    return launch_gram_ffma(ctx, p, dt, s);
}

#define CU(x)                                  \
    do {                                       \
        cudaError_t e__ = (x);                 \
        if (e__ != cudaSuccess) return ADA_ERR_CUDA; \
    } while (0)

}  // namespace

namespace ada {

void prof_begin(ada_ctx* ctx, int kid, cudaStream_t s) {
    Profiler& pr = ctx->prof;
    if (!pr.on || pr.n >= Profiler::MAXREC) return;
    if (pr.n >= pr.created) {
        cudaEventCreate(&pr.ev0[pr.n]);
        cudaEventCreate(&pr.ev1[pr.n]);
        pr.created = pr.n + 1;
    }
    pr.kid[pr.n] = kid;
    cudaEventRecord(pr.ev0[pr.n], s);
}

void prof_end(ada_ctx* ctx, cudaStream_t s) {
    Profiler& pr = ctx->prof;
    if (!pr.on || pr.n >= Profiler::MAXREC) return;
    cudaEventRecord(pr.ev1[pr.n], s);
    ++pr.n;
}

}  // namespace ada

extern "C" {

const char* ada_status_string(ada_status s) {
    switch (s) {
        case ADA_OK: return "ADA_OK";
        case ADA_ERR_INVALID_ARG: return "ADA_ERR_INVALID_ARG";
        case ADA_ERR_UNSUPPORTED: return "ADA_ERR_UNSUPPORTED";
        case ADA_ERR_WORKSPACE: return "ADA_ERR_WORKSPACE";
        case ADA_ERR_CUDA: return "ADA_ERR_CUDA";
        case ADA_ERR_BAD_INDEX_SET: return "ADA_ERR_BAD_INDEX_SET";
        case ADA_ERR_NONFINITE: return "ADA_ERR_NONFINITE";
        case ADA_ERR_TIMEOUT: return "ADA_ERR_TIMEOUT";
        case ADA_ERR_BAD_TAU: return "ADA_ERR_BAD_TAU";
    }
    return "ADA_ERR_UNKNOWN";
}

uint64_t ada_gram_op_count(int cascade, int64_t T, int64_t d, int64_t r) {
    if (T < 0 || d < 0 || r < 0) return 0;
    const uint64_t t = (uint64_t)T, dd = (uint64_t)d, rr = (uint64_t)r;
    if (!cascade) return t * t * dd;
    if (r > T) return 0;
    return rr * rr * dd + (t - rr) * rr * dd;
}

ada_status ada_create(ada_ctx** out, int device, int64_t maxB, int64_t maxT, int64_t maxd,
                      ada_dtype dt) {
    if (out == nullptr) return ADA_ERR_INVALID_ARG;
    *out = nullptr;
    if (maxB < 1 || maxT < 1 || maxd < 1 || (dt != ADA_F32 && dt != ADA_BF16))
        return ADA_ERR_INVALID_ARG;
    // the compaction packs three per-sequence counts into 21-bit fields
    if (maxT > ADA_MAX_T || maxB * maxT > (int64_t)1 << 30) return ADA_ERR_INVALID_ARG;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev)
        return ADA_ERR_CUDA;
    DeviceGuard guard(device);
    ada_ctx* ctx = new (std::nothrow) ada_ctx();
    if (ctx == nullptr) return ADA_ERR_CUDA;
    ctx->device = device;
    ctx->maxB = maxB; ctx->maxT = maxT; ctx->maxd = maxd;
    ctx->dt = dt;
    ctx->es = dt == ADA_F32 ? 4 : 2;
    ctx->engine = ADA_ENGINE_AUTO;
    ctx->stage = nullptr; ctx->stage_bytes = 0; ctx->host_stream = nullptr;
    ctx->attn_ws = nullptr; ctx->attn_ws_bytes = 0;
    ctx->tc_attr_set = false;
    ctx->cooperative = true;
    ctx->dep_launch = true;
    ctx->tc2_attr_set = false;
    ctx->tc2_pairs = 0;
    ctx->compact_min_rows = 8192;
    cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device);

    const size_t n_tok = (size_t)maxB * (size_t)maxT;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    // role, g_tok, g_rep are contiguous so that one memset clears them
    const size_t o_role = take(n_tok * 4), o_gtok = take(n_tok * 4), o_grep = take(n_tok * 4);
    const size_t o_ctr = take(32);
    const int agg_stride = (int)((maxT + 1023) / 1024);
    const size_t o_done = take(32), o_agg = take((size_t)maxB * agg_stride * 8);
    const size_t o_near = take(n_tok * 8);
    const size_t o_inv = take(n_tok * 4), o_invr = take(n_tok * 4);
    const size_t o_reff = take((size_t)maxB * 4), o_stat = take(32), o_thr = take((size_t)maxB * 4);
    const size_t o_xrep = take(n_tok * (size_t)maxd * ctx->es + 1024);
    // bf16: the rows outside a large inherited set, copied out for the cross step (Algorithm 1 line 6)
    const size_t o_ntok = take(dt == ADA_BF16 ? n_tok * 4 : 0);
    const size_t o_xnon = take(dt == ADA_BF16 ? n_tok * (size_t)maxd * 2 + 1024 : 0);
    const size_t split_bytes = dt == ADA_F32 ? n_tok * (size_t)maxd * 12 + 1024 : 0;
    const size_t o_sxa = take(split_bytes), o_sxb = take(split_bytes), o_sra = take(split_bytes),
                 o_srb = take(split_bytes);
    if (cudaMalloc(&ctx->ws, off) != cudaSuccess) {
        cudaGetLastError();
        delete ctx;
        return ADA_ERR_CUDA;
    }
    ctx->role = reinterpret_cast<int32_t*>(ctx->ws + o_role);
    ctx->g_tok = reinterpret_cast<unsigned*>(ctx->ws + o_gtok);
    ctx->g_rep = reinterpret_cast<unsigned*>(ctx->ws + o_grep);
    ctx->inv_norm = reinterpret_cast<float*>(ctx->ws + o_inv);
    ctx->inv_rep = reinterpret_cast<float*>(ctx->ws + o_invr);
    ctx->r_eff = reinterpret_cast<int32_t*>(ctx->ws + o_reff);
    ctx->thr_seq = reinterpret_cast<float*>(ctx->ws + o_thr);
    ctx->status = reinterpret_cast<unsigned*>(ctx->ws + o_stat);
    ctx->tile_ctr = reinterpret_cast<unsigned*>(ctx->ws + o_ctr);
    ctx->done_ctr = reinterpret_cast<unsigned*>(ctx->ws + o_done);
    ctx->agg = reinterpret_cast<unsigned long long*>(ctx->ws + o_agg);
    ctx->agg_stride = agg_stride;
    ctx->near_key = reinterpret_cast<unsigned long long*>(ctx->ws + o_near);
    ctx->Xrep = ctx->ws + o_xrep;
    ctx->Xnon = dt == ADA_BF16 ? ctx->ws + o_xnon : nullptr;
    ctx->non_tok = dt == ADA_BF16 ? reinterpret_cast<int32_t*>(ctx->ws + o_ntok) : nullptr;
    ctx->splitXA = split_bytes ? ctx->ws + o_sxa : nullptr;
    ctx->splitXB = split_bytes ? ctx->ws + o_sxb : nullptr;
    ctx->splitRA = split_bytes ? ctx->ws + o_sra : nullptr;
    ctx->splitRB = split_bytes ? ctx->ws + o_srb : nullptr;
    if (cudaMemset(ctx->ws, 0, o_xrep) != cudaSuccess ||
        (dt == ADA_BF16 && cudaMemset(ctx->ws + o_ntok, 0, n_tok * 4) != cudaSuccess)) {
        cudaFree(ctx->ws);
        delete ctx;
        return ADA_ERR_CUDA;
    }
    *out = ctx;
    return ADA_OK;
}

ada_status ada_destroy(ada_ctx* ctx) {
    if (ctx == nullptr) return ADA_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaDeviceSynchronize();
    for (int i = 0; i < ctx->prof.created; ++i) {
        cudaEventDestroy(ctx->prof.ev0[i]);
        cudaEventDestroy(ctx->prof.ev1[i]);
    }
    if (ctx->stage) cudaFree(ctx->stage);
    if (ctx->attn_ws) cudaFree(ctx->attn_ws);
    if (ctx->host_stream) cudaStreamDestroy(ctx->host_stream);
    cudaFree(ctx->ws);
    delete ctx;
    return ADA_OK;
}

ada_status ada_set_engine(ada_ctx* ctx, ada_engine e) {
    if (ctx == nullptr) return ADA_ERR_INVALID_ARG;
    if (e != ADA_ENGINE_AUTO && e != ADA_ENGINE_FFMA && e != ADA_ENGINE_TCGEN05 &&
        e != ADA_ENGINE_TCGEN05_PAIR)
        return ADA_ERR_INVALID_ARG;
    if ((e == ADA_ENGINE_TCGEN05 || e == ADA_ENGINE_TCGEN05_PAIR) && !gram_tc_available())
        return ADA_ERR_UNSUPPORTED;
    ctx->engine = e;
    return ADA_OK;
}

ada_status ada_set_row_compaction(ada_ctx* ctx, int64_t min_rows) {
    if (ctx == nullptr || min_rows < 1) return ADA_ERR_INVALID_ARG;
    ctx->compact_min_rows = min_rows > 0x7fffffff ? 0x7fffffff : (int)min_rows;
    return ADA_OK;
}

ada_status ada_set_cooperative(ada_ctx* ctx, int on) {
    if (ctx == nullptr) return ADA_ERR_INVALID_ARG;
    ctx->cooperative = on != 0;
    return ADA_OK;
}

ada_status ada_set_dependent_launch(ada_ctx* ctx, int on) {
    if (ctx == nullptr) return ADA_ERR_INVALID_ARG;
    ctx->dep_launch = on != 0;
    return ADA_OK;
}

ada_status ada_normalize(ada_ctx* ctx, const void* X, int64_t B, int64_t T, int64_t d,
                         int64_t ldx, ada_dtype dt, void* Xhat, float* inv_norm,
                         const int32_t* rep_idx, const int32_t* rep_cnt, void* Xrep,
                         void* stream) {
    ada_status st = check_common(ctx, X, B, T, d, ldx, dt);
    if (st != ADA_OK) return st;
    const bool gather = rep_idx != nullptr || rep_cnt != nullptr || Xrep != nullptr;
    if (gather && (rep_idx == nullptr || rep_cnt == nullptr || Xrep == nullptr))
        return ADA_ERR_INVALID_ARG;
    if ((Xhat != nullptr && !aligned16(Xhat)) || (Xrep != nullptr && !aligned16(Xrep)))
        return ADA_ERR_UNSUPPORTED;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CU(launch_norm_gather(ctx, X, (int)B, (int)T, (int)d, ldx, T * ldx, dt, inv_norm, Xhat,
                          gather ? rep_idx : nullptr, rep_cnt, nullptr, nullptr, Xrep, ctx->inv_rep,
                          s));
    return ADA_OK;
}

// Definition 1 for B independent problems; row (b, t) of X starts at element b * xb + t * ldx
static ada_status select_full_impl(ada_ctx* ctx, const void* X, int64_t B, int64_t T, int64_t d,
                                   int64_t ldx, int64_t xb, ada_dtype dt, double tau,
                                   int32_t* rep_idx, int32_t* rep_cnt, float* gamma, void* stream) {
    if (rep_idx == nullptr || rep_cnt == nullptr || !tau_ok(tau)) return ADA_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const float thr = (float)(1.0 - tau * tau);

    // the gamma scratch is zero on entry (workspace invariant kept by the compaction kernels)
    // long-K tensor-core launches compute the row norms themselves, hidden behind the MMAs
    const bool split = use_split(ctx, dt);
    const bool tc = use_tc(ctx, dt), fuse = tc && d >= 2048 && B * T >= 4096 && xb == T * ldx;
    if (split)   // one pass: 1/||x|| and the bf16 terms of X
        CU(launch_split(ctx, X, (int)B, (int)T, (int)d, ldx, xb, false, s));
    else if (!fuse)
        CU(launch_norm_gather(ctx, X, (int)B, (int)T, (int)d, ldx, xb, dt, ctx->inv_norm, nullptr,
                              nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, s));
    NormJob nj;
    nj.X = X; nj.ldx = ldx; nj.n_rows = B * T; nj.d = (int)d; nj.inv_norm = ctx->inv_norm;
    nj.batch = 0; nj.rows_per_seq = 0;
    GramProblem p;
    memset(&p, 0, sizeof(p));
    p.A = X; p.Bm = X;
    p.lda = ldx; p.ldb = ldx;
    p.a_batch = xb; p.b_batch = xb;
    p.inv_a = ctx->inv_norm; p.inv_b = ctx->inv_norm;
    p.out = ctx->g_tok;
    p.n_dev = nullptr; p.n_host = (int)T;
    p.rows = (int)T; p.cap = (int)T; p.d = (int)d; p.B = (int)B;
    p.tri = 1;
    p.wait_norm_a = p.wait_norm_b = fuse ? 1 : 0;
    if (split) {
        p.A = ctx->splitXA; p.Bm = ctx->splitXB;
        p.lda = p.ldb = 6 * d;
        p.a_batch = p.b_batch = T * 6 * d;
        p.d = (int)(6 * d);
        CU(launch_tc(ctx, &p, nullptr, nullptr, s));
    } else if (tc) CU(launch_tc(ctx, &p, nullptr, fuse ? &nj : nullptr, s));
    else CU(run_gram(ctx, p, dt, s));
    CU(launch_compact_full(ctx, (int)B, (int)T, thr, rep_idx, rep_cnt, gamma, s));
    return ADA_OK;
}

ada_status ada_select_full(ada_ctx* ctx, const void* X, int64_t B, int64_t T, int64_t d,
                           int64_t ldx, ada_dtype dt, double tau, int32_t* rep_idx,
                           int32_t* rep_cnt, float* gamma, void* stream) {
    ada_status st = check_common(ctx, X, B, T, d, ldx, dt);
    if (st != ADA_OK) return st;
    return select_full_impl(ctx, X, B, T, d, ldx, T * ldx, dt, tau, rep_idx, rep_cnt, gamma, stream);
}

// heads interleaved inside each token's row: head j of token t starts at t * ldx + j * d_h
static ada_status check_heads(ada_ctx* ctx, const void* X, int64_t T, int64_t h, int64_t d_h,
                              int64_t ldx, ada_dtype dt) {
    ada_status st = check_common(ctx, X, h, T, d_h, ldx, dt);
    if (st != ADA_OK) return st;
    return ldx < h * d_h ? ADA_ERR_INVALID_ARG : ADA_OK;
}

ada_status ada_select_full_heads(ada_ctx* ctx, const void* X, int64_t T, int64_t h, int64_t d_h,
                                 int64_t ldx, ada_dtype dt, double tau, int32_t* rep_idx,
                                 int32_t* rep_cnt, float* gamma, void* stream) {
    ada_status st = check_heads(ctx, X, T, h, d_h, ldx, dt);
    if (st != ADA_OK) return st;
    return select_full_impl(ctx, X, h, T, d_h, ldx, d_h, dt, tau, rep_idx, rep_cnt, gamma, stream);
}

// Algorithm 1 for B independent problems; row (b, t) of X starts at element b * xb + t * ldx
static ada_status cascade_impl(ada_ctx* ctx, const void* X, int64_t B, int64_t T, int64_t d,
                               int64_t ldx, int64_t xb, ada_dtype dt, double tau,
                               const int32_t* rep_in, const int32_t* rep_in_cnt, int32_t* rep_out,
                               int32_t* rep_out_cnt, int32_t* add_idx, int32_t* add_cnt,
                               int32_t* rem_idx, int32_t* rem_cnt, float* gamma_rep,
                               float* gamma_cross, uint32_t flags, void* stream,
                               const TauUpdate* tu = nullptr) {
    if (rep_in == nullptr || rep_in_cnt == nullptr || rep_out == nullptr ||
        rep_out_cnt == nullptr || add_idx == nullptr || add_cnt == nullptr ||
        rem_idx == nullptr || rem_cnt == nullptr || !tau_ok(tau))
        return ADA_ERR_INVALID_ARG;
    if (rep_out == rep_in || (flags & ~ADA_CROSS_CAUSAL) != 0) return ADA_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const float thr = (float)(1.0 - tau * tau);
    TauUpdate tau_upd;
    memset(&tau_upd, 0, sizeof(tau_upd));
    if (tu != nullptr) tau_upd = *tu;
    const bool adaptive = tau_upd.tau_state != nullptr;
    if (adaptive) CU(launch_tau_thr(ctx, (int)B, tau_upd.tau_state, s));   // thresholds of this step

    // role map, gamma scratch and dependency counters are zero on entry (workspace invariant
    // kept by the compaction kernels).
    const bool split = use_split(ctx, dt);
    const bool fuse = use_tc(ctx, dt) || split;
    // bf16 on the pair kernel: ONE Gram launch does lines 1-8.  Its helper warps validate the
    // inherited list, scatter the role map and gather the rows (lines 1-2); the r x r tiles
    // (lines 3-5) and the cross tiles (lines 6-8) follow; the norms of X come out of the cross
    // tiles while they sit in shared memory, and the row's own factor 1/||x_t|| is left to the
    // compaction.
    const bool inl = fuse && !split && use_pair(ctx, B, T, d);
    // otherwise lines 1-2 are a launch of their own: inverse norms of all rows, inherited list
    // validated, scattered into the role map and its rows gathered into Xrep; for long K the
    // one-CTA tensor-core launch computes line 1's row norms itself
    const bool fuse_norm = !inl && !split && fuse && d >= 2048 && B * T >= 4096 && xb == T * ldx;
    if (!inl)
        CU(launch_norm_gather(ctx, X, (int)B, (int)T, (int)d, ldx, xb, dt,
                              (fuse_norm || split) ? nullptr : ctx->inv_norm,
                              nullptr, rep_in, rep_in_cnt, ctx->role, ctx->r_eff, ctx->Xrep,
                              ctx->inv_rep, s));
    NormJob nj;
    nj.X = X; nj.ldx = ldx; nj.n_rows = B * T; nj.d = (int)d; nj.inv_norm = ctx->inv_norm;
    nj.batch = 0; nj.rows_per_seq = 0;
    GatherJob gj;
    memset(&gj, 0, sizeof(gj));
    gj.X = X; gj.ldx = ldx; gj.xb = xb;
    gj.rep_in = rep_in; gj.rep_in_cnt = rep_in_cnt;
    gj.role = ctx->role; gj.r_eff = ctx->r_eff; gj.Xrep = ctx->Xrep; gj.inv_rep = ctx->inv_rep;
    gj.T = (int)T; gj.d = (int)d; gj.B = (int)B;
    gj.Xnon = ctx->Xnon; gj.non_tok = ctx->non_tok; gj.inv_norm = ctx->inv_norm;
    gj.compact_min_rows = ctx->compact_min_rows;
    if (split)   // 1/||x|| of all rows; bf16 terms of X and of the gathered rows
        CU(launch_split(ctx, X, (int)B, (int)T, (int)d, ldx, xb, true, s));
    // lines 3-4: r x r Gram among inherited reps, max over earlier ones
    GramProblem p;
    memset(&p, 0, sizeof(p));
    p.A = ctx->Xrep; p.Bm = ctx->Xrep;
    p.lda = d; p.ldb = d;
    p.a_batch = T * d; p.b_batch = T * d;
    p.inv_a = ctx->inv_rep; p.inv_b = ctx->inv_rep;
    p.out = ctx->g_rep;
    p.n_dev = inl ? rep_in_cnt : ctx->r_eff; p.n_host = 0;
    p.n_clamp = inl ? 1 : 0;
    p.rows = (int)T; p.cap = (int)T; p.d = (int)d; p.B = (int)B;
    p.tri = 1;
    if (!fuse) CU(run_gram(ctx, p, dt, s));
    // lines 6-8: cross-Gram of all rows against the valid inherited reps
    GramProblem q;
    memset(&q, 0, sizeof(q));
    q.A = X; q.Bm = ctx->Xrep;
    q.lda = ldx; q.ldb = d;
    q.a_batch = xb; q.b_batch = T * d;
    q.inv_a = ctx->inv_norm; q.inv_b = ctx->inv_rep;
    q.out = ctx->g_tok;
    q.n_dev = p.n_dev; q.n_host = 0;
    q.n_clamp = p.n_clamp;
    q.rows = (int)T; q.cap = (int)T; q.d = (int)d; q.B = (int)B;
    q.tri = 0;
    q.col_gate = ctx->g_rep;
    q.thr_bits = 0;
    memcpy(&q.thr_bits, &thr, 4);
    q.thr_seq = adaptive ? reinterpret_cast<const unsigned*>(ctx->thr_seq) : nullptr;
    q.col_token = rep_in;
    q.row_role = ctx->role;
    q.causal = (flags & ADA_CROSS_CAUSAL) ? 1 : 0;
    q.wait_norm_a = fuse_norm ? 1 : 0;
    if (inl) {
        q.defer_row = 1;
        q.inv_out = ctx->inv_norm;
        q.hb_rows = gram_tc2_hb_rows(ctx, (int)B, (int)T);
        if (q.hb_rows == 0) return ADA_ERR_CUDA;
    }
    if (split) {
        p.A = ctx->splitRA; p.Bm = ctx->splitRB;
        q.A = ctx->splitXA; q.Bm = ctx->splitRB;
        p.lda = p.ldb = q.lda = q.ldb = 6 * d;
        p.a_batch = p.b_batch = q.a_batch = q.b_batch = T * 6 * d;
        p.d = q.d = (int)(6 * d);
    }
    if (inl) CU(launch_gram_tc2(ctx, &p, &q, nullptr, &gj, s));
    else if (fuse) CU(launch_tc(ctx, &p, &q, fuse_norm ? &nj : nullptr, s));
    else CU(run_gram(ctx, q, dt, s));
    // lines 5, 9, 10-11
    CU(launch_compact_cascade(ctx, (int)B, (int)T, thr, rep_out, rep_out_cnt, add_idx, add_cnt,
                              rem_idx, rem_cnt, gamma_rep, gamma_cross, tau_upd, inl, s));
    return ADA_OK;
}

ada_status ada_cascade_step_adaptive(ada_ctx* ctx, const void* X, int64_t B, int64_t T, int64_t d,
                                     int64_t ldx, ada_dtype dt, double* tau_state,
                                     const ada_tau_policy* policy, const int32_t* rep_in,
                                     const int32_t* rep_in_cnt, int32_t* rep_out,
                                     int32_t* rep_out_cnt, int32_t* add_idx, int32_t* add_cnt,
                                     int32_t* rem_idx, int32_t* rem_cnt, float* gamma_rep,
                                     float* gamma_cross, float* turnover, uint32_t flags,
                                     void* stream) {
    ada_status st = check_common(ctx, X, B, T, d, ldx, dt);
    if (st != ADA_OK) return st;
    if (tau_state == nullptr) return ADA_ERR_INVALID_ARG;
    TauUpdate tu;
    memset(&tu, 0, sizeof(tu));
    tu.tau_state = tau_state;
    tu.turnover = turnover;
    if (policy != nullptr) {
        // also rejects NaN in any field
        if (!(policy->gain >= 0.0) || !(policy->target_turnover >= 0.0) || !(policy->tau_min > 0.0) ||
            !(policy->tau_max < 1.0) || !(policy->tau_min <= policy->tau_max))
            return ADA_ERR_INVALID_ARG;
        tu.update = 1;
        tu.target = policy->target_turnover; tu.gain = policy->gain;
        tu.tau_min = policy->tau_min; tu.tau_max = policy->tau_max;
    }
    // the host-side tau of the fixed-threshold call is not used; 0.5 passes its range check
    return cascade_impl(ctx, X, B, T, d, ldx, T * ldx, dt, 0.5, rep_in, rep_in_cnt, rep_out,
                        rep_out_cnt, add_idx, add_cnt, rem_idx, rem_cnt, gamma_rep, gamma_cross,
                        flags, stream, &tu);
}

ada_status ada_cascade_step(ada_ctx* ctx, const void* X, int64_t B, int64_t T, int64_t d,
                            int64_t ldx, ada_dtype dt, double tau, const int32_t* rep_in,
                            const int32_t* rep_in_cnt, int32_t* rep_out, int32_t* rep_out_cnt,
                            int32_t* add_idx, int32_t* add_cnt, int32_t* rem_idx,
                            int32_t* rem_cnt, float* gamma_rep, float* gamma_cross,
                            uint32_t flags, void* stream) {
    ada_status st = check_common(ctx, X, B, T, d, ldx, dt);
    if (st != ADA_OK) return st;
    return cascade_impl(ctx, X, B, T, d, ldx, T * ldx, dt, tau, rep_in, rep_in_cnt, rep_out,
                        rep_out_cnt, add_idx, add_cnt, rem_idx, rem_cnt, gamma_rep, gamma_cross,
                        flags, stream);
}

ada_status ada_cascade_step_heads(ada_ctx* ctx, const void* X, int64_t T, int64_t h, int64_t d_h,
                                  int64_t ldx, ada_dtype dt, double tau, const int32_t* rep_in,
                                  const int32_t* rep_in_cnt, int32_t* rep_out,
                                  int32_t* rep_out_cnt, int32_t* add_idx, int32_t* add_cnt,
                                  int32_t* rem_idx, int32_t* rem_cnt, float* gamma_rep,
                                  float* gamma_cross, uint32_t flags, void* stream) {
    ada_status st = check_heads(ctx, X, T, h, d_h, ldx, dt);
    if (st != ADA_OK) return st;
    return cascade_impl(ctx, X, h, T, d_h, ldx, d_h, dt, tau, rep_in, rep_in_cnt, rep_out,
                        rep_out_cnt, add_idx, add_cnt, rem_idx, rem_cnt, gamma_rep, gamma_cross,
                        flags, stream);
}

ada_status ada_nearest_rep(ada_ctx* ctx, const void* X, int64_t B, int64_t T, int64_t d,
                           int64_t ldx, ada_dtype dt, const int32_t* rep_idx,
                           const int32_t* rep_cnt, int32_t* nearest_idx, float* nearest_gamma,
                           void* stream) {
    ada_status st = check_common(ctx, X, B, T, d, ldx, dt);
    if (st != ADA_OK) return st;
    if (rep_idx == nullptr || rep_cnt == nullptr || nearest_idx == nullptr) return ADA_ERR_INVALID_ARG;
    const bool split = dt == ADA_F32;
    if (!gram_tc_available() || (split && ctx->splitXA == nullptr)) return ADA_ERR_UNSUPPORTED;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // role map and keys are zero on entry (workspace invariant); the finish kernel clears them
    CU(launch_norm_gather(ctx, X, (int)B, (int)T, (int)d, ldx, T * ldx, dt, split ? nullptr : ctx->inv_norm,
                          nullptr, rep_idx, rep_cnt, ctx->role, ctx->r_eff, ctx->Xrep, ctx->inv_rep, s));
    if (split) CU(launch_split(ctx, X, (int)B, (int)T, (int)d, ldx, T * ldx, true, s));
    GramProblem q;
    memset(&q, 0, sizeof(q));
    q.A = X; q.Bm = ctx->Xrep;
    q.lda = ldx; q.ldb = d;
    q.a_batch = T * ldx; q.b_batch = T * d;
    if (split) {
        q.A = ctx->splitXA; q.Bm = ctx->splitRB;
        q.lda = q.ldb = 6 * d;
        q.a_batch = q.b_batch = T * 6 * d;
    }
    q.inv_a = ctx->inv_norm; q.inv_b = ctx->inv_rep;
    q.out = ctx->g_tok;
    q.out_arg = ctx->near_key;
    q.n_dev = ctx->r_eff; q.n_host = 0;
    q.rows = (int)T; q.cap = (int)T; q.d = (int)(split ? 6 * d : d); q.B = (int)B;
    q.tri = 0;
    q.col_gate = ctx->g_rep;          // all zero: every column passes the gate
    q.thr_bits = 0xFFFFFFFFu;
    q.col_token = rep_idx;
    q.row_role = ctx->role;           // representatives are resolved by the finish kernel
    q.causal = 0;
    CU(launch_gram_tc(ctx, nullptr, &q, nullptr, s));
    CU(launch_nearest_finish(ctx, (int)B, (int)T, rep_idx, nearest_idx, nearest_gamma, s));
    return ADA_OK;
}

ada_status ada_attention_reps(ada_ctx* ctx, const void* Q, const void* K, const void* V, int64_t T,
                              int64_t h, int64_t d_h, int64_t ld, ada_dtype dt, const int32_t* rep_idx,
                              const int32_t* rep_cnt, const int32_t* nearest_idx, float* out,
                              int64_t ldo, uint32_t flags, void* stream) {
    if (ctx == nullptr || Q == nullptr || K == nullptr || V == nullptr || rep_idx == nullptr ||
        rep_cnt == nullptr || out == nullptr)
        return ADA_ERR_INVALID_ARG;
    if (T < 1 || h < 1 || d_h < 1 || ld < h * d_h || ldo < h * d_h || (flags & ~ADA_ATTN_CAUSAL) != 0)
        return ADA_ERR_INVALID_ARG;
    if (dt != ADA_F32 && dt != ADA_BF16) return ADA_ERR_INVALID_ARG;
    // bf16 operands on the tensor cores; head widths the two contractions' tiles cover
    if (dt != ADA_BF16 || ctx->dt != ADA_BF16 || d_h % 16 != 0 || d_h > 128 || !gram_tc_available())
        return ADA_ERR_UNSUPPORTED;
    if (T > ctx->maxT || h * d_h > ctx->maxd) return ADA_ERR_WORKSPACE;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(out) || (ld * 2) % 16 != 0 ||
        (ldo * 4) % 16 != 0)
        return ADA_ERR_UNSUPPORTED;
    DeviceGuard guard(ctx->device);
    CU(launch_attention_reps(ctx, Q, K, V, (int)T, (int)h, (int)d_h, ld, rep_idx, rep_cnt, nearest_idx, out,
                             ldo, (flags & ADA_ATTN_CAUSAL) ? 1 : 0, static_cast<cudaStream_t>(stream)));
    return ADA_OK;
}

ada_status ada_device_status(ada_ctx* ctx, void* stream, int64_t* n_zero_norm_rows) {
    if (ctx == nullptr) return ADA_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned h[8];
    CU(cudaMemcpyAsync(h, ctx->status, sizeof(h), cudaMemcpyDeviceToHost, s));
    CU(cudaMemsetAsync(ctx->status, 0, sizeof(h), s));
    CU(cudaStreamSynchronize(s));
    if (n_zero_norm_rows != nullptr) *n_zero_norm_rows = (int64_t)h[1];
    if (h[0] != 0) {
        // a faulted call may have left scratch behind: restore the all-zero workspace invariant
        CU(cudaMemsetAsync(ctx->role, 0, (size_t)((char*)ctx->inv_norm - (char*)ctx->role), s));
        CU(cudaStreamSynchronize(s));
    }
    if (h[0] & ST_TIMEOUT) return ADA_ERR_TIMEOUT;
    if (h[0] & (ST_BAD_INDEX | ST_BAD_COUNT)) return ADA_ERR_BAD_INDEX_SET;
    if (h[0] & ST_NONFINITE) return ADA_ERR_NONFINITE;
    if (h[0] & ST_BAD_TAU) return ADA_ERR_BAD_TAU;
    return ADA_OK;
}

// ---------------------------------------------------------------------------
// host-buffer entry points
// ---------------------------------------------------------------------------
static ada_status ensure_stage(ada_ctx* ctx) {
    if (ctx->stage != nullptr) return ADA_OK;
    const size_t n_tok = (size_t)ctx->maxB * ctx->maxT;
    // X | 5 index lists | 2 gamma arrays | 4 count arrays
    const size_t bytes = align_up(n_tok * ctx->maxd * ctx->es, 256) + 7 * align_up(n_tok * 4, 256) +
                         4 * align_up((size_t)ctx->maxB * 4, 256);
    if (cudaMalloc(&ctx->stage, bytes) != cudaSuccess) {
        cudaGetLastError();
        return ADA_ERR_CUDA;
    }
    ctx->stage_bytes = bytes;
    return ADA_OK;
}

struct Stage {
    char* X;
    int32_t *l0, *l1, *l2, *l3;
    float *g0, *g1;
    int32_t *c0, *c1, *c2, *c3;
};

static Stage carve(ada_ctx* ctx) {
    const size_t n_tok = (size_t)ctx->maxB * ctx->maxT;
    const size_t lx = align_up(n_tok * ctx->maxd * ctx->es, 256), ll = align_up(n_tok * 4, 256),
                 lc = align_up((size_t)ctx->maxB * 4, 256);
    Stage st;
    char* p = ctx->stage;
    st.X = p; p += lx;
    st.l0 = (int32_t*)p; p += ll;
    st.l1 = (int32_t*)p; p += ll;
    st.l2 = (int32_t*)p; p += ll;
    st.l3 = (int32_t*)p; p += ll;
    st.g0 = (float*)p; p += ll;
    st.g1 = (float*)p; p += ll;
    p += ll;
    st.c0 = (int32_t*)p; p += lc;
    st.c1 = (int32_t*)p; p += lc;
    st.c2 = (int32_t*)p; p += lc;
    st.c3 = (int32_t*)p;
    return st;
}

ada_status ada_select_full_host(ada_ctx* ctx, const void* X, int64_t B, int64_t T, int64_t d,
                                ada_dtype dt, double tau, int32_t* rep_idx, int32_t* rep_cnt,
                                float* gamma, void* stream) {
    if (ctx == nullptr || X == nullptr || rep_idx == nullptr || rep_cnt == nullptr)
        return ADA_ERR_INVALID_ARG;
    if (B < 1 || T < 1 || d < 1) return ADA_ERR_INVALID_ARG;
    if (dt != ADA_F32 && dt != ADA_BF16) return ADA_ERR_INVALID_ARG;
    // before anything is copied: the copies below are sized by the context's element type
    if (dt != ctx->dt || (d * ctx->es) % 16 != 0) return ADA_ERR_UNSUPPORTED;
    if (B > ctx->maxB || T > ctx->maxT || d > ctx->maxd) return ADA_ERR_WORKSPACE;
    DeviceGuard guard(ctx->device);
    ada_status st = ensure_stage(ctx);
    if (st != ADA_OK) return st;
    Stage sg = carve(ctx);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t n_tok = (size_t)B * T;
    CU(cudaMemcpyAsync(sg.X, X, n_tok * d * ctx->es, cudaMemcpyHostToDevice, s));
    st = ada_select_full(ctx, sg.X, B, T, d, d, dt, tau, sg.l0, sg.c0, gamma ? sg.g0 : nullptr, s);
    if (st != ADA_OK) return st;
    CU(cudaMemcpyAsync(rep_idx, sg.l0, n_tok * 4, cudaMemcpyDeviceToHost, s));
    CU(cudaMemcpyAsync(rep_cnt, sg.c0, (size_t)B * 4, cudaMemcpyDeviceToHost, s));
    if (gamma) CU(cudaMemcpyAsync(gamma, sg.g0, n_tok * 4, cudaMemcpyDeviceToHost, s));
    CU(cudaStreamSynchronize(s));
    return ADA_OK;
}

ada_status ada_cascade_step_host(ada_ctx* ctx, const void* X, int64_t B, int64_t T, int64_t d,
                                 ada_dtype dt, double tau, const int32_t* rep_in,
                                 const int32_t* rep_in_cnt, int32_t* rep_out,
                                 int32_t* rep_out_cnt, int32_t* add_idx, int32_t* add_cnt,
                                 int32_t* rem_idx, int32_t* rem_cnt, float* gamma_rep,
                                 float* gamma_cross, uint32_t flags, void* stream) {
    if (ctx == nullptr || X == nullptr || rep_in == nullptr || rep_in_cnt == nullptr ||
        rep_out == nullptr || rep_out_cnt == nullptr || add_idx == nullptr ||
        add_cnt == nullptr || rem_idx == nullptr || rem_cnt == nullptr)
        return ADA_ERR_INVALID_ARG;
    if (B < 1 || T < 1 || d < 1) return ADA_ERR_INVALID_ARG;
    if (dt != ADA_F32 && dt != ADA_BF16) return ADA_ERR_INVALID_ARG;
    // before anything is copied: the copies below are sized by the context's element type
    if (dt != ctx->dt || (d * ctx->es) % 16 != 0) return ADA_ERR_UNSUPPORTED;
    if (B > ctx->maxB || T > ctx->maxT || d > ctx->maxd) return ADA_ERR_WORKSPACE;
    DeviceGuard guard(ctx->device);
    ada_status st = ensure_stage(ctx);
    if (st != ADA_OK) return st;
    Stage sg = carve(ctx);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t n_tok = (size_t)B * T;
    CU(cudaMemcpyAsync(sg.X, X, n_tok * d * ctx->es, cudaMemcpyHostToDevice, s));
    CU(cudaMemcpyAsync(sg.l0, rep_in, n_tok * 4, cudaMemcpyHostToDevice, s));
    CU(cudaMemcpyAsync(sg.c0, rep_in_cnt, (size_t)B * 4, cudaMemcpyHostToDevice, s));
    st = ada_cascade_step(ctx, sg.X, B, T, d, d, dt, tau, sg.l0, sg.c0, sg.l1, sg.c1, sg.l2, sg.c2,
                          sg.l3, sg.c3, gamma_rep ? sg.g0 : nullptr, gamma_cross ? sg.g1 : nullptr,
                          flags, s);
    if (st != ADA_OK) return st;
    CU(cudaMemcpyAsync(rep_out, sg.l1, n_tok * 4, cudaMemcpyDeviceToHost, s));
    CU(cudaMemcpyAsync(add_idx, sg.l2, n_tok * 4, cudaMemcpyDeviceToHost, s));
    CU(cudaMemcpyAsync(rem_idx, sg.l3, n_tok * 4, cudaMemcpyDeviceToHost, s));
    CU(cudaMemcpyAsync(rep_out_cnt, sg.c1, (size_t)B * 4, cudaMemcpyDeviceToHost, s));
    CU(cudaMemcpyAsync(add_cnt, sg.c2, (size_t)B * 4, cudaMemcpyDeviceToHost, s));
    CU(cudaMemcpyAsync(rem_cnt, sg.c3, (size_t)B * 4, cudaMemcpyDeviceToHost, s));
    if (gamma_rep) CU(cudaMemcpyAsync(gamma_rep, sg.g0, n_tok * 4, cudaMemcpyDeviceToHost, s));
    if (gamma_cross) CU(cudaMemcpyAsync(gamma_cross, sg.g1, n_tok * 4, cudaMemcpyDeviceToHost, s));
    CU(cudaStreamSynchronize(s));
    return ADA_OK;
}

ada_status ada_selftest_wait_timeout(ada_ctx* ctx, int limit_ms, void* stream) {
    if (ctx == nullptr || limit_ms < 1 || limit_ms > 2000) return ADA_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    CU(launch_selftest_wait(ctx, limit_ms, static_cast<cudaStream_t>(stream)));
    return ADA_OK;
}

ada_status ada_profile_enable(ada_ctx* ctx, int on) {
    if (ctx == nullptr) return ADA_ERR_INVALID_ARG;
    ctx->prof.on = on != 0;
    ctx->prof.n = 0;
    return ADA_OK;
}

int ada_profile_read(ada_ctx* ctx, const char** names, int64_t* launches, double* total_ms,
                     int cap) {
    if (ctx == nullptr) return 0;
    DeviceGuard guard(ctx->device);
    Profiler& pr = ctx->prof;
    int64_t cnt[K_COUNT] = {0};
    double ms[K_COUNT] = {0};
    for (int i = 0; i < pr.n; ++i) {
        cudaEventSynchronize(pr.ev1[i]);
        float t = 0.f;
        if (cudaEventElapsedTime(&t, pr.ev0[i], pr.ev1[i]) == cudaSuccess) {
            cnt[pr.kid[i]] += 1;
            ms[pr.kid[i]] += t;
        }
    }
    pr.n = 0;
    for (int k = 0; k < K_COUNT && k < cap; ++k) {
        if (names) names[k] = kKernelNames[k];
        if (launches) launches[k] = cnt[k];
        if (total_ms) total_ms[k] = ms[k];
    }
    return K_COUNT;
}

}  // extern "C"
