// HBM-bound helper kernels of the selection path: fused row-norm + representative
// gather (with validation of the inherited list), and the prefix-sum compaction that
// turns gamma into sorted index lists.
#include "common.cuh"

namespace ada {

// ---------------------------------------------------------------------------
// Row normalisation fused with the representative gather (Section 2.1;
// Algorithm 1 lines 1-2).  One warp per row, 128-bit loads.  inv_norm[t] =
// 1/||x_t|| in fp32 (0 for a zero row).  The rows of the inherited list are
// copied, raw, to Xrep[position] together with their inverse norm.
// ---------------------------------------------------------------------------
template <typename T>
struct Vec16;
template <>
struct Vec16<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ float sumsq(const uint4& v) {
        const float a = __uint_as_float(v.x), b = __uint_as_float(v.y), c = __uint_as_float(v.z),
                    e = __uint_as_float(v.w);
        return a * a + b * b + c * c + e * e;
    }
    static __device__ __forceinline__ uint4 scale(const uint4& v, float f) {
        uint4 o;
        o.x = __float_as_uint(__uint_as_float(v.x) * f);
        o.y = __float_as_uint(__uint_as_float(v.y) * f);
        o.z = __float_as_uint(__uint_as_float(v.z) * f);
        o.w = __float_as_uint(__uint_as_float(v.w) * f);
        return o;
    }
};
template <>
struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ float2 up(unsigned w) {
        // a bf16 is the upper half of an fp32
        return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
    }
    static __device__ __forceinline__ float sumsq(const uint4& v) {
        const float2 a = up(v.x), b = up(v.y), c = up(v.z), e = up(v.w);
        return (a.x * a.x + a.y * a.y) + (b.x * b.x + b.y * b.y) + (c.x * c.x + c.y * c.y) +
               (e.x * e.x + e.y * e.y);
    }
    static __device__ __forceinline__ unsigned scale2(unsigned w, float f) {
        const float2 a = up(w);
        const __nv_bfloat162 r = __floats2bfloat162_rn(a.x * f, a.y * f);
        return *reinterpret_cast<const unsigned*>(&r);
    }
    static __device__ __forceinline__ uint4 scale(const uint4& v, float f) {
        return make_uint4(scale2(v.x, f), scale2(v.y, f), scale2(v.z, f), scale2(v.w, f));
    }
};

// Sum of squares of one row, one warp, four independent 128-bit loads in flight per lane.
template <typename T>
__device__ __forceinline__ float warp_row_sumsq(const uint4* __restrict__ src, int nvec, int lane) {
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
    int v = lane;
    for (; v + 96 < nvec; v += 128) {
        const uint4 a = __ldg(src + v), b = __ldg(src + v + 32), c = __ldg(src + v + 64),
                    e = __ldg(src + v + 96);
        s0 += Vec16<T>::sumsq(a);
        s1 += Vec16<T>::sumsq(b);
        s2 += Vec16<T>::sumsq(c);
        s3 += Vec16<T>::sumsq(e);
    }
    for (; v < nvec; v += 32) s0 += Vec16<T>::sumsq(__ldg(src + v));
    float ss = (s0 + s1) + (s2 + s3);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    return ss;
}

// Warps [0, n_rows) normalise: inv_norm[row] (and Xhat).  Warps [n_rows, 2 n_rows) serve the
// inherited list (Algorithm 1 "Require" and line 2): warp (b, i) with i < count validates
// entry i (in range, strictly above entry i-1), records role[token] = i+1, copies the raw
// row to Xrep[b, i] and stores its inverse norm.  Both halves read X directly, so there is
// no dependency between them and no separate scatter pass.
template <typename T>
__global__ void __launch_bounds__(256)
k_norm_gather(const T* __restrict__ X, int64_t n_rows, int Tseq, int d, int64_t ldx, int64_t xb,
              float* __restrict__ inv_norm, T* __restrict__ Xhat,
              const int32_t* __restrict__ rep_in, const int32_t* __restrict__ rep_in_cnt,
              int32_t* __restrict__ role, int32_t* __restrict__ r_eff, T* __restrict__ Xrep,
              float* __restrict__ inv_rep, unsigned* __restrict__ status) {
    grid_dep_wait();
    const int lane = threadIdx.x & 31;
    int64_t w = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (inv_norm == nullptr && Xhat == nullptr) w += n_rows;   // gather-only launch: list warps only
    constexpr int N = Vec16<T>::N;
    const int nvec = d / N;  // d*es is a multiple of 16 bytes
    if (w < n_rows) {
        const int64_t row = w;
        // row (b, t) of X starts at b * xb + t * ldx (xb = Tseq * ldx for stacked sequences,
        // the head width for heads interleaved inside one row)
        const uint4* src = reinterpret_cast<const uint4*>(X + (row / Tseq) * xb + (row % Tseq) * ldx);
        const float ss = warp_row_sumsq<T>(src, nvec, lane);
        float inv = 0.f;
        if (!(ss <= 3.0e38f)) {  // NaN or overflow to Inf
            if (lane == 0) atomicOr(status, ST_NONFINITE);
        } else if (ss > 0.f) {
            inv = 1.0f / sqrtf(ss);
        } else if (lane == 0) {
            atomicAdd(status + 1, 1u);
        }
        if (inv_norm != nullptr && lane == 0) inv_norm[row] = inv;
        if (Xhat != nullptr) {
            uint4* dst = reinterpret_cast<uint4*>(Xhat + row * (int64_t)d);
            for (int v = lane; v < nvec; v += 32) dst[v] = Vec16<T>::scale(__ldg(src + v), inv);
        }
        return;
    }
    w -= n_rows;
    if (rep_in == nullptr || w >= n_rows) return;
    const int b = (int)(w / Tseq), i = (int)(w % Tseq);
    int cnt = rep_in_cnt[b];
    if (cnt < 0 || cnt > Tseq) {
        if (i == 0 && lane == 0) atomicOr(status, ST_BAD_COUNT);
        cnt = cnt < 0 ? 0 : Tseq;
    }
    if (i == 0 && lane == 0 && r_eff != nullptr) r_eff[b] = cnt;
    if (i >= cnt) return;
    const int32_t* list = rep_in + (int64_t)b * Tseq;
    const int32_t idx = list[i];
    bool ok = idx >= 0 && idx < Tseq;
    if (ok && i > 0) ok = list[i - 1] < idx;
    if (!ok) {
        if (lane == 0) atomicOr(status, ST_BAD_INDEX);
        return;
    }
    const int64_t prow = (int64_t)b * Tseq + i;
    const uint4* src = reinterpret_cast<const uint4*>(X + (int64_t)b * xb + (int64_t)idx * ldx);
    uint4* dst = reinterpret_cast<uint4*>(Xrep + prow * (int64_t)d);
    float ss = 0.f;
    int v = lane;
    for (; v + 224 < nvec; v += 256) {          // eight loads in flight per lane
        uint4 x[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) x[q] = __ldg(src + v + 32 * q);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            ss += Vec16<T>::sumsq(x[q]);
            dst[v + 32 * q] = x[q];
        }
    }
    for (; v < nvec; v += 32) {
        const uint4 x = __ldg(src + v);
        ss += Vec16<T>::sumsq(x);
        dst[v] = x;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if (lane == 0) {
        inv_rep[prow] = (ss <= 3.0e38f && ss > 0.f) ? 1.0f / sqrtf(ss) : 0.f;
        if (role != nullptr) role[(int64_t)b * Tseq + idx] = i + 1;
    }
}

constexpr int NORM_U = 4;   // rows per lane group of the short-row kernel

// The same work for short rows (at most 16 vectors, e.g. one attention head), where a warp
// per row would leave most lanes idle behind a single load.  Warps [0, n_norm_warps) take
// rpw rows each, the warps after them rpw consecutive positions of one sequence's list.
template <typename T>
__global__ void __launch_bounds__(256)
k_norm_gather_short(const T* __restrict__ X, int64_t n_rows, int Tseq, int d, int64_t ldx, int64_t xb,
                    int rpw, int64_t n_norm_warps, float* __restrict__ inv_norm, T* __restrict__ Xhat,
                    const int32_t* __restrict__ rep_in, const int32_t* __restrict__ rep_in_cnt,
                    int32_t* __restrict__ role, int32_t* __restrict__ r_eff, T* __restrict__ Xrep,
                    float* __restrict__ inv_rep, unsigned* __restrict__ status) {
    grid_dep_wait();
    const int lane = threadIdx.x & 31;
    int64_t w = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (inv_norm == nullptr && Xhat == nullptr) w += n_norm_warps;   // gather-only launch: list warps only
    constexpr int N = Vec16<T>::N;
    const int nvec = d / N;  // d*es is a multiple of 16 bytes
    if (w < n_norm_warps) {
        // Short rows (at most 16 vectors, e.g. one attention head): a group of G lanes owns a
        // row, the warp's 32/G groups take NORM_U rows each, and every lane has NORM_U loads in
        // flight; a warp per row would leave most lanes idle behind one load.  Rows are taken
        // in memory order: head-fastest when the heads of a token lie side by side.
        const int R = rpw / NORM_U, G = 32 / R, sub = lane / G, gl = lane % G;
        // (row counts fit 31 bits; 32-bit division is several times cheaper than 64-bit)
        const unsigned nseq = (unsigned)n_rows / (unsigned)Tseq;
        uint4 x[NORM_U];
        int64_t orow[NORM_U];
#pragma unroll
        for (int u = 0; u < NORM_U; ++u) {
            const int64_t r = w * rpw + u * R + sub;
            x[u] = make_uint4(0u, 0u, 0u, 0u);
            orow[u] = -1;
            if (r < n_rows) {
                const unsigned r32 = (unsigned)r;
                const int64_t b = xb < ldx ? r32 % nseq : r32 / (unsigned)Tseq,
                              t = xb < ldx ? r32 / nseq : r32 % (unsigned)Tseq;
                orow[u] = b * Tseq + t;
                if (gl < nvec) x[u] = __ldg(reinterpret_cast<const uint4*>(X + b * xb + t * ldx) + gl);
            }
        }
#pragma unroll
        for (int u = 0; u < NORM_U; ++u) {
            float ss = Vec16<T>::sumsq(x[u]);
            for (int o = G >> 1; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
            if (orow[u] < 0) continue;
            float inv = 0.f;
            if (!(ss <= 3.0e38f)) {
                if (gl == 0) atomicOr(status, ST_NONFINITE);
            } else if (ss > 0.f) {
                inv = 1.0f / sqrtf(ss);
            } else if (gl == 0) {
                atomicAdd(status + 1, 1u);
            }
            if (inv_norm != nullptr && gl == 0) inv_norm[orow[u]] = inv;
            if (Xhat != nullptr && gl < nvec)
                reinterpret_cast<uint4*>(Xhat + orow[u] * (int64_t)d)[gl] = Vec16<T>::scale(x[u], inv);
        }
        return;
    }
    w -= n_norm_warps;
    if (rep_in == nullptr) return;
    {
        // short rows: a lane group per list entry, NORM_U entries per group, as above; a warp
        // covers rpw consecutive positions of one sequence's list
        const int R = rpw / NORM_U, G = 32 / R, sub = lane / G, gl = lane % G;
        const unsigned wps = (unsigned)(Tseq + rpw - 1) / (unsigned)rpw;   // warps per sequence
        if (w >= (int64_t)wps * ((unsigned)n_rows / (unsigned)Tseq)) return;
        const int b = (int)((unsigned)w / wps);
        const int i0 = (int)((unsigned)w % wps) * rpw;
        int cnt = rep_in_cnt[b];
        if (cnt < 0 || cnt > Tseq) {
            if (i0 == 0 && lane == 0) atomicOr(status, ST_BAD_COUNT);
            cnt = cnt < 0 ? 0 : Tseq;
        }
        if (i0 == 0 && lane == 0 && r_eff != nullptr) r_eff[b] = cnt;
        if (i0 >= cnt) return;
        const int32_t* list = rep_in + (int64_t)b * Tseq;
        int32_t idx[NORM_U], prev[NORM_U];
#pragma unroll
        for (int u = 0; u < NORM_U; ++u) {
            const int i = i0 + u * R + sub;
            idx[u] = i < cnt ? list[i] : -1;
            prev[u] = (i < cnt && i > 0) ? list[i - 1] : -1;
        }
        uint4 x[NORM_U];
        bool ok[NORM_U];
#pragma unroll
        for (int u = 0; u < NORM_U; ++u) {
            const int i = i0 + u * R + sub;
            ok[u] = i < cnt && idx[u] >= 0 && idx[u] < Tseq && prev[u] < idx[u];
            if (i < cnt && !ok[u] && gl == 0) atomicOr(status, ST_BAD_INDEX);
            x[u] = make_uint4(0u, 0u, 0u, 0u);
            if (ok[u] && gl < nvec)
                x[u] = __ldg(reinterpret_cast<const uint4*>(X + (int64_t)b * xb + (int64_t)idx[u] * ldx) + gl);
        }
#pragma unroll
        for (int u = 0; u < NORM_U; ++u) {
            const int i = i0 + u * R + sub;
            float ss = Vec16<T>::sumsq(x[u]);
            for (int o = G >> 1; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
            if (!ok[u]) continue;
            const int64_t prow = (int64_t)b * Tseq + i;
            if (gl < nvec) reinterpret_cast<uint4*>(Xrep + prow * (int64_t)d)[gl] = x[u];
            if (gl == 0) {
                inv_rep[prow] = (ss <= 3.0e38f && ss > 0.f) ? 1.0f / sqrtf(ss) : 0.f;
                if (role != nullptr) role[(int64_t)b * Tseq + idx[u]] = i + 1;
            }
        }
        return;
    }
}

cudaError_t launch_norm_gather(ada_ctx* ctx, const void* X, int B, int T, int d, int64_t ldx,
                               int64_t xb, ada_dtype dt, float* inv_norm, void* Xhat, const int32_t* rep_in,
                               const int32_t* rep_in_cnt, int32_t* role, int32_t* r_eff, void* Xrep,
                               float* inv_rep, cudaStream_t s) {
    const int64_t n_rows = (int64_t)B * T;
    const int warps = 8;
    const bool gather_only = inv_norm == nullptr && Xhat == nullptr;
    // rows per norm warp: lane groups of the next power of two at or above the row's vector count
    const int nvec = d / (dt == ADA_F32 ? 4 : 8);
    int G = 32;
    if (nvec <= 16) for (G = 1; G < nvec; G <<= 1) {}
    const int rpw = G == 32 ? 1 : (32 / G) * NORM_U;
    const int64_t n_norm_warps = (n_rows + rpw - 1) / rpw;
    // list warps: one per list position, or one per rpw positions of a sequence (short rows)
    const int64_t n_list_warps = rpw == 1 ? n_rows : (int64_t)B * ((T + rpw - 1) / rpw);
    const int64_t n_warps = gather_only ? n_list_warps
                                        : (rep_in != nullptr ? n_norm_warps + n_list_warps : n_norm_warps);
    const unsigned grid = (unsigned)((n_warps + warps - 1) / warps);
    prof_begin(ctx, K_NORM_GATHER, s);
    if (rpw > 1) {
        if (dt == ADA_F32) {
            launch_k(ctx, k_norm_gather_short<float>, dim3(grid), dim3(warps * 32), 0, s,
                (const float*)X, n_rows, T, d, ldx, xb, rpw, n_norm_warps, inv_norm, (float*)Xhat, rep_in,
                rep_in_cnt, role, r_eff, (float*)Xrep, inv_rep, ctx->status);
        } else {
            launch_k(ctx, k_norm_gather_short<__nv_bfloat16>, dim3(grid), dim3(warps * 32), 0, s,
                (const __nv_bfloat16*)X, n_rows, T, d, ldx, xb, rpw, n_norm_warps, inv_norm,
                (__nv_bfloat16*)Xhat, rep_in, rep_in_cnt, role, r_eff, (__nv_bfloat16*)Xrep, inv_rep,
                ctx->status);
        }
    } else if (dt == ADA_F32) {
        launch_k(ctx, k_norm_gather<float>, dim3(grid), dim3(warps * 32), 0, s,
            (const float*)X, n_rows, T, d, ldx, xb, inv_norm, (float*)Xhat, rep_in, rep_in_cnt, role,
            r_eff, (float*)Xrep, inv_rep, ctx->status);
    } else {
        launch_k(ctx, k_norm_gather<__nv_bfloat16>, dim3(grid), dim3(warps * 32), 0, s,
            (const __nv_bfloat16*)X, n_rows, T, d, ldx, xb, inv_norm, (__nv_bfloat16*)Xhat, rep_in,
            rep_in_cnt, role, r_eff, (__nv_bfloat16*)Xrep, inv_rep, ctx->status);
    }
    prof_end(ctx, s);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// fp32 on the bf16 tensor cores: every fp32 value is split into three bf16 terms
//   x = hi + mid + lo,  hi = bf16(x), mid = bf16(x - hi), lo = bf16(x - hi - mid)
// (both differences are exact in fp32), and a dot product is evaluated as the six largest
// of the nine cross terms, hi.hi + hi.mid + mid.hi + hi.lo + lo.hi + mid.mid, all of whose
// bf16 x bf16 products are exact in the fp32 accumulator.  What is dropped is below
// 2^-23 |x||y|, i.e. fp32 rounding level.  The six terms become ONE bf16 contraction of
// length 6d by laying the terms side by side:
//   A' = [hi | hi | mid | hi | lo | mid],   B' = [hi | mid | hi | lo | hi | mid].
// This kernel writes A' and B' for the rows of X (job 0, which also yields 1/||x||) and for
// the gathered representative rows (job 1, row count resident on the device).
// ---------------------------------------------------------------------------
struct SplitJob {
    const float* X;          // rows to split
    int64_t ldx;             // row stride of X in elements
    int64_t xb;              // sequence stride of X in elements
    int rows_per_seq;        // rows per sequence (capacity)
    const int32_t* n_dev;    // [B] rows actually present per sequence, or NULL = all
    __nv_bfloat16* A;        // [B*rows_per_seq][6d]
    __nv_bfloat16* Bm;       // [B*rows_per_seq][6d]
    float* inv_norm;         // optional
};

__device__ __forceinline__ void split3(float x, __nv_bfloat16& hi, __nv_bfloat16& mid, __nv_bfloat16& lo) {
    hi = __float2bfloat16_rn(x);
    const float r1 = x - __bfloat162float(hi);
    mid = __float2bfloat16_rn(r1);
    const float r2 = r1 - __bfloat162float(mid);
    lo = __float2bfloat16_rn(r2);
}

__global__ void __launch_bounds__(256)
k_split_bf16(const SplitJob j0, const SplitJob j1, int64_t n_rows, int d, unsigned* __restrict__ status) {
    grid_dep_wait();
    const int lane = threadIdx.x & 31;
    int64_t w = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const bool second = w >= n_rows;
    if (second) w -= n_rows;
    const SplitJob& j = second ? j1 : j0;
    if (j.X == nullptr || w >= n_rows) return;
    if (j.n_dev != nullptr) {
        const int b = (int)(w / j.rows_per_seq), i = (int)(w % j.rows_per_seq);
        if (i >= j.n_dev[b]) return;
    }
    const float4* src = reinterpret_cast<const float4*>(j.X + (w / j.rows_per_seq) * j.xb +
                                                        (w % j.rows_per_seq) * j.ldx);
    __nv_bfloat16* a = j.A + w * (int64_t)(6 * d);
    __nv_bfloat16* bm = j.Bm + w * (int64_t)(6 * d);
    float ss = 0.f;
    for (int v = lane; v < (d >> 2); v += 32) {            // d is a multiple of 4
        const float4 x = __ldg(src + v);
        const float xs[4] = {x.x, x.y, x.z, x.w};
        __nv_bfloat16 hi[4], mid[4], lo[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            ss = fmaf(xs[q], xs[q], ss);
            split3(xs[q], hi[q], mid[q], lo[q]);
        }
        const uint2 H = *reinterpret_cast<const uint2*>(hi), M = *reinterpret_cast<const uint2*>(mid),
                    L = *reinterpret_cast<const uint2*>(lo);
        const int k = v * 4;
        // A' = [hi | hi | mid | hi | lo | mid]
        *reinterpret_cast<uint2*>(a + 0 * d + k) = H;
        *reinterpret_cast<uint2*>(a + 1 * d + k) = H;
        *reinterpret_cast<uint2*>(a + 2 * d + k) = M;
        *reinterpret_cast<uint2*>(a + 3 * d + k) = H;
        *reinterpret_cast<uint2*>(a + 4 * d + k) = L;
        *reinterpret_cast<uint2*>(a + 5 * d + k) = M;
        // B' = [hi | mid | hi | lo | hi | mid]
        *reinterpret_cast<uint2*>(bm + 0 * d + k) = H;
        *reinterpret_cast<uint2*>(bm + 1 * d + k) = M;
        *reinterpret_cast<uint2*>(bm + 2 * d + k) = H;
        *reinterpret_cast<uint2*>(bm + 3 * d + k) = L;
        *reinterpret_cast<uint2*>(bm + 4 * d + k) = H;
        *reinterpret_cast<uint2*>(bm + 5 * d + k) = M;
    }
    if (j.inv_norm != nullptr) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        float inv = 0.f;
        if (!(ss <= 3.0e38f)) {
            if (lane == 0) atomicOr(status, ST_NONFINITE);
        } else if (ss > 0.f) {
            inv = 1.0f / sqrtf(ss);
        } else if (lane == 0) {
            atomicAdd(status + 1, 1u);
        }
        if (lane == 0) j.inv_norm[w] = inv;
    }
}

// X (B*T rows) -> ctx->splitXA/XB (+ inv_norm); with_rep: ctx->Xrep rows below r_eff -> splitRA/RB
cudaError_t launch_split(ada_ctx* ctx, const void* X, int B, int T, int d, int64_t ldx, int64_t xb,
                         bool with_rep, cudaStream_t s) {
    const int64_t n_rows = (int64_t)B * T;
    SplitJob j0, j1;
    j0.X = static_cast<const float*>(X); j0.ldx = ldx; j0.xb = xb; j0.rows_per_seq = T; j0.n_dev = nullptr;
    j0.A = static_cast<__nv_bfloat16*>(ctx->splitXA); j0.Bm = static_cast<__nv_bfloat16*>(ctx->splitXB);
    j0.inv_norm = ctx->inv_norm;
    j1 = j0;
    j1.X = with_rep ? static_cast<const float*>(ctx->Xrep) : nullptr; j1.ldx = d; j1.xb = (int64_t)T * d; j1.n_dev = ctx->r_eff;
    j1.A = static_cast<__nv_bfloat16*>(ctx->splitRA); j1.Bm = static_cast<__nv_bfloat16*>(ctx->splitRB);
    j1.inv_norm = nullptr;
    const int warps = 8;
    const int64_t n_warps = with_rep ? 2 * n_rows : n_rows;
    prof_begin(ctx, K_SPLIT, s);
    launch_k(ctx, k_split_bf16, dim3((unsigned)((n_warps + warps - 1) / warps)), dim3(warps * 32), 0, s, j0, j1, n_rows, d,
                                                                                  ctx->status);
    prof_end(ctx, s);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Compaction (Definition 1's threshold; Algorithm 1 lines 5, 9, 10-11 and the lists of
// Eq. 6).  Every 1024-thread block owns 1024 consecutive tokens of one sequence, one token
// per thread, so all loads are coalesced and the whole sequence is in flight at once.
// A block reduces its own counts, publishes them (one 64-bit word: three 21-bit counts
// and a READY bit), then sums the words of the blocks before it -- those never wait on
// anything, so the look-back is one round trip -- and writes its slice of the ascending
// lists.  The last block to finish clears the published words and the counters, and every
// thread clears the scratch it read, so the workspace is all-zero again when the kernel
// ends and no memset is needed between calls.
// ---------------------------------------------------------------------------
constexpr unsigned long long AGG_READY = 1ull << 63;
constexpr unsigned long long AGG_MASK = (1ull << 21) - 1;

struct CompactArgs {
    unsigned* g_tok;             // gamma (full) / gamma_cross by token, bit patterns
    unsigned* g_rep;             // gamma_rep by position (cascade) or NULL
    int32_t* role;               // 0 / position+1 (cascade) or NULL
    unsigned long long* agg;     // [B][agg_stride] published block counts
    unsigned* done_ctr;          // blocks finished
    unsigned* dep_ctr;           // dependency counter of the fused Gram launch (cleared here)
    unsigned* status;
    int agg_stride, T;
    float thr;
    int32_t *keep_idx, *keep_cnt, *add_idx, *add_cnt, *rem_idx, *rem_cnt;
    float *gamma_a, *gamma_b;    // full: gamma | cascade: gamma_rep, gamma_cross (optional)
    const float* row_scale;      // cascade: 1/||x_t|| still to be applied to g_tok, or NULL
    // adaptive threshold (Section 8.1)
    const float* thr_seq;        // [B] thresholds of this step, or NULL = thr
    const int32_t* r_in;         // [B] inherited counts (Eq. 6 denominator)
    TauUpdate tu;
};

// thr_seq[b] = (float)(1 - tau_b^2), 1 - tau^2 in fp64 as for a host-side tau
__global__ void k_tau_thr(const double* __restrict__ tau_state, int B, float* __restrict__ thr_seq,
                          unsigned* __restrict__ status) {
    grid_dep_wait();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const double tau = tau_state[b];
    if (!(tau > 0.0 && tau < 1.0)) atomicOr(status, ST_BAD_TAU);
    thr_seq[b] = (float)__dsub_rn(1.0, __dmul_rn(tau, tau));
}

__device__ __forceinline__ unsigned long long block_exclusive_scan(unsigned long long v,
                                                                   unsigned long long* s_warp,
                                                                   unsigned long long& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const unsigned long long wv = s_warp[lane];
        unsigned long long wi = wv;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long n = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += n;
        }
        s_warp[lane] = wi - wv;
        if (lane == 31) s_warp[32] = wi;
    }
    __syncthreads();
    const unsigned long long off = s_warp[warp] + incl - v;
    total = s_warp[32];
    __syncthreads();   // s_warp is reused
    return off;
}

__global__ void __launch_bounds__(1024) k_compact(const CompactArgs a) {
    __shared__ unsigned long long s_warp[33];
    grid_dep_wait();
    grid_dep_launch_next();
    const int b = blockIdx.y, blk = blockIdx.x, nblk = gridDim.x;
    const int t = blk * 1024 + threadIdx.x;
    const int64_t o = (int64_t)b * a.T;
    const bool in = t < a.T;
    const bool cascade = a.role != nullptr;
    const unsigned faulted = a.status[0];
    const float thr = a.thr_seq != nullptr ? a.thr_seq[b] : a.thr;

    // independent loads first, the position-indexed gather second
    const int pos = (cascade && in) ? a.role[o + t] : 0;
    const unsigned gt = in ? a.g_tok[o + t] : 0u;
    const float rs = (in && a.row_scale != nullptr) ? a.row_scale[o + t] : 1.0f;
    const unsigned gp = pos > 0 ? a.g_rep[o + pos - 1] : 0u;
    bool keep = false, add = false, rem = false;
    if (in) {
        float ga = 0.f, gb = 0.f;
        if (pos > 0) {                    // inherited representative: line 5
            ga = __uint_as_float(gp);
            keep = ga < thr;
            rem = !keep;
            a.g_rep[o + pos - 1] = 0u;
            a.role[o + t] = 0;
        } else {                          // Definition 1 / line 9
            // (an untouched entry is a maximum over nothing: 0 whatever the row's norm)
            gb = gt != 0u ? __uint_as_float(gt) * rs : 0.f;
            keep = gb < thr;
            add = cascade && keep;
        }
        a.g_tok[o + t] = 0u;
        if (cascade) {
            if (a.gamma_a != nullptr) a.gamma_a[o + t] = ga;
            if (a.gamma_b != nullptr) a.gamma_b[o + t] = gb;
            if (faulted != 0u) a.g_rep[o + t] = 0u;   // a rejected list leaves positions without a token
        } else if (a.gamma_a != nullptr) {
            a.gamma_a[o + t] = gb;
        }
    }
    const unsigned long long mine = (keep ? 1ull : 0ull) | (add ? 1ull << 21 : 0ull) | (rem ? 1ull << 42 : 0ull);
    unsigned long long total;
    const unsigned long long off = block_exclusive_scan(mine, s_warp, total);

    unsigned long long* agg = a.agg + (int64_t)b * a.agg_stride;
    if (threadIdx.x == 0) atomicExch(agg + blk, total | AGG_READY);
    // look-back over the blocks before this one (bounded spin; they wait on nothing)
    unsigned long long before = 0;
    for (int j = threadIdx.x; j < blk; j += 1024) {
        unsigned long long v;
        unsigned polls = 0;
        long long t0 = 0;
        while (true) {
            v = *reinterpret_cast<volatile unsigned long long*>(agg + j);
            if (v & AGG_READY) break;
            if ((++polls & 1023u) == 0) {
                const long long now = clock64();
                if (t0 == 0) t0 = now;
                else if (now - t0 > 4000000000ll) { atomicOr(a.status, ST_TIMEOUT); v = 0; break; }
            }
        }
        before += v & ~AGG_READY;
    }
    unsigned long long base;
    block_exclusive_scan(before, s_warp, base);

    const int nk = (int)((base + off) & AGG_MASK);
    const int na = (int)(((base + off) >> 21) & AGG_MASK);
    const int nr = (int)(((base + off) >> 42) & AGG_MASK);
    if (keep) a.keep_idx[o + nk] = t;
    if (add) a.add_idx[o + na] = t;
    if (rem) a.rem_idx[o + nr] = t;
    if (blk == nblk - 1 && threadIdx.x == 0) {
        const unsigned long long all = base + total;
        a.keep_cnt[b] = (int)(all & AGG_MASK);
        if (cascade) {
            const int n_add = (int)((all >> 21) & AGG_MASK), n_rem = (int)((all >> 42) & AGG_MASK);
            a.add_cnt[b] = n_add;
            a.rem_cnt[b] = n_rem;
            if (a.tu.tau_state != nullptr) {
                // Eq. (6), then the threshold of the next layer: one rounded fp64 operation at a
                // time (no fused multiply-add), so that the state is reproducible bit for bit
                const int r_in = a.r_in[b];
                const bool defined = r_in > 0;
                const double rho = defined ? __ddiv_rn((double)(n_add + n_rem), (double)r_in) : 0.0;
                if (a.tu.turnover != nullptr)
                    a.tu.turnover[b] = defined ? (float)rho : __int_as_float(0x7fc00000);
                if (a.tu.update) {
                    double t = a.tu.tau_state[b];
                    if (defined) t = __dadd_rn(t, __dmul_rn(a.tu.gain, __dsub_rn(a.tu.target, rho)));
                    if (t < a.tu.tau_min) t = a.tu.tau_min;
                    if (t > a.tu.tau_max) t = a.tu.tau_max;
                    a.tu.tau_state[b] = t;
                }
            }
        }
    }
    // the last block to finish restores the zero state of the shared words
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned n_blocks = gridDim.x * gridDim.y;
        if (atomicAdd(a.done_ctr, 1u) == n_blocks - 1) {
            for (unsigned q = 0; q < gridDim.y; ++q)
                for (unsigned j = 0; j < gridDim.x; ++j) a.agg[(int64_t)q * a.agg_stride + j] = 0ull;
            *a.done_ctr = 0u;
            a.dep_ctr[0] = 0u;
            a.dep_ctr[1] = 0u;   // norm warps' counter of the Gram launch
            a.dep_ctr[3] = 0u;   // in-launch gather counter
        }
    }
}

// Nearest-representative map (Section 2.3): turns the packed keys of the argmax Gram launch
// into token indices.  A representative is its own nearest representative; a token whose
// correlations are all zero gets the first representative (lowest index among equals); an
// empty set gives -1.  Clears the keys and the role map it reads.
__global__ void __launch_bounds__(256)
k_nearest_finish(unsigned long long* __restrict__ near_key, int32_t* __restrict__ role,
                 const int32_t* __restrict__ r_eff, const float* __restrict__ inv_norm,
                 const int32_t* __restrict__ rep_idx, int T, int32_t* __restrict__ nearest_idx,
                 float* __restrict__ nearest_gamma) {
    grid_dep_wait();
    const int b = blockIdx.y, t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    const int64_t o = (int64_t)b * T;
    const unsigned long long key = near_key[o + t];
    const int p = role[o + t];
    near_key[o + t] = 0ull;
    role[o + t] = 0;
    int idx;
    float g;
    if (p > 0) {
        idx = t;
        g = inv_norm[o + t] > 0.f ? 1.f : 0.f;
    } else if (r_eff[b] <= 0) {
        idx = -1;
        g = 0.f;
    } else if (key == 0ull) {
        idx = rep_idx[o];
        g = 0.f;
    } else {
        const unsigned pos = 0xFFFFFFFFu - (unsigned)(key & 0xFFFFFFFFull);
        idx = rep_idx[o + pos];
        g = __uint_as_float((unsigned)(key >> 32));
    }
    nearest_idx[o + t] = idx;
    if (nearest_gamma != nullptr) nearest_gamma[o + t] = g;
}

cudaError_t launch_nearest_finish(ada_ctx* ctx, int B, int T, const int32_t* rep_idx,
                                  int32_t* nearest_idx, float* nearest_gamma, cudaStream_t s) {
    prof_begin(ctx, K_NEAREST_FINISH, s);
    launch_k(ctx, k_nearest_finish, dim3((T + 255) / 256, B), dim3(256), 0, s, ctx->near_key, ctx->role, ctx->r_eff,
                                                               ctx->inv_norm, rep_idx, T, nearest_idx,
                                                               nearest_gamma);
    prof_end(ctx, s);
    return cudaGetLastError();
}

static cudaError_t launch_compact(ada_ctx* ctx, int kid, const CompactArgs& a, int B, cudaStream_t s) {
    const int nblk = (a.T + 1023) / 1024;
    if (nblk > a.agg_stride) return cudaErrorInvalidValue;
    prof_begin(ctx, kid, s);
    launch_k(ctx, k_compact, dim3(nblk, B), dim3(1024), 0, s, a);
    prof_end(ctx, s);
    return cudaGetLastError();
}

cudaError_t launch_compact_full(ada_ctx* ctx, int B, int T, float thr, int32_t* rep_idx,
                                int32_t* rep_cnt, float* gamma, cudaStream_t s) {
    CompactArgs a;
    a.g_tok = ctx->g_tok; a.g_rep = nullptr; a.role = nullptr;
    a.agg = ctx->agg; a.done_ctr = ctx->done_ctr; a.dep_ctr = ctx->tile_ctr; a.status = ctx->status;
    a.agg_stride = ctx->agg_stride; a.T = T; a.thr = thr;
    a.keep_idx = rep_idx; a.keep_cnt = rep_cnt;
    a.add_idx = nullptr; a.add_cnt = nullptr; a.rem_idx = nullptr; a.rem_cnt = nullptr;
    a.gamma_a = gamma; a.gamma_b = nullptr; a.row_scale = nullptr;
    a.thr_seq = nullptr; a.r_in = nullptr;
    memset(&a.tu, 0, sizeof(a.tu));
    return launch_compact(ctx, K_COMPACT_FULL, a, B, s);
}

cudaError_t launch_compact_cascade(ada_ctx* ctx, int B, int T, float thr, int32_t* rep_out,
                                   int32_t* rep_out_cnt, int32_t* add_idx, int32_t* add_cnt,
                                   int32_t* rem_idx, int32_t* rem_cnt, float* gamma_rep,
                                   float* gamma_cross, const TauUpdate& tu, bool row_scale,
                                   cudaStream_t s) {
    CompactArgs a;
    a.g_tok = ctx->g_tok; a.g_rep = ctx->g_rep; a.role = ctx->role;
    a.agg = ctx->agg; a.done_ctr = ctx->done_ctr; a.dep_ctr = ctx->tile_ctr; a.status = ctx->status;
    a.agg_stride = ctx->agg_stride; a.T = T; a.thr = thr;
    a.keep_idx = rep_out; a.keep_cnt = rep_out_cnt;
    a.add_idx = add_idx; a.add_cnt = add_cnt; a.rem_idx = rem_idx; a.rem_cnt = rem_cnt;
    a.gamma_a = gamma_rep; a.gamma_b = gamma_cross;
    a.row_scale = row_scale ? ctx->inv_norm : nullptr;
    a.thr_seq = tu.tau_state != nullptr ? ctx->thr_seq : nullptr;
    a.r_in = ctx->r_eff;
    a.tu = tu;
    return launch_compact(ctx, K_COMPACT_CASCADE, a, B, s);
}

cudaError_t launch_tau_thr(ada_ctx* ctx, int B, const double* tau_state, cudaStream_t s) {
    launch_k(ctx, k_tau_thr, dim3((B + 127) / 128), dim3(128), 0, s, tau_state, B, ctx->thr_seq, ctx->status);
    return cudaGetLastError();
}

}  // namespace ada
