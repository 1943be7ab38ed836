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
k_norm_gather(const T* __restrict__ X, int64_t n_rows, int Tseq, int d, int64_t ldx,
              float* __restrict__ inv_norm, T* __restrict__ Xhat,
              const int32_t* __restrict__ rep_in, const int32_t* __restrict__ rep_in_cnt,
              int32_t* __restrict__ role, int32_t* __restrict__ r_eff, T* __restrict__ Xrep,
              float* __restrict__ inv_rep, unsigned* __restrict__ status) {
    const int lane = threadIdx.x & 31;
    int64_t w = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    constexpr int N = Vec16<T>::N;
    const int nvec = d / N;  // d*es is a multiple of 16 bytes
    if (w < n_rows) {
        const int64_t row = w;
        const uint4* src = reinterpret_cast<const uint4*>(X + row * ldx);
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
    const uint4* src = reinterpret_cast<const uint4*>(X + ((int64_t)b * Tseq + idx) * ldx);
    uint4* dst = reinterpret_cast<uint4*>(Xrep + prow * (int64_t)d);
    float ss = 0.f;
    for (int v = lane; v < nvec; v += 32) {
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

cudaError_t launch_norm_gather(ada_ctx* ctx, const void* X, int B, int T, int d, int64_t ldx,
                               ada_dtype dt, float* inv_norm, void* Xhat, const int32_t* rep_in,
                               const int32_t* rep_in_cnt, int32_t* role, int32_t* r_eff, void* Xrep,
                               float* inv_rep, cudaStream_t s) {
    const int64_t n_rows = (int64_t)B * T;
    const int warps = 8;
    const int64_t n_warps = rep_in != nullptr ? 2 * n_rows : n_rows;
    const unsigned grid = (unsigned)((n_warps + warps - 1) / warps);
    prof_begin(ctx, K_NORM_GATHER, s);
    if (dt == ADA_F32) {
        k_norm_gather<float><<<grid, warps * 32, 0, s>>>(
            (const float*)X, n_rows, T, d, ldx, inv_norm, (float*)Xhat, rep_in, rep_in_cnt, role,
            r_eff, (float*)Xrep, inv_rep, ctx->status);
    } else {
        k_norm_gather<__nv_bfloat16><<<grid, warps * 32, 0, s>>>(
            (const __nv_bfloat16*)X, n_rows, T, d, ldx, inv_norm, (__nv_bfloat16*)Xhat, rep_in,
            rep_in_cnt, role, r_eff, (__nv_bfloat16*)Xrep, inv_rep, ctx->status);
    }
    prof_end(ctx, s);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Compaction.  One 1024-thread block per sequence.  Each thread owns 8 consecutive
// tokens of an 8192-token chunk, so a chunk needs one block-wide prefix sum (warp
// shuffles + 32 warp totals) and the lists come out ascending.  The three running
// counts of the cascade update travel through the scan packed in one 64-bit word.
// The kernels also restore the workspace invariant: the gamma scratch, the role map
// and the dependency counter are zero again when they finish, so no memset is needed
// between calls.
// ---------------------------------------------------------------------------
constexpr int CPT = 8;                       // tokens per thread per chunk
constexpr int CHUNK = 1024 * CPT;

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
    __syncthreads();   // s_warp is reused by the next chunk
    return off;
}

// Definition 1: R = { t : gamma_t < thr }.
__global__ void __launch_bounds__(1024)
k_compact_full(unsigned* __restrict__ g_tok, int T, float thr, int32_t* __restrict__ rep_idx,
               int32_t* __restrict__ rep_cnt, float* __restrict__ gamma) {
    __shared__ unsigned long long s_warp[33];
    const int b = blockIdx.x;
    unsigned* g = g_tok + (int64_t)b * T;
    int32_t* out = rep_idx + (int64_t)b * T;
    float* go = gamma != nullptr ? gamma + (int64_t)b * T : nullptr;
    int base = 0;
    for (int t0 = 0; t0 < T; t0 += CHUNK) {
        const int first = t0 + threadIdx.x * CPT;
        float gv[CPT];
        unsigned flags = 0;
#pragma unroll
        for (int k = 0; k < CPT; ++k) {
            const int t = first + k;
            gv[k] = 0.f;
            if (t < T) {
                gv[k] = __uint_as_float(g[t]);
                g[t] = 0u;                                   // leave the scratch clean
                if (gv[k] < thr) flags |= 1u << k;
                if (go != nullptr) go[t] = gv[k];
            }
        }
        unsigned long long total;
        int off = base + (int)block_exclusive_scan((unsigned long long)__popc(flags), s_warp, total);
#pragma unroll
        for (int k = 0; k < CPT; ++k)
            if (flags & (1u << k)) out[off++] = first + k;
        base += (int)total;
    }
    if (threadIdx.x == 0) rep_cnt[b] = base;
}

cudaError_t launch_compact_full(ada_ctx* ctx, int B, int T, float thr, int32_t* rep_idx,
                                int32_t* rep_cnt, float* gamma, cudaStream_t s) {
    prof_begin(ctx, K_COMPACT_FULL, s);
    k_compact_full<<<B, 1024, 0, s>>>(ctx->g_tok, T, thr, rep_idx, rep_cnt, gamma);
    prof_end(ctx, s);
    return cudaGetLastError();
}

// Algorithm 1 lines 5, 9, 10-11 and the lists of Eq. (6).
__global__ void __launch_bounds__(1024)
k_compact_cascade(unsigned* __restrict__ g_tok, unsigned* __restrict__ g_rep,
                  int32_t* __restrict__ role, unsigned* __restrict__ dep_ctr,
                  const unsigned* __restrict__ status, int T, float thr,
                  int32_t* __restrict__ rep_out, int32_t* __restrict__ rep_out_cnt,
                  int32_t* __restrict__ add_idx, int32_t* __restrict__ add_cnt,
                  int32_t* __restrict__ rem_idx, int32_t* __restrict__ rem_cnt,
                  float* __restrict__ gamma_rep, float* __restrict__ gamma_cross) {
    __shared__ unsigned long long s_warp[33];
    const int b = blockIdx.x;
    const int64_t o = (int64_t)b * T;
    const unsigned faulted = status[0];
    int base_keep = 0, base_add = 0, base_rem = 0;
    for (int t0 = 0; t0 < T; t0 += CHUNK) {
        const int first = t0 + threadIdx.x * CPT;
        unsigned keep = 0, add = 0, rem = 0;
        int pos[CPT];
        unsigned gt[CPT], gp[CPT];
        // independent loads first, the position-indexed gather second: two round trips in all
#pragma unroll
        for (int k = 0; k < CPT; ++k) {
            const bool in = first + k < T;
            pos[k] = in ? role[o + first + k] : 0;
            gt[k] = in ? g_tok[o + first + k] : 0u;
        }
#pragma unroll
        for (int k = 0; k < CPT; ++k) gp[k] = pos[k] > 0 ? g_rep[o + pos[k] - 1] : 0u;
#pragma unroll
        for (int k = 0; k < CPT; ++k) {
            const int t = first + k;
            if (t >= T) continue;
            float gr = 0.f, gc = 0.f;
            if (pos[k] > 0) {       // inherited representative: line 5
                gr = __uint_as_float(gp[k]);
                g_rep[o + pos[k] - 1] = 0u;
                role[o + t] = 0;
                if (gr < thr) keep |= 1u << k; else rem |= 1u << k;
            } else {                // line 9
                gc = __uint_as_float(gt[k]);
                if (gc < thr) { add |= 1u << k; keep |= 1u << k; }
            }
            g_tok[o + t] = 0u;      // rows of inherited reps are never written, clearing is harmless
            if (gamma_rep != nullptr) gamma_rep[o + t] = gr;
            if (gamma_cross != nullptr) gamma_cross[o + t] = gc;
        }
        // three counts (each <= 8192 per chunk, running totals < 2^21) in one scan
        const unsigned long long packed = (unsigned long long)__popc(keep) |
                                          ((unsigned long long)__popc(add) << 21) |
                                          ((unsigned long long)__popc(rem) << 42);
        unsigned long long total;
        const unsigned long long off = block_exclusive_scan(packed, s_warp, total);
        int ok = base_keep + (int)(off & 0x1FFFFFu);
        int oa = base_add + (int)((off >> 21) & 0x1FFFFFu);
        int om = base_rem + (int)((off >> 42) & 0x1FFFFFu);
#pragma unroll
        for (int k = 0; k < CPT; ++k) {
            const int t = first + k;
            if (keep & (1u << k)) rep_out[o + ok++] = t;
            if (add & (1u << k)) add_idx[o + oa++] = t;
            if (rem & (1u << k)) rem_idx[o + om++] = t;
        }
        base_keep += (int)(total & 0x1FFFFFu);
        base_add += (int)((total >> 21) & 0x1FFFFFu);
        base_rem += (int)((total >> 42) & 0x1FFFFFu);
    }
    if (faulted != 0u) {
        // a rejected inherited list leaves positions without a token: clear them all
        for (int i = threadIdx.x; i < T; i += blockDim.x) g_rep[o + i] = 0u;
    }
    if (threadIdx.x == 0) {
        rep_out_cnt[b] = base_keep;
        add_cnt[b] = base_add;
        rem_cnt[b] = base_rem;
        if (b == 0) *dep_ctr = 0u;
    }
}

cudaError_t launch_compact_cascade(ada_ctx* ctx, int B, int T, float thr, int32_t* rep_out,
                                   int32_t* rep_out_cnt, int32_t* add_idx, int32_t* add_cnt,
                                   int32_t* rem_idx, int32_t* rem_cnt, float* gamma_rep,
                                   float* gamma_cross, cudaStream_t s) {
    prof_begin(ctx, K_COMPACT_CASCADE, s);
    k_compact_cascade<<<B, 1024, 0, s>>>(ctx->g_tok, ctx->g_rep, ctx->role, ctx->tile_ctr, ctx->status, T, thr,
                                         rep_out, rep_out_cnt, add_idx, add_cnt, rem_idx, rem_cnt,
                                         gamma_rep, gamma_cross);
    prof_end(ctx, s);
    return cudaGetLastError();
}

}  // namespace ada
