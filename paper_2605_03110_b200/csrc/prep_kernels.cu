// HBM-bound helper kernels of the selection path: inherited-set scatter and
// validation, fused row-norm + representative gather, and the ballot /
// prefix-sum compaction that turns gamma into sorted index lists.
#include "common.cuh"

namespace ada {

// ---------------------------------------------------------------------------
// Scatter the inherited list into a per-token role map (0 = not inherited,
// p+1 = position p) and validate it.  Algorithm 1 "Require": R^(l).
// The role map must be zero on entry.
// ---------------------------------------------------------------------------
__global__ void k_scatter_roles(const int32_t* __restrict__ rep_in,
                                const int32_t* __restrict__ rep_in_cnt, int T,
                                int32_t* __restrict__ role, int32_t* __restrict__ r_eff,
                                unsigned* __restrict__ status) {
    const int b = blockIdx.y;
    int cnt = rep_in_cnt[b];
    if (cnt < 0 || cnt > T) {
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicOr(status, ST_BAD_COUNT);
        cnt = cnt < 0 ? 0 : T;
    }
    if (threadIdx.x == 0 && blockIdx.x == 0) r_eff[b] = cnt;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= cnt) return;
    const int32_t* list = rep_in + (int64_t)b * T;
    const int32_t idx = list[i];
    bool ok = idx >= 0 && idx < T;
    if (ok && i > 0) ok = list[i - 1] < idx;
    if (ok) role[(int64_t)b * T + idx] = i + 1;
    else atomicOr(status, ST_BAD_INDEX);
}

cudaError_t launch_scatter(ada_ctx* ctx, const int32_t* rep_in, const int32_t* rep_in_cnt, int B,
                           int T, cudaStream_t s) {
    dim3 grid((T + 255) / 256, B);
    prof_begin(ctx, K_SCATTER, s);
    k_scatter_roles<<<grid, 256, 0, s>>>(rep_in, rep_in_cnt, T, ctx->role, ctx->r_eff, ctx->status);
    prof_end(ctx, s);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Row normalisation fused with the representative gather (Section 2.1;
// Algorithm 1 lines 1-2).  One warp per row, 128-bit loads.  inv_norm[t] =
// 1/||x_t|| in fp32 (0 for a zero row).  Rows whose role is non-zero are also
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

template <typename T>
__global__ void __launch_bounds__(256)
k_norm_gather(const T* __restrict__ X, int64_t n_rows, int Tseq, int d, int64_t ldx,
              float* __restrict__ inv_norm, T* __restrict__ Xhat,
              const int32_t* __restrict__ role, T* __restrict__ Xrep,
              float* __restrict__ inv_rep, unsigned* __restrict__ status) {
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= n_rows) return;
    constexpr int N = Vec16<T>::N;
    const int nvec = d / N;  // d*es is a multiple of 16 bytes
    const uint4* src = reinterpret_cast<const uint4*>(X + row * ldx);
    float ss = 0.f;
    for (int v = lane; v < nvec; v += 32) ss += Vec16<T>::sumsq(__ldg(src + v));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
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
    if (role != nullptr) {
        const int p = role[row];
        if (p > 0) {
            const int64_t b = row / Tseq;
            const int64_t prow = b * Tseq + (p - 1);
            uint4* dst = reinterpret_cast<uint4*>(Xrep + prow * (int64_t)d);
            for (int v = lane; v < nvec; v += 32) dst[v] = __ldg(src + v);
            if (lane == 0) inv_rep[prow] = inv;
        }
    }
}

cudaError_t launch_norm_gather(ada_ctx* ctx, const void* X, int B, int T, int d, int64_t ldx,
                               ada_dtype dt, float* inv_norm, void* Xhat, const int32_t* role,
                               void* Xrep, float* inv_rep, cudaStream_t s) {
    const int64_t n_rows = (int64_t)B * T;
    const int warps = 8;
    const unsigned grid = (unsigned)((n_rows + warps - 1) / warps);
    prof_begin(ctx, K_NORM_GATHER, s);
    if (dt == ADA_F32) {
        k_norm_gather<float><<<grid, warps * 32, 0, s>>>(
            (const float*)X, n_rows, T, d, ldx, inv_norm, (float*)Xhat, role, (float*)Xrep,
            inv_rep, ctx->status);
    } else {
        k_norm_gather<__nv_bfloat16><<<grid, warps * 32, 0, s>>>(
            (const __nv_bfloat16*)X, n_rows, T, d, ldx, inv_norm, (__nv_bfloat16*)Xhat, role,
            (__nv_bfloat16*)Xrep, inv_rep, ctx->status);
    }
    prof_end(ctx, s);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Compaction.  One 1024-thread block per sequence walks the tokens in order;
// every 1024-token chunk is reduced with warp ballots and a prefix sum over
// the 32 warp totals, so the output lists come out ascending.
// ---------------------------------------------------------------------------
struct Scan3 {
    int a, b, c;
};

// Exclusive offsets of up to three flag streams inside one 1024-token chunk.
__device__ __forceinline__ Scan3 block_offsets(bool fa, bool fb, bool fc, int* s_tot /*[3][33]*/,
                                               Scan3& chunk_total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned lt = (1u << lane) - 1u;
    const unsigned ba = __ballot_sync(0xffffffffu, fa);
    const unsigned bb = __ballot_sync(0xffffffffu, fb);
    const unsigned bc = __ballot_sync(0xffffffffu, fc);
    if (lane == 0) {
        s_tot[warp] = __popc(ba);
        s_tot[33 + warp] = __popc(bb);
        s_tot[66 + warp] = __popc(bc);
    }
    __syncthreads();
    if (warp < 3) {
        const int v = s_tot[33 * warp + lane];
        int incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int n = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += n;
        }
        s_tot[33 * warp + lane] = incl - v;                 // exclusive prefix of warp totals
        if (lane == 31) s_tot[33 * warp + 32] = incl;       // chunk total
    }
    __syncthreads();
    Scan3 off;
    off.a = s_tot[warp] + __popc(ba & lt);
    off.b = s_tot[33 + warp] + __popc(bb & lt);
    off.c = s_tot[66 + warp] + __popc(bc & lt);
    chunk_total.a = s_tot[32];
    chunk_total.b = s_tot[33 + 32];
    chunk_total.c = s_tot[66 + 32];
    __syncthreads();  // s_tot is reused by the next chunk
    return off;
}

// Definition 1: R = { t : gamma_t < thr }.
__global__ void __launch_bounds__(1024)
k_compact_full(const unsigned* __restrict__ g_tok, int T, float thr,
               int32_t* __restrict__ rep_idx, int32_t* __restrict__ rep_cnt,
               float* __restrict__ gamma) {
    __shared__ int s_tot[99];
    const int b = blockIdx.x;
    const unsigned* g = g_tok + (int64_t)b * T;
    int32_t* out = rep_idx + (int64_t)b * T;
    int base_a = 0;
    for (int t0 = 0; t0 < T; t0 += 1024) {
        const int t = t0 + threadIdx.x;
        float gv = 0.f;
        bool rep = false;
        if (t < T) {
            gv = __uint_as_float(g[t]);
            rep = gv < thr;
            if (gamma != nullptr) gamma[(int64_t)b * T + t] = gv;
        }
        Scan3 tot;
        const Scan3 off = block_offsets(rep, false, false, s_tot, tot);
        if (rep) out[base_a + off.a] = t;
        base_a += tot.a;
    }
    if (threadIdx.x == 0) rep_cnt[b] = base_a;
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
k_compact_cascade(const unsigned* __restrict__ g_tok, const unsigned* __restrict__ g_rep,
                  const int32_t* __restrict__ role, int T, float thr,
                  int32_t* __restrict__ rep_out, int32_t* __restrict__ rep_out_cnt,
                  int32_t* __restrict__ add_idx, int32_t* __restrict__ add_cnt,
                  int32_t* __restrict__ rem_idx, int32_t* __restrict__ rem_cnt,
                  float* __restrict__ gamma_rep, float* __restrict__ gamma_cross) {
    __shared__ int s_tot[99];
    const int b = blockIdx.x;
    const int64_t o = (int64_t)b * T;
    int base_keep = 0, base_add = 0, base_rem = 0;
    for (int t0 = 0; t0 < T; t0 += 1024) {
        const int t = t0 + threadIdx.x;
        bool keep = false, add = false, rem = false;
        if (t < T) {
            const int p = role[o + t];
            float gr = 0.f, gc = 0.f;
            if (p > 0) {  // inherited representative: line 5
                gr = __uint_as_float(g_rep[o + p - 1]);
                keep = gr < thr;
                rem = !keep;
            } else {      // line 9
                gc = __uint_as_float(g_tok[o + t]);
                add = gc < thr;
                keep = add;
            }
            if (gamma_rep != nullptr) gamma_rep[o + t] = gr;
            if (gamma_cross != nullptr) gamma_cross[o + t] = gc;
        }
        Scan3 tot;
        const Scan3 off = block_offsets(keep, add, rem, s_tot, tot);
        if (keep) rep_out[o + base_keep + off.a] = t;
        if (add) add_idx[o + base_add + off.b] = t;
        if (rem) rem_idx[o + base_rem + off.c] = t;
        base_keep += tot.a;
        base_add += tot.b;
        base_rem += tot.c;
    }
    if (threadIdx.x == 0) {
        rep_out_cnt[b] = base_keep;
        add_cnt[b] = base_add;
        rem_cnt[b] = base_rem;
    }
}

cudaError_t launch_compact_cascade(ada_ctx* ctx, int B, int T, float thr, const int32_t* rep_in,
                                   int32_t* rep_out, int32_t* rep_out_cnt, int32_t* add_idx,
                                   int32_t* add_cnt, int32_t* rem_idx, int32_t* rem_cnt,
                                   float* gamma_rep, float* gamma_cross, cudaStream_t s) {
    (void)rep_in;
    prof_begin(ctx, K_COMPACT_CASCADE, s);
    k_compact_cascade<<<B, 1024, 0, s>>>(ctx->g_tok, ctx->g_rep, ctx->role, T, thr, rep_out,
                                         rep_out_cnt, add_idx, add_cnt, rem_idx, rem_cnt,
                                         gamma_rep, gamma_cross);
    prof_end(ctx, s);
    return cudaGetLastError();
}

}  // namespace ada
