// Attention on the representative set (Section 2.3, Eq. 2) for sm_100a:
//     Attn_R = softmax(Q_R K_R^T / sqrt(d_h)) V_R,   one r x r problem per head,
// and the expansion of Section 2.3: a token outside R takes the output of its nearest
// representative.  Three kernels:
//   k_attn_gather   rows rho_i of Q and K go to contiguous per-head buffers (K-major, what the
//                   TMA unit and the MMA descriptors want); V_R is written TRANSPOSED per head
//                   (d_h x r, K-major for the second contraction), through a shared-memory tile
//   k_attn_reps     one CTA per (128 query rows, head).  Both contractions run on tcgen05:
//                   S = Q K^T into TMEM (two 128 x 128 fp32 buffers), softmax by four warps
//                   straight out of TMEM (one row per thread, so maxima and sums are
//                   thread-local), P rounded to bf16 into shared memory in the 128-byte
//                   swizzled K-major layout, O += P V^T into a third TMEM accumulator.  The
//                   softmax is two-pass (first the row maxima and sums over all key tiles, then
//                   the normalised probabilities), which costs a second Q K^T but needs no
//                   rescaling of the accumulator; r is a few thousand at most.
//   k_attn_expand   out[t] = out[nearest[t]] for the tokens outside R
// Every wait is bounded (see gram_tc_dev.cuh).
#include "gram_tc_dev.cuh"

namespace ada {

using namespace tc;

namespace {

constexpr int AQ = 128;                 // query rows per CTA (TMEM lanes)
constexpr int AKV = 128;                // keys per tile
constexpr int KB_BYTES = 128 * BK * 2;  // one 64-element K block of a 128-row tile: 16 KiB
constexpr int ATT_THREADS = 192;        // TMA producer, MMA issuer, four softmax warps

struct alignas(16) AttnShared {
    unsigned long long q_full, k_full[2], k_empty[2], v_full[2], v_empty[2];
    unsigned long long s_full[2], s_empty[2], p_full, p_empty, o_full;
    unsigned tmem_base;
    int abort_flag;
};
// Q (2 K blocks) | K ring 2 x 2 | V^T ring 2 x 2 | P (2 K blocks)
constexpr int ATT_SMEM = (2 + 4 + 4 + 2) * KB_BYTES + (int)sizeof(AttnShared) + 1024;
static_assert(ATT_SMEM <= 227 * 1024, "shared memory budget");

struct AttnMaps {
    CUtensorMap q, k, v;
};

__device__ __forceinline__ int clamp_count(const int32_t* cnt, int T) {
    return min(max(cnt[0], 0), T);
}

// ---------------------------------------------------------------- gather
// grid (Tp / 32, h), 256 threads.  Positions at or past r (up to the next multiple of 128)
// are filled with zeros, so that the padding of the last key tile is harmless.
__global__ void __launch_bounds__(256)
k_attn_gather(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K,
              const __nv_bfloat16* __restrict__ V, int T, int Tp, int h, int d_h, int64_t ld,
              const int32_t* __restrict__ rep_idx, const int32_t* __restrict__ rep_cnt,
              __nv_bfloat16* __restrict__ Qr, __nv_bfloat16* __restrict__ Kr,
              __nv_bfloat16* __restrict__ Vt, unsigned* __restrict__ status) {
    grid_dep_wait();
    __shared__ __nv_bfloat16 vs[32][128 + 8];
    __shared__ int tok[32];
    const int head = blockIdx.y, p0 = blockIdx.x * 32;
    const int r = clamp_count(rep_cnt, T);
    const int rpad = (r + AKV - 1) / AKV * AKV;
    if (p0 >= rpad) return;
    if (threadIdx.x < 32) {
        const int p = p0 + threadIdx.x;
        int t = p < r ? rep_idx[p] : -1;
        if (p < r && (t < 0 || t >= T)) { atomicOr(status, ST_BAD_INDEX); t = -1; }
        tok[threadIdx.x] = t;
    }
    __syncthreads();
    const int nvec = d_h >> 3;                       // 16-byte vectors per head row
    for (int i = threadIdx.x; i < 32 * nvec; i += blockDim.x) {
        const int pl = i / nvec, v = i % nvec;
        const int t = tok[pl];
        uint4 q = make_uint4(0u, 0u, 0u, 0u), k = q, w = q;
        if (t >= 0) {
            const int64_t off = (int64_t)t * ld + (int64_t)head * d_h + v * 8;
            q = __ldg(reinterpret_cast<const uint4*>(Q + off));
            k = __ldg(reinterpret_cast<const uint4*>(K + off));
            w = __ldg(reinterpret_cast<const uint4*>(V + off));
        }
        const int64_t row = ((int64_t)head * Tp + p0 + pl) * d_h + v * 8;
        *reinterpret_cast<uint4*>(Qr + row) = q;
        *reinterpret_cast<uint4*>(Kr + row) = k;
        *reinterpret_cast<uint4*>(&vs[pl][v * 8]) = w;
    }
    __syncthreads();
    // V^T: thread (c, half) writes 16 consecutive positions of feature c
    const int c = threadIdx.x >> 1, half = threadIdx.x & 1;
    if (c < d_h) {
        __align__(16) __nv_bfloat16 o[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) o[i] = vs[half * 16 + i][c];
        uint4* dst = reinterpret_cast<uint4*>(Vt + ((int64_t)head * d_h + c) * Tp + p0 + half * 16);
        dst[0] = *reinterpret_cast<const uint4*>(&o[0]);
        dst[1] = *reinterpret_cast<const uint4*>(&o[8]);
    }
}

// ---------------------------------------------------------------- attention
__global__ void __launch_bounds__(ATT_THREADS, 1)
k_attn_reps(const __grid_constant__ AttnMaps maps, int T, int d_h, int h,
            const int32_t* __restrict__ rep_idx, const int32_t* __restrict__ rep_cnt,
            float* __restrict__ out, int64_t ldo, int causal, unsigned* __restrict__ status) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    unsigned char* qs = smem;                          // Q tile: nkb K blocks
    unsigned char* ks = smem + 2 * KB_BYTES;           // K ring: 2 slots x 2 K blocks
    unsigned char* vs = smem + 6 * KB_BYTES;           // V^T ring: 2 slots x 2 K blocks of d_h rows
    unsigned char* ps = smem + 10 * KB_BYTES;          // P: 2 K blocks
    AttnShared& sh = *reinterpret_cast<AttnShared*>(smem + 12 * KB_BYTES);
    volatile int* abort_flag = &sh.abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int head = blockIdx.y, q0 = blockIdx.x * AQ;

    // The grid is sized for T because r lives on the device: a CTA whose query rows lie past r
    // leaves before it sets anything up (no barriers, no TMEM).
    grid_dep_wait();
    const int n = clamp_count(rep_cnt, T);
    if (q0 >= n) return;
    if (threadIdx.x == 0) {
        mbar_init(&sh.q_full, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sh.k_full[i], 1); mbar_init(&sh.k_empty[i], 1);
            mbar_init(&sh.v_full[i], 1); mbar_init(&sh.v_empty[i], 1);
            mbar_init(&sh.s_full[i], 1); mbar_init(&sh.s_empty[i], 4);
        }
        mbar_init(&sh.p_full, 4); mbar_init(&sh.p_empty, 1); mbar_init(&sh.o_full, 1);
        sh.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&sh.tmem_base)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const unsigned tmem_base = sh.tmem_base;
    const bool active = true;
    int nkv = (n + AKV - 1) / AKV;
    if (causal) nkv = min(nkv, (int)blockIdx.x + 1);   // keys at or before the tile's last row
    const int nkb = (d_h + BK - 1) / BK;               // 64-element K blocks of the first contraction
    const int v_kb_bytes = d_h * BK * 2;               // one K block (64 keys) of the V^T tile

    if (active && warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            bool ok = true;
            mbar_expect_tx(&sh.q_full, (unsigned)(nkb * KB_BYTES));
            for (int kb = 0; kb < nkb; ++kb) tma_load_3d(&maps.q, &sh.q_full, qs + kb * KB_BYTES, kb * BK, q0, head);
            unsigned kfill = 0, vfill = 0;             // per slot: parity of the number of fills
            int kit = 0;
            for (int pass = 0; pass < 2 && ok; ++pass) {
                for (int j = 0; j < nkv && ok; ++j, ++kit) {
                    const int s = kit & 1;
                    if (!mbar_wait(&sh.k_empty[s], ((kfill >> s) & 1u) ^ 1u, abort_flag, 31)) { ok = false; break; }
                    mbar_expect_tx(&sh.k_full[s], (unsigned)(nkb * KB_BYTES));
                    for (int kb = 0; kb < nkb; ++kb)
                        tma_load_3d(&maps.k, &sh.k_full[s], ks + (s * 2 + kb) * KB_BYTES, kb * BK, j * AKV, head);
                    kfill ^= 1u << s;
                    if (pass == 1) {
                        const int v = j & 1;
                        if (!mbar_wait(&sh.v_empty[v], ((vfill >> v) & 1u) ^ 1u, abort_flag, 32)) { ok = false; break; }
                        mbar_expect_tx(&sh.v_full[v], (unsigned)(2 * v_kb_bytes));
                        for (int u = 0; u < 2; ++u)
                            tma_load_3d(&maps.v, &sh.v_full[v], vs + v * 2 * KB_BYTES + u * v_kb_bytes,
                                        j * AKV + u * BK, 0, head);
                        vfill ^= 1u << v;
                    }
                }
            }
            // every copy has to land before the CTA may exit: a slot's release implies it
            for (int s = 0; s < 2; ++s) {
                if (kit > s) {
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try(&sh.k_empty[s], ((kfill >> s) & 1u) ^ 1u))
                        if (*abort_flag != 0 || global_ns() - t0 > WAIT_LIMIT_NS / 2) { *abort_flag = 33; break; }
                }
                if (nkv > s) {
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try(&sh.v_empty[s], ((vfill >> s) & 1u) ^ 1u))
                        if (*abort_flag != 0 || global_ns() - t0 > WAIT_LIMIT_NS / 2) { *abort_flag = 34; break; }
                }
            }
        }
    } else if (active && warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            bool ok = mbar_wait(&sh.q_full, 0u, abort_flag, 35);
            unsigned kuse = 0, suse = 0;               // parities per slot / buffer
            int kit = 0, sit = 0;
            const unsigned idesc1 = instr_desc(AKV);
            const unsigned idesc2 = instr_desc(d_h);
            // S[buf] = Q K_j^T
            auto issue_s = [&]() {
                const int s = kit & 1, b = sit & 1;
                if (!mbar_wait(&sh.k_full[s], (kuse >> s) & 1u, abort_flag, 36)) { ok = false; return; }
                if (!mbar_wait(&sh.s_empty[b], ((suse >> b) & 1u) ^ 1u, abort_flag, 37)) { ok = false; return; }
                tcgen05_fence_after();
                for (int kb = 0; kb < nkb; ++kb) {
                    const unsigned long long adesc = smem_desc_sw128(smem_u32(qs + kb * KB_BYTES));
                    const unsigned long long bdesc = smem_desc_sw128(smem_u32(ks + (s * 2 + kb) * KB_BYTES));
                    const int steps = min(BK, d_h - kb * BK) / UMMA_K;
                    for (int k = 0; k < steps; ++k)
                        umma_bf16(tmem_base + b * AKV, adesc + 2 * k, bdesc + 2 * k, idesc1, (kb | k) != 0);
                }
                umma_commit(&sh.k_empty[s]);
                umma_commit(&sh.s_full[b]);
                kuse ^= 1u << s; suse ^= 1u << b;
                ++kit; ++sit;
            };
            for (int j = 0; j < nkv && ok; ++j) issue_s();          // pass 1: statistics only
            if (ok) issue_s();                                       // pass 2, tile 0
            unsigned vuse = 0;
            for (int j = 0; j < nkv && ok; ++j) {
                if (j + 1 < nkv) issue_s();                          // keeps one S tile ahead of the softmax
                if (!ok) break;
                const int v = j & 1;
                if (!mbar_wait(&sh.p_full, (unsigned)(j & 1), abort_flag, 38)) { ok = false; break; }
                if (!mbar_wait(&sh.v_full[v], (vuse >> v) & 1u, abort_flag, 39)) { ok = false; break; }
                tcgen05_fence_after();
                for (int u = 0; u < 2; ++u) {                        // O += P V_j
                    const unsigned long long adesc = smem_desc_sw128(smem_u32(ps + u * KB_BYTES));
                    const unsigned long long bdesc = smem_desc_sw128(smem_u32(vs + v * 2 * KB_BYTES + u * v_kb_bytes));
                    for (int k = 0; k < BK / UMMA_K; ++k)
                        umma_bf16(tmem_base + 2 * AKV, adesc + 2 * k, bdesc + 2 * k, idesc2, (j | u | k) != 0);
                }
                umma_commit(&sh.v_empty[v]);
                umma_commit(&sh.p_empty);
                vuse ^= 1u << v;
            }
            if (ok) umma_commit(&sh.o_full);
            else { /* the softmax warps time out on their own */ }
        }
    } else if (active && warp >= 2) {
        // ------------------------------------------------ softmax and output (warps 2..5)
        const int quad = warp & 3;
        const int i = quad * 32 + lane;                // this thread's row of the tile
        const int qrow = q0 + i;                       // position in the representative list
        const unsigned tlane = tmem_base + ((unsigned)(quad * 32) << 16);
        const float sc = 1.4426950408889634f / sqrtf((float)d_h);   // log2(e) / sqrt(d_h)
        float m = -INFINITY, l = 0.f;
        unsigned suse = 0;
        int sit = 0;
        bool ok = true;
        // pass 1: row maximum and sum of exponentials over all key tiles
        for (int j = 0; j < nkv && ok; ++j, ++sit) {
            const int b = sit & 1;
            const bool got = mbar_wait(&sh.s_full[b], (suse >> b) & 1u, abort_flag, 40);
            if (!__all_sync(0xffffffffu, got)) { ok = false; break; }
            tcgen05_fence_after();
            for (int c0 = 0; c0 < AKV; c0 += 32) {
                float v[32];
                tmem_ld32(tlane + b * AKV + c0, v);
                float cm = -INFINITY;
#pragma unroll
                for (int q = 0; q < 32; ++q) {
                    const int col = j * AKV + c0 + q;
                    const bool valid = col < n && (!causal || col <= qrow);
                    v[q] = valid ? v[q] * sc : -INFINITY;
                    cm = fmaxf(cm, v[q]);
                }
                if (cm > -INFINITY) {
                    const float mn = fmaxf(m, cm);
                    float add = 0.f;
#pragma unroll
                    for (int q = 0; q < 32; ++q) add += exp2f(v[q] - mn);
                    l = l * exp2f(m - mn) + add;
                    m = mn;
                }
            }
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.s_empty[b]);
            suse ^= 1u << b;
        }
        // pass 2: P = exp2(S - m) / l as bf16 into shared memory, K-major with the 128-byte swizzle
        const float inv_l = l > 0.f ? 1.0f / l : 0.f;
        for (int j = 0; j < nkv && ok; ++j, ++sit) {
            const int b = sit & 1;
            bool got = mbar_wait(&sh.s_full[b], (suse >> b) & 1u, abort_flag, 41);
            // the previous tile's P has been consumed by its MMAs
            got = got && mbar_wait(&sh.p_empty, (unsigned)((j & 1) ^ 1), abort_flag, 42);
            if (!__all_sync(0xffffffffu, got)) { ok = false; break; }
            tcgen05_fence_after();
            for (int c0 = 0; c0 < AKV; c0 += 32) {
                float v[32];
                tmem_ld32(tlane + b * AKV + c0, v);
                unsigned w[16];
#pragma unroll
                for (int q = 0; q < 32; q += 2) {
                    const int col = j * AKV + c0 + q;
                    const bool v0 = col < n && (!causal || col <= qrow);
                    const bool v1 = col + 1 < n && (!causal || col + 1 <= qrow);
                    const float p0 = v0 ? exp2f(v[q] * sc - m) * inv_l : 0.f;
                    const float p1 = v1 ? exp2f(v[q + 1] * sc - m) * inv_l : 0.f;
                    const __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
                    w[q >> 1] = *reinterpret_cast<const unsigned*>(&pk);
                }
                unsigned char* rowp = ps + (c0 >> 6) * KB_BYTES + i * 128;
                const int cc0 = (c0 & 63) >> 3;        // first 16-byte chunk of these 32 columns
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    *reinterpret_cast<uint4*>(rowp + (((cc0 + q) ^ (i & 7)) << 4)) =
                        make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the MMA reads P through the async proxy
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) { mbar_arrive(&sh.p_full); mbar_arrive(&sh.s_empty[b]); }
            suse ^= 1u << b;
        }
        // output rows of this tile's representatives, at their token positions
        if (ok) {
            const bool got = mbar_wait(&sh.o_full, 0u, abort_flag, 43);
            if (__all_sync(0xffffffffu, got)) {
                tcgen05_fence_after();
                const int tok = qrow < n ? rep_idx[qrow] : -1;
                float* dst = (tok >= 0 && tok < T) ? out + (int64_t)tok * ldo + (int64_t)head * d_h : nullptr;
                for (int c0 = 0; c0 < d_h; c0 += 32) {
                    float v[32];
                    tmem_ld32(tlane + 2 * AKV + c0, v);
                    if (dst != nullptr) {
#pragma unroll
                        for (int q = 0; q < 32; q += 4)
                            if (c0 + q < d_h)
                                *reinterpret_cast<float4*>(dst + c0 + q) = make_float4(v[q], v[q + 1], v[q + 2], v[q + 3]);
                    }
                }
            }
        }
        tcgen05_fence_before();
    }
    __syncthreads();
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
    if (threadIdx.x == 0 && sh.abort_flag != 0) {
        atomicOr(status, ST_TIMEOUT);
        status[2] = 200u + (unsigned)sh.abort_flag;
    }
}

// ---------------------------------------------------------------- expansion (Section 2.3)
// One warp per token: a token outside the set takes its nearest representative's output; a
// token without one (empty set) gets zeros.
__global__ void __launch_bounds__(256)
k_attn_expand(float* __restrict__ out, int64_t ldo, int T, int width, const int32_t* __restrict__ nearest) {
    grid_dep_wait();
    const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (t >= T) return;
    const int s = nearest[t];
    if (s == t) return;
    float4* dst = reinterpret_cast<float4*>(out + (int64_t)t * ldo);
    if (s < 0 || s >= T) {
        for (int v = lane; v < (width >> 2); v += 32) dst[v] = make_float4(0.f, 0.f, 0.f, 0.f);
        return;
    }
    const float4* src = reinterpret_cast<const float4*>(out + (int64_t)s * ldo);
    for (int v = lane; v < (width >> 2); v += 32) dst[v] = __ldcg(src + v);
}

}  // namespace

cudaError_t launch_attention_reps(ada_ctx* ctx, const void* Q, const void* K, const void* V, int T, int h,
                                  int d_h, int64_t ld, const int32_t* rep_idx, const int32_t* rep_cnt,
                                  const int32_t* nearest_idx, float* out, int64_t ldo, int causal,
                                  cudaStream_t s) {
    const int Tp = (T + AKV - 1) / AKV * AKV;
    const size_t n_el = (size_t)h * Tp * d_h;
    const size_t need = 3 * (n_el * 2 + 1024);
    if (ctx->attn_ws == nullptr || ctx->attn_ws_bytes < need) {
        // first use (or a larger problem): the gathered Q_R, K_R and V_R^T live here
        if (ctx->attn_ws != nullptr) { cudaStreamSynchronize(s); cudaFree(ctx->attn_ws); ctx->attn_ws = nullptr; }
        if (cudaMalloc(&ctx->attn_ws, need) != cudaSuccess) { cudaGetLastError(); return cudaErrorMemoryAllocation; }
        ctx->attn_ws_bytes = need;
        cudaError_t e = cudaFuncSetAttribute(k_attn_reps, cudaFuncAttributeMaxDynamicSharedMemorySize, ATT_SMEM);
        if (e != cudaSuccess) return e;
    }
    const size_t stride = (n_el * 2 + 1023) / 1024 * 1024;
    __nv_bfloat16* Qr = reinterpret_cast<__nv_bfloat16*>(ctx->attn_ws);
    __nv_bfloat16* Kr = reinterpret_cast<__nv_bfloat16*>(ctx->attn_ws + stride);
    __nv_bfloat16* Vt = reinterpret_cast<__nv_bfloat16*>(ctx->attn_ws + 2 * stride);
    AttnMaps maps;
    memset(&maps, 0, sizeof(maps));
    if (!make_map(&maps.q, Qr, d_h, Tp, h, d_h, (int64_t)Tp * d_h, AQ) ||
        !make_map(&maps.k, Kr, d_h, Tp, h, d_h, (int64_t)Tp * d_h, AKV) ||
        !make_map(&maps.v, Vt, Tp, d_h, h, Tp, (int64_t)d_h * Tp, d_h))
        return cudaErrorInvalidValue;
    launch_k(ctx, k_attn_gather, dim3(Tp / 32, h), dim3(256), 0, s, (const __nv_bfloat16*)Q,
             (const __nv_bfloat16*)K, (const __nv_bfloat16*)V, T, Tp, h, d_h, ld, rep_idx, rep_cnt, Qr, Kr, Vt,
             ctx->status);
    launch_k(ctx, k_attn_reps, dim3(Tp / AQ, h), dim3(ATT_THREADS), ATT_SMEM, s, maps, T, d_h, h, rep_idx, rep_cnt,
             out, ldo, causal, ctx->status);
    if (nearest_idx != nullptr)
        launch_k(ctx, k_attn_expand, dim3((T + 7) / 8), dim3(256), 0, s, out, ldo, T, h * d_h, nearest_idx);
    return cudaGetLastError();
}

}  // namespace ada
