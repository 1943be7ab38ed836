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
//                   thread-local), P rounded to bf16 into shared memory (two buffers) in the
//                   128-byte swizzled K-major layout, O += P V^T into a third TMEM accumulator.
//                   One pass over the key tiles: probabilities are taken against a per-row
//                   reference maximum that is raised (and the accumulator rescaled, in TMEM) only
//                   when the running maximum has moved by more than 8 powers of two, which after
//                   the first tile is rare; the division by the row sum happens at the output.
//   k_attn_expand   out[t] = out[nearest[t]] for the tokens outside R
// Every wait is bounded (see gram_tc_dev.cuh).
#include "gram_tc_dev.cuh"

namespace ada {

using namespace tc;

// Time stamps for in-kernel timelines (development builds only: -DADA_TRACE): the first 16 query
// tiles of head 0.
#ifdef ADA_TRACE
__device__ unsigned long long g_atrace[16 * 32];
#define ATRACE(slot) do { if (blockIdx.y == 0 && blockIdx.x < 16) g_atrace[blockIdx.x * 32 + (slot)] = tc::global_ns(); } while (0)
#else
#define ATRACE(slot) do { } while (0)
#endif

namespace {

constexpr int AQ = 128;                 // query rows per CTA (TMEM lanes)
constexpr int AKV = 128;                // keys per tile
constexpr int KB_BYTES = 128 * BK * 2;  // one 64-element K block of a 128-row tile: 16 KiB
constexpr int ATT_THREADS = 320;        // TMA producer, MMA issuer, eight softmax warps

struct alignas(16) AttnShared {
    unsigned long long q_full, q_empty, k_full[2], k_empty[2], v_full[2], v_empty[2];
    unsigned long long s_full[2], s_empty[2], p_full[2], p_empty[2], o_full, o_empty;
    unsigned long long x_put[4];             // per 32-row group: the two warps of a row exchange their statistics
    unsigned tmem_base;
    int abort_flag;
    float2 xstat[2][AQ];                     // (m_ref, l) of each warp set, by row
};
// Q (2 K blocks) | K ring 2 x 2 | V^T ring 2 x 2 | P 2 x 2.  The dynamic shared memory is declared
// 1024-byte aligned (the swizzled tiles need it); the kernel checks the address it gets.
constexpr int ATT_SMEM = (2 + 4 + 4 + 4) * KB_BYTES + (int)sizeof(AttnShared);
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
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void tmem_st32(unsigned taddr, const float (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};\n\t"
        "tcgen05.wait::st.sync.aligned;"
        ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
          "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])),
          "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])),
          "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
          "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
          "r"(__float_as_uint(v[15])), "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])),
          "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])), "r"(__float_as_uint(v[20])),
          "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
          "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])),
          "r"(__float_as_uint(v[27])), "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])),
          "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
        : "memory");
}
// The softmax warps run one or two per scheduler with little to hide latency behind, so the
// per-element code is kept to a max, an fma, an ex2, an add and half a convert, in
// independent chains; the mask is applied only on tiles that need one.
// 32 raw scores of one row: (mask,) maximum.  lim: how many of the 32 columns are admissible
// (columns ascend, so both the end of the set and the causal bound cut a suffix)
template <bool MASKED>
__device__ __forceinline__ float tile_max32(unsigned (&r)[32], int lim, float cm) {
    float m0 = cm, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
    for (int q = 0; q < 32; q += 4) {
        if (MASKED) {
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (q + e >= lim) r[q + e] = 0xff800000u;   // -inf
        }
        m0 = fmaxf(m0, __uint_as_float(r[q]));
        m1 = fmaxf(m1, __uint_as_float(r[q + 1]));
        m2 = fmaxf(m2, __uint_as_float(r[q + 2]));
        m3 = fmaxf(m3, __uint_as_float(r[q + 3]));
    }
    return fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
}
// p = 2^(s * sc - mref) for 32 raw scores, as bf16 into the row's 64 bytes of the swizzled P tile;
// returns their sum
__device__ __forceinline__ float exp_store(const unsigned (&r)[32], float sc, float mref, unsigned char* rowp,
                                           int cc0, int row) {
    unsigned w[16];
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
    for (int q = 0; q < 32; q += 4) {
        const float p0 = ex2_approx(fmaf(__uint_as_float(r[q]), sc, -mref));
        const float p1 = ex2_approx(fmaf(__uint_as_float(r[q + 1]), sc, -mref));
        const float p2 = ex2_approx(fmaf(__uint_as_float(r[q + 2]), sc, -mref));
        const float p3 = ex2_approx(fmaf(__uint_as_float(r[q + 3]), sc, -mref));
        s0 += p0; s1 += p1; s2 += p2; s3 += p3;
        const __nv_bfloat162 lo = __floats2bfloat162_rn(p0, p1), hi = __floats2bfloat162_rn(p2, p3);
        w[q >> 1] = *reinterpret_cast<const unsigned*>(&lo);
        w[(q >> 1) + 1] = *reinterpret_cast<const unsigned*>(&hi);
    }
#pragma unroll
    for (int q = 0; q < 4; ++q)
        *reinterpret_cast<uint4*>(rowp + (((cc0 + q) ^ (row & 7)) << 4)) =
            make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
    return (s0 + s1) + (s2 + s3);
}

// How far a row's reference maximum may lag behind its true running maximum (in powers of two)
// before the accumulator is rescaled: the probabilities of a tile are 2^(s - m_ref) <= 2^LAG.
constexpr float ATT_LAG = 8.0f;

__global__ void __launch_bounds__(ATT_THREADS, 1)
k_attn_reps(const __grid_constant__ AttnMaps maps, int T, int d_h, int h,
            const int32_t* __restrict__ rep_idx, const int32_t* __restrict__ rep_cnt,
            float* __restrict__ out, int64_t ldo, int causal, unsigned* __restrict__ status) {
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char* qs = smem;                          // Q tile: nkb K blocks
    unsigned char* ks = smem + 2 * KB_BYTES;           // K ring: 2 slots x 2 K blocks
    unsigned char* vs = smem + 6 * KB_BYTES;           // V^T ring: 2 slots x 2 K blocks of d_h rows
    unsigned char* ps = smem + 10 * KB_BYTES;          // P: 2 buffers x 2 K blocks
    AttnShared& sh = *reinterpret_cast<AttnShared*>(smem + 14 * KB_BYTES);
    volatile int* abort_flag = &sh.abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // Persistent CTAs: the work items are (128 query rows, head) pairs, nq * h of them with
    // nq = ceil(r / 128) known only on the device; CTA c takes items c, c + gridDim.x, ...
    // Barriers, TMEM and the rings live across items (a buffer's uses are counted on, so every
    // wait's parity follows from a running count), and the next item's Q, first keys and first
    // score tiles are under way while the softmax warps still write the previous item's rows.
    grid_dep_wait();
    const int n = clamp_count(rep_cnt, T);
    const int nq = (n + AQ - 1) / AQ;
    const int total = nq * h;
    if ((int)blockIdx.x >= total) return;              // before anything is set up
    if ((smem_u32(smem) & 1023u) != 0u) {              // the tiles would not be where the swizzle assumes
        if (threadIdx.x == 0) { atomicOr(status, ST_TIMEOUT); status[2] = 299u; }
        return;
    }
    if (threadIdx.x == 0) ATRACE(0);
    if (threadIdx.x == 0) {
        mbar_init(&sh.q_full, 1); mbar_init(&sh.q_empty, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sh.k_full[i], 1); mbar_init(&sh.k_empty[i], 1);
            mbar_init(&sh.v_full[i], 1); mbar_init(&sh.v_empty[i], 1);
            mbar_init(&sh.s_full[i], 1); mbar_init(&sh.s_empty[i], 4);
            mbar_init(&sh.p_full[i], 4); mbar_init(&sh.p_empty[i], 1);
        }
        for (int i = 0; i < 4; ++i) mbar_init(&sh.x_put[i], 2);
        mbar_init(&sh.o_full, 1); mbar_init(&sh.o_empty, 8);
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
    if (threadIdx.x == 0) ATRACE(1);
    const int nkv_all = (n + AKV - 1) / AKV;
    const int nkb = (d_h + BK - 1) / BK;               // 64-element K blocks of the first contraction
    const int v_kb_bytes = d_h * BK * 2;               // one K block (64 keys) of the V^T tile
    // Buffer b = j & 1 of every ring serves the key tiles j = b, b + 2, ... of an item; with
    // base[b] uses in the CTA's earlier items, tile j is use number base[b] + (j >> 1).

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            bool ok = true;
            unsigned base[2] = {0u, 0u};
            int k = 0;
            for (int item = blockIdx.x; item < total && ok; item += gridDim.x, ++k) {
                const int qt = item % nq, head = item / nq, q0 = qt * AQ;
                const int nkv = causal ? min(nkv_all, qt + 1) : nkv_all;   // keys at or before the tile's last row
                // the previous item's Q K^T MMAs have read Q
                if (k > 0 && !mbar_wait(&sh.q_empty, (unsigned)(k - 1) & 1u, abort_flag, 30)) { ok = false; break; }
                mbar_expect_tx(&sh.q_full, (unsigned)(nkb * KB_BYTES));
                for (int kb = 0; kb < nkb; ++kb)
                    tma_load_3d(&maps.q, &sh.q_full, qs + kb * KB_BYTES, kb * BK, q0, head);
                for (int j = 0; j < nkv && ok; ++j) {
                    const int s = j & 1;
                    const unsigned prev = ((base[s] + ((unsigned)j >> 1)) & 1u) ^ 1u;
                    if (!mbar_wait(&sh.k_empty[s], prev, abort_flag, 31)) { ok = false; break; }
                    mbar_expect_tx(&sh.k_full[s], (unsigned)(nkb * KB_BYTES));
                    for (int kb = 0; kb < nkb; ++kb)
                        tma_load_3d(&maps.k, &sh.k_full[s], ks + (s * 2 + kb) * KB_BYTES, kb * BK, j * AKV, head);
                    if (!mbar_wait(&sh.v_empty[s], prev, abort_flag, 32)) { ok = false; break; }
                    mbar_expect_tx(&sh.v_full[s], (unsigned)(2 * v_kb_bytes));
                    for (int u = 0; u < 2; ++u)
                        tma_load_3d(&maps.v, &sh.v_full[s], vs + s * 2 * KB_BYTES + u * v_kb_bytes, j * AKV + u * BK,
                                    0, head);
                }
                base[0] += (unsigned)(nkv + 1) >> 1;
                base[1] += (unsigned)nkv >> 1;
            }
            // every copy has to land before the CTA may exit: a slot's last release implies it
            for (int s = 0; s < 2 && ok; ++s) {
                if (base[s] == 0u) continue;
                const unsigned ph = (base[s] - 1u) & 1u;
                const unsigned long long t0 = global_ns();
                while (!(mbar_try(&sh.k_empty[s], ph) && mbar_try(&sh.v_empty[s], ph)))
                    if (*abort_flag != 0 || global_ns() - t0 > WAIT_LIMIT_NS / 2) { *abort_flag = 33; break; }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            bool ok = true;
            unsigned base[2] = {0u, 0u};
            const unsigned idesc1 = instr_desc(AKV);
            const unsigned idesc2 = instr_desc(d_h);
            int k = 0;
            for (int item = blockIdx.x; item < total && ok; item += gridDim.x, ++k) {
                const int qt = item % nq;
                const int nkv = causal ? min(nkv_all, qt + 1) : nkv_all;
                if (!mbar_wait(&sh.q_full, (unsigned)k & 1u, abort_flag, 35)) { ok = false; break; }
                // S[j & 1] = Q K_j^T
                auto issue_s = [&](int j) {
                    const int b = j & 1;
                    const unsigned ph = (base[b] + ((unsigned)j >> 1)) & 1u;
                    if (!mbar_wait(&sh.k_full[b], ph, abort_flag, 36)) { ok = false; return; }
                    if (!mbar_wait(&sh.s_empty[b], ph ^ 1u, abort_flag, 37)) { ok = false; return; }
                    tcgen05_fence_after();
                    for (int kb = 0; kb < nkb; ++kb) {
                        const unsigned long long adesc = smem_desc_sw128(smem_u32(qs + kb * KB_BYTES));
                        const unsigned long long bdesc = smem_desc_sw128(smem_u32(ks + (b * 2 + kb) * KB_BYTES));
                        const int steps = min(BK, d_h - kb * BK) / UMMA_K;
                        for (int q = 0; q < steps; ++q)
                            umma_bf16(tmem_base + b * AKV, adesc + 2 * q, bdesc + 2 * q, idesc1, (kb | q) != 0);
                    }
                    umma_commit(&sh.k_empty[b]);
                    umma_commit(&sh.s_full[b]);
                    if (j == nkv - 1) umma_commit(&sh.q_empty);          // Q may be replaced
                };
                issue_s(0);
                for (int j = 0; j < nkv && ok; ++j) {
                    if (j + 1 < nkv) issue_s(j + 1);                     // each warp set one score tile ahead
                    if (!ok) break;
                    const int b = j & 1;
                    const unsigned ph = (base[b] + ((unsigned)j >> 1)) & 1u;
                    if (!mbar_wait(&sh.p_full[b], ph, abort_flag, 38)) { ok = false; break; }
                    if (!mbar_wait(&sh.v_full[b], ph, abort_flag, 39)) { ok = false; break; }
                    // the accumulators are overwritten: the previous item's rows have been read out
                    if (j == 0 && k > 0 && !mbar_wait(&sh.o_empty, (unsigned)(k - 1) & 1u, abort_flag, 47)) { ok = false; break; }
                    tcgen05_fence_after();
                    for (int u = 0; u < 2; ++u) {                        // O[j & 1] += P_j V_j
                        const unsigned long long adesc = smem_desc_sw128(smem_u32(ps + (b * 2 + u) * KB_BYTES));
                        const unsigned long long bdesc = smem_desc_sw128(smem_u32(vs + b * 2 * KB_BYTES + u * v_kb_bytes));
                        for (int q = 0; q < BK / UMMA_K; ++q)
                            umma_bf16(tmem_base + (2 + b) * AKV, adesc + 2 * q, bdesc + 2 * q, idesc2,
                                      ((j >> 1) | u | q) != 0);
                    }
                    umma_commit(&sh.v_empty[b]);
                    umma_commit(&sh.p_empty[b]);
                }
                if (ok) umma_commit(&sh.o_full);
                base[0] += (unsigned)(nkv + 1) >> 1;
                base[1] += (unsigned)nkv >> 1;
            }
            /* on failure the softmax warps time out on their own */
        }
    } else {
        // ------------------------------------------------ softmax and output (warps 2..9)
        // One pass over the key tiles.  A row keeps a reference maximum m_ref that is raised only
        // when the running maximum exceeds it by more than ATT_LAG; the tile's probabilities are
        // 2^(s - m_ref) (at most 2^ATT_LAG, unnormalised), their sum goes into l, and O and l are
        // rescaled by 2^(m_old - m_new) on the rare tile where m_ref moves.  O / l does not
        // depend on m_ref.
        // Two sets of four warps (a warp reaches the TMEM lanes 32 (warp % 4) ..) take ALTERNATE
        // key tiles: warps 2..5 the even ones, warps 6..9 the odd ones, each set with its own score
        // buffer, P buffer, accumulator and (m_ref, l), so that one set's exponentials overlap the
        // other's loads and maxima with nothing exchanged per tile.  The two partial results are
        // merged at the output like two halves of any split softmax.
        const int quad = warp & 3;
        const int half = (warp - 2) >> 2;              // = parity of this set's key tiles = its buffers
        const int i = quad * 32 + lane;                // this thread's row of the tile
        const unsigned tlane = tmem_base + ((unsigned)(quad * 32) << 16);
        const unsigned t_s = tlane + half * AKV, t_o = tlane + (2 + half) * AKV;
        const float sc = 1.4426950408889634f / sqrtf((float)d_h);   // log2(e) / sqrt(d_h)
        bool ok = true;
        unsigned base = 0u;                            // uses of this set's buffers in earlier items
        int k = 0;
        for (int item = blockIdx.x; item < total && ok; item += gridDim.x, ++k) {
            const int qt = item % nq, head = item / nq, q0 = qt * AQ;
            const int nkv = causal ? min(nkv_all, qt + 1) : nkv_all;
            const int qrow = q0 + i;                                    // position in the representative list
            const int lim_abs = min(n, causal ? qrow + 1 : n);          // admissible keys of this row: [0, lim_abs)
            float m_ref = -INFINITY, l = 0.f;
            for (int j = half; j < nkv && ok; j += 2) {
                const unsigned ph = (base + ((unsigned)j >> 1)) & 1u;
                bool got = mbar_wait(&sh.s_full[half], ph, abort_flag, 40);
                if (!__all_sync(0xffffffffu, got)) { ok = false; break; }
                if (k == 0 && j == 0 && threadIdx.x == 64) ATRACE(2);
                if (k == 0 && j == 2 && threadIdx.x == 64) ATRACE(20);
                tcgen05_fence_after();
                // columns past r, and under the causal mask the keys after the query, count as -inf
                const int c0 = j * AKV;
                const bool masked = (c0 + AKV > n) || (causal && c0 + AKV - 1 > q0);
                // sweep 1: the row maximum of the raw scores
                float cm = -INFINITY;
#pragma unroll
                for (int c = 0; c < AKV; c += 64) {
                    unsigned r0[32], r1[32];
                    tmem_ld32_issue(t_s + c, r0);
                    tmem_ld32_issue(t_s + c + 32, r1);
                    tmem_ld_wait(r0); tmem_ld_wait(r1);
                    if (masked) {
                        cm = tile_max32<true>(r0, lim_abs - (c0 + c), cm);
                        cm = tile_max32<true>(r1, lim_abs - (c0 + c + 32), cm);
                    } else {
                        cm = tile_max32<false>(r0, 32, cm);
                        cm = tile_max32<false>(r1, 32, cm);
                    }
                }
                cm *= sc;                                          // sc > 0: the maximum of the scaled scores
                if (k == 0 && j == 2 && threadIdx.x == 64) ATRACE(21);
                const float m_new = fmaxf(m_ref, cm);
                const bool raise = m_new > m_ref + ATT_LAG;        // also true for the first finite maximum
                // the MMAs of this set's previous tile have retired: its P buffer is free and nothing
                // is adding to its accumulator
                got = mbar_wait(&sh.p_empty[half], ph ^ 1u, abort_flag, 42);
                if (!__all_sync(0xffffffffu, got)) { ok = false; break; }
                if (j < 2) {
                    m_ref = m_new;                                 // nothing accumulated yet
                } else if (__any_sync(0xffffffffu, raise)) {
                    tcgen05_fence_after();
                    const float f = raise ? ex2_approx(m_ref - m_new) : 1.0f;   // 0 for a row without a finite score so far
                    for (int o0 = 0; o0 < d_h; o0 += 32) {
                        float v[32];
                        tmem_ld32(t_o + o0, v);
#pragma unroll
                        for (int q = 0; q < 32; ++q) v[q] *= f;
                        tmem_st32(t_o + o0, v);
                    }
                    l *= f;
                    if (raise) m_ref = m_new;
                }
                if (k == 0 && j == 2 && threadIdx.x == 64) ATRACE(22);
                // sweep 2: the probabilities
                const float mref = m_ref > -INFINITY ? m_ref : 0.f;   // all scores -inf so far: every p is 0
                unsigned char* prow = ps + half * 2 * KB_BYTES + i * 128;
                float sum = 0.f;
#pragma unroll
                for (int c = 0; c < AKV; c += 64) {
                    unsigned r0[32], r1[32];
                    tmem_ld32_issue(t_s + c, r0);
                    tmem_ld32_issue(t_s + c + 32, r1);
                    tmem_ld_wait(r0); tmem_ld_wait(r1);
                    if (masked) {
                        tile_max32<true>(r0, lim_abs - (c0 + c), 0.f);
                        tile_max32<true>(r1, lim_abs - (c0 + c + 32), 0.f);
                    }
                    sum += exp_store(r0, sc, mref, prow + (c >> 6) * KB_BYTES, 0, i);
                    sum += exp_store(r1, sc, mref, prow + (c >> 6) * KB_BYTES, 4, i);
                }
                l += sum;
                if (k == 0 && j == 2 && threadIdx.x == 64) ATRACE(23);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the MMA reads P through the async proxy
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) { mbar_arrive(&sh.s_empty[half]); mbar_arrive(&sh.p_full[half]); }
                if (k == 0 && threadIdx.x == 64) ATRACE(3 + min(j, 12));
            }
            if (!ok) break;
            base += (half == 0) ? (unsigned)(nkv + 1) >> 1 : (unsigned)nkv >> 1;
            // output rows of this tile's representatives, at their token positions
            bool got = mbar_wait(&sh.o_full, (unsigned)k & 1u, abort_flag, 43);
            // (the statistics' slots are reused: everybody is done with the previous item's)
            if (k > 0) got = got && mbar_wait(&sh.o_empty, (unsigned)(k - 1) & 1u, abort_flag, 48);
            if (!__all_sync(0xffffffffu, got)) { ok = false; break; }
            if (k == 0 && threadIdx.x == 64) ATRACE(16);
            tcgen05_fence_after();
            sh.xstat[half][i] = make_float2(m_ref, l);
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.x_put[quad]);
            got = mbar_wait(&sh.x_put[quad], (unsigned)k & 1u, abort_flag, 45);
            if (!__all_sync(0xffffffffu, got)) { ok = false; break; }
            {
                const float2 other = sh.xstat[half ^ 1][i];
                const float m = fmaxf(m_ref, other.x);
                const float f_own = m_ref > -INFINITY ? ex2_approx(m_ref - m) : 0.f;
                const float f_oth = other.x > -INFINITY ? ex2_approx(other.x - m) : 0.f;
                const float lt = l * f_own + other.y * f_oth;
                const float inv_l = lt > 0.f ? 1.0f / lt : 0.f;
                const float fa = (half == 0 ? f_own : f_oth) * inv_l;      // factor of the even tiles' accumulator
                const float fb = (half == 0 ? f_oth : f_own) * inv_l;
                const bool use_b = nkv > 1;                                  // was the odd accumulator written for this item
                const int tok = qrow < n ? rep_idx[qrow] : -1;
                float* dst = (tok >= 0 && tok < T) ? out + (int64_t)tok * ldo + (int64_t)head * d_h : nullptr;
                // Rows leave through this set's own (now idle) P buffer: a thread owns a row, so its
                // 32 columns go to shared memory (16-byte pieces permuted by row, free of bank
                // conflicts both ways) and the warp then writes them out four rows at a time,
                // 128 contiguous bytes per row, instead of 32 scattered 16-byte pieces per store.
                unsigned char* stg = ps + half * 2 * KB_BYTES + quad * 8192;
                const unsigned long long dst_bits = reinterpret_cast<unsigned long long>(dst);
                int ci = 0;
                for (int o0 = half * 32; o0 < d_h; o0 += 64, ++ci) {
                    float va[32], vb[32];
                    tmem_ld32(tlane + 2 * AKV + o0, va);
                    if (use_b) tmem_ld32(tlane + 3 * AKV + o0, vb);
#pragma unroll
                    for (int q = 0; q < 32; q += 4) {
                        float4 w = make_float4(va[q] * fa, va[q + 1] * fa, va[q + 2] * fa, va[q + 3] * fa);
                        if (use_b) {
                            w.x = fmaf(vb[q], fb, w.x); w.y = fmaf(vb[q + 1], fb, w.y);
                            w.z = fmaf(vb[q + 2], fb, w.z); w.w = fmaf(vb[q + 3], fb, w.w);
                        }
                        *reinterpret_cast<float4*>(stg + ci * 4096 + lane * 128 + ((((q >> 2) ^ lane) & 7) << 4)) = w;
                    }
                }
                __syncwarp();
                ci = 0;
                for (int o0 = half * 32; o0 < d_h; o0 += 64, ++ci) {
#pragma unroll
                    for (int it = 0; it < 8; ++it) {
                        const int r = it * 4 + (lane >> 3), pc = lane & 7;
                        const float4 w = *reinterpret_cast<const float4*>(stg + ci * 4096 + r * 128 + (((pc ^ r) & 7) << 4));
                        const unsigned lo = __shfl_sync(0xffffffffu, (unsigned)dst_bits, r);
                        const unsigned hi = __shfl_sync(0xffffffffu, (unsigned)(dst_bits >> 32), r);
                        float* drow = reinterpret_cast<float*>(((unsigned long long)hi << 32) | lo);
                        if (drow != nullptr && o0 + pc * 4 < d_h) *reinterpret_cast<float4*>(drow + o0 + pc * 4) = w;
                    }
                }
                __syncwarp();
            }
            // the accumulators (and the statistics' slots) may be reused
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.o_empty);
            if (k == 0 && threadIdx.x == 64) ATRACE(18);
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
    if (threadIdx.x == 0) ATRACE(17);
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
    // persistent CTAs, at most one per SM; r (hence the number of work items) lives on the device
    const int n_items_max = (Tp / AQ) * h;
    launch_k(ctx, k_attn_reps, dim3(n_items_max < ctx->sm_count ? n_items_max : ctx->sm_count), dim3(ATT_THREADS),
             ATT_SMEM, s, maps, T, d_h, h, rep_idx, rep_cnt, out, ldo, causal, ctx->status);
    if (nearest_idx != nullptr)
        launch_k(ctx, k_attn_expand, dim3((T + 7) / 8), dim3(256), 0, s, out, ldo, T, h * d_h, nearest_idx);
    return cudaGetLastError();
}

}  // namespace ada

#ifdef ADA_TRACE
extern "C" int ada_trace_read_attn(unsigned long long* host, int clear) {
    if (cudaMemcpyFromSymbol(host, ada::g_atrace, sizeof(ada::g_atrace)) != cudaSuccess) return 1;
    if (clear) {
        static unsigned long long zeros[16 * 32];
        if (cudaMemcpyToSymbol(ada::g_atrace, zeros, sizeof(zeros)) != cudaSuccess) return 2;
    }
    return 0;
}
#endif
