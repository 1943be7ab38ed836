// Device-side building blocks shared by the tcgen05 Gram kernels: tile constants, the
// shared-memory control block, PTX wrappers (mbarrier, TMA, tcgen05), descriptors.
#pragma once

#include <cuda.h>
#include <string.h>

#include "common.cuh"

namespace ada {
namespace tc {


static constexpr int BM = 128;          // accumulator rows per tile (TMEM lanes)
static constexpr int BN = 256;          // accumulator columns per tile
static constexpr int BK = 64;           // bf16 elements per K block = one 128-byte swizzle row
static constexpr int MAX_STAGES = 9;
static constexpr int RING_BYTES = 216 * 1024;               // TMA ring: 4 stages of a 256-wide tile ... 9 of a 64-wide one
static constexpr int UMMA_K = 16;
static constexpr int A_BYTES = BM * BK * 2;                 // 16 KiB
static constexpr int BOX_N = 64;                            // B rows per TMA box
static constexpr int BOX_BYTES = BOX_N * BK * 2;            // 8 KiB
static constexpr int NORM_WARPS = 8;
static constexpr int NUM_THREADS = 192 + 32 * NORM_WARPS;   // producer, MMA, 4 epilogue warps, norm warps
static constexpr int TMEM_COLS = 512;
static constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;   // 2 s

// one output tile: `ncols` (multiple of 16, <= 256) columns from col0 of the 128-row tile at row0
struct Piece {
    int b, row0, col0, ncols, n, m;
};

struct alignas(16) Shared {
    unsigned long long full[MAX_STAGES];
    unsigned long long empty[MAX_STAGES];
    unsigned long long tmem_full[2];
    unsigned long long tmem_empty[2];
    unsigned long long drain;
    unsigned tmem_base;
    int abort_flag;
    int tiles0, tiles1, par0, par1;
    // per epilogue warp, so that staging needs no barrier across warps
    alignas(16) float col_scale[4][BN];
    alignas(16) int col_token[4][BN];
};
static constexpr int SMEM_BYTES = RING_BYTES + (int)sizeof(Shared) + 1024;   // +1024: alignment slack
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");

// ---------------------------------------------------------------- PTX wrappers
static __device__ __forceinline__ unsigned smem_u32(const void* p) {
    return static_cast<unsigned>(__cvta_generic_to_shared(p));
}
static __device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
static __device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
                 "r"(bytes)
                 : "memory");
}
static __device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
static __device__ __forceinline__ bool mbar_try(unsigned long long* bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// non-blocking form: try_wait may suspend the thread for a while before it reports failure
static __device__ __forceinline__ bool mbar_test(unsigned long long* bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
static __device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait.  Returns false when the CTA is aborting (this or another wait ran out).
// try_wait itself suspends the thread for a while before it reports failure, so the wall
// clock (a slow special register) is consulted only once per 256 failed polls.
static __device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned parity,
                                          volatile int* abort_flag, int where) {
    unsigned polls = 0;
    unsigned long long t0 = 0;
    while (!mbar_try(bar, parity)) {
        if ((++polls & 255u) == 0) {
            if (*abort_flag != 0) return false;
            const unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > WAIT_LIMIT_NS) {
                *abort_flag = where;
                return false;
            }
        }
    }
    return true;
}
static __device__ __forceinline__ void tma_load_3d(const CUtensorMap* map, unsigned long long* bar,
                                            void* dst, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<unsigned long long>(map)), "r"(smem_u32(bar)),
          "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
static __device__ __forceinline__ void tcgen05_fence_before() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
static __device__ __forceinline__ void tcgen05_fence_after() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
static __device__ __forceinline__ void umma_commit(unsigned long long* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(smem_u32(bar))
                 : "memory");
}
static __device__ __forceinline__ void umma_bf16(unsigned tmem_d, unsigned long long adesc,
                                          unsigned long long bdesc, unsigned idesc,
                                          unsigned accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
static __device__ __forceinline__ void tmem_ld32(unsigned taddr, float (&v)[32]) {
    unsigned r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n\t"
        // the wait sits in the same statement so that no use of the registers can be
        // scheduled ahead of it
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
          "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
          "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]),
          "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]),
          "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// The same load as two statements.  After tmem_ld32_issue the registers are undefined; the
// wait takes them as in/out operands, so every use in the code that follows depends on it.
static __device__ __forceinline__ void tmem_ld32_issue(unsigned taddr, unsigned (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
          "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
          "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]),
          "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]),
          "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
static __device__ __forceinline__ void tmem_ld_wait(unsigned (&r)[32]) {
    asm volatile(
        "tcgen05.wait::ld.sync.aligned;"
        : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]),
          "+r"(r[7]), "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]),
          "+r"(r[14]), "+r"(r[15]), "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]),
          "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]), "+r"(r[25]),
          "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
        :
        : "memory");
}

// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes wide and
// stored with the 128-byte swizzle: 8-row groups are 1024 bytes apart (stride byte offset),
// the leading byte offset is unused for swizzled K-major tiles, descriptor version 1.
static __device__ __forceinline__ unsigned long long smem_desc_sw128(unsigned addr) {
    unsigned long long d = 0;
    d |= (unsigned long long)((addr & 0x3FFFFu) >> 4);        // start address, 16-byte units
    d |= (unsigned long long)1 << 16;                         // leading byte offset (ignored)
    d |= (unsigned long long)(1024 >> 4) << 32;               // stride byte offset
    d |= (unsigned long long)1 << 46;                         // descriptor version (sm_100)
    d |= (unsigned long long)2 << 61;                         // layout: 128-byte swizzle
    return d;
}
// Instruction descriptor: D = fp32, A = B = bf16, both K-major, M = 128, N = n.
static __device__ __forceinline__ unsigned instr_desc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((unsigned)(n >> 3) << 17) | ((unsigned)(BM >> 4) << 24);
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) ==
                cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

// 3-D map over a stack of K-major bf16 matrices: (k, row, sequence).
static inline bool make_map(CUtensorMap* map, const void* base, int d, int rows, int B, int64_t ld,
              int64_t batch, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)rows, (cuuint64_t)B};
    // the stride of the last dimension is unused when B == 1 but must still be legal
    const cuuint64_t strides[2] = {(cuuint64_t)ld * 2, (cuuint64_t)(B > 1 ? batch : (int64_t)rows * ld) * 2};
    const cuuint32_t box[3] = {(cuuint32_t)BK, (cuuint32_t)box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box,
              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


// ---------------------------------------------------------------- in-launch row norms
// bf16 pairs are the halves of 32-bit words; a bf16 is the upper half of an fp32
static __device__ __forceinline__ float sumsq_bf16x8(const uint4& v) {
    float s = 0.f;
    const unsigned w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xffff0000u);
        s = fmaf(lo, lo, s);
        s = fmaf(hi, hi, s);
    }
    return s;
}
// Executed by the norm warps of every CTA: warp `w` of `nw` takes rows w, w+nw, ...; when a
// warp has stored its last row it bumps the counter, so counter == nw means "all rows done".
static __device__ __forceinline__ void norm_rows(const NormJob& job, int w, int nw, int lane,
                                                 unsigned* counter, unsigned* status) {
    const int nvec = job.d >> 3;
    const __nv_bfloat16* X = reinterpret_cast<const __nv_bfloat16*>(job.X);
    for (int64_t row = w; row < job.n_rows; row += nw) {
        const int64_t off = job.rows_per_seq > 0
            ? (row / job.rows_per_seq) * job.batch + (row % job.rows_per_seq) * job.ldx
            : row * job.ldx;
        const uint4* src = reinterpret_cast<const uint4*>(X + off);
        // sixteen (then eight) independent 128-bit loads in flight per lane: these few warps
        // have to cover the memory latency that a dedicated kernel would hide with occupancy
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
        int v = lane;
        for (; v + 480 < nvec; v += 512) {
            uint4 x[16];
#pragma unroll
            for (int q = 0; q < 16; ++q) x[q] = __ldg(src + v + 32 * q);
#pragma unroll
            for (int q = 0; q < 16; q += 4) {
                s0 += sumsq_bf16x8(x[q]); s1 += sumsq_bf16x8(x[q + 1]);
                s2 += sumsq_bf16x8(x[q + 2]); s3 += sumsq_bf16x8(x[q + 3]);
            }
        }
        for (; v + 224 < nvec; v += 256) {
            uint4 x[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) x[q] = __ldg(src + v + 32 * q);
#pragma unroll
            for (int q = 0; q < 8; q += 4) {
                s0 += sumsq_bf16x8(x[q]); s1 += sumsq_bf16x8(x[q + 1]);
                s2 += sumsq_bf16x8(x[q + 2]); s3 += sumsq_bf16x8(x[q + 3]);
            }
        }
        for (; v < nvec; v += 32) s0 += sumsq_bf16x8(__ldg(src + v));
        float ss = (s0 + s1) + (s2 + s3);
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
        if (lane == 0) job.inv_norm[row] = inv;
    }
    __threadfence();
    __syncwarp();
    if (lane == 0) atomicAdd(counter, 1u);
}
// Bounded, warp-uniform wait until a global counter reaches `target`.
static __device__ __forceinline__ bool wait_counter(const unsigned* counter, unsigned target, int lane,
                                                    volatile int* abort_flag, int where,
                                                    unsigned long long limit_ns = WAIT_LIMIT_NS) {
    int good = 1;
    if (lane == 0) {
        const unsigned long long t0 = global_ns();
        unsigned seen;
        while (true) {
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
            if (seen >= target) break;
            if (*abort_flag != 0) { good = 0; break; }
            if (global_ns() - t0 > limit_ns) { *abort_flag = where; good = 0; break; }
            __nanosleep(64);
        }
    }
    return __shfl_sync(0xffffffffu, good, 0) != 0;
}

// ---------------------------------------------------------------- in-launch gather (cascade step)
// bounded wait of ONE thread until a global counter reaches `target`
static __device__ __forceinline__ bool wait_counter_1(const unsigned* counter, unsigned target,
                                               volatile int* abort_flag, int where) {
    const unsigned long long t0 = global_ns();
    unsigned seen;
    while (true) {
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
        if (seen >= target) return true;
        if (*abort_flag != 0) return false;
        if (global_ns() - t0 > WAIT_LIMIT_NS) { *abort_flag = where; return false; }
        __nanosleep(64);
    }
}

// Algorithm 1 lines 1-2, by the helper warps of every CTA (warp `g` of `nw`): entry i of
// sequence b is checked (in range, strictly above entry i-1), role[token] = i + 1, the raw row
// goes to Xrep[b, i] and its inverse norm to inv_rep[b, i]; a rejected entry gets inverse norm
// 0 (its column then counts for nothing) and raises the status.  Ends with one arrival per warp
// on `counter`.
// one warp: copy a row of nvec 16-byte vectors, return its sum of squares (all lanes)
static __device__ __forceinline__ float copy_row_sumsq(const uint4* __restrict__ src, uint4* __restrict__ dst,
                                                       int nvec, int lane) {
    float ss = 0.f;
    int v = lane;
    for (; v + 480 < nvec; v += 512) {            // sixteen loads in flight per lane
        uint4 x[16];
#pragma unroll
        for (int q = 0; q < 16; ++q) x[q] = __ldg(src + v + 32 * q);
#pragma unroll
        for (int q = 0; q < 16; ++q) { ss += sumsq_bf16x8(x[q]); dst[v + 32 * q] = x[q]; }
    }
    for (; v < nvec; v += 32) {
        const uint4 x = __ldg(src + v);
        ss += sumsq_bf16x8(x);
        dst[v] = x;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    return ss;
}

// `compact`: also Algorithm 1 line 6's row set as a matrix of its own.  Line 6 builds the
// cross-Gram from the (T - r) tokens OUTSIDE the inherited set; when the set is large, streaming
// all T rows and masking the inherited ones wastes r/T of the loads and MMAs, so the rows
// between consecutive inherited tokens are copied, in order, to Xnon (row t goes to t minus the
// number of inherited tokens before it), with their token index in non_tok and 1/||x_t|| in
// inv_norm.  A warp takes one gap between two list entries at a time.
static __device__ __forceinline__ void gather_rows(const GatherJob& gj, int g, int nw, int lane,
                                            unsigned* counter, unsigned* status, bool compact) {
    const __nv_bfloat16* X = reinterpret_cast<const __nv_bfloat16*>(gj.X);
    __nv_bfloat16* Xrep = reinterpret_cast<__nv_bfloat16*>(gj.Xrep);
    __nv_bfloat16* Xnon = reinterpret_cast<__nv_bfloat16*>(gj.Xnon);
    const int nvec = gj.d >> 3;
    int b = 0;
    int64_t item = g;
    // this warp's first entry is most often entry g of sequence 0: fetch it (and its
    // predecessor) beside the count instead of after it
    int32_t first_idx = 0, first_prev = -1;
    if (g < gj.T) {
        first_idx = __ldg(gj.rep_in + g);
        if (g > 0) first_prev = __ldg(gj.rep_in + g - 1);
    }
    while (b < gj.B) {
        int cnt = gj.rep_in_cnt[b];
        if (cnt < 0 || cnt > gj.T) {
            if (g == 0 && lane == 0) atomicOr(status, ST_BAD_COUNT);
            cnt = cnt < 0 ? 0 : gj.T;
        }
        if (g == 0 && lane == 0) gj.r_eff[b] = cnt;
        const int n_items = compact ? 2 * cnt + 1 : cnt;     // list entries, then the gaps around them
        if (item >= n_items) { item -= n_items; ++b; continue; }
        const int i = (int)item;
        item += nw;                                   // this warp's next item (maybe in a later sequence)
        const int32_t* list = gj.rep_in + (int64_t)b * gj.T;
        if (i >= cnt) {
            // gap number gp: the tokens after entry gp - 1 and before entry gp
            const int gp = i - cnt;
            int lo = gp > 0 ? list[gp - 1] + 1 : 0;
            int hi = gp < cnt ? list[gp] : gj.T;
            lo = max(lo, 0); hi = min(hi, gj.T);      // (a bad list is reported by the entries' check)
            for (int t = lo; t < hi; ++t) {
                const int dstrow = t - gp;
                if (dstrow < 0 || dstrow >= gj.T) continue;
                const uint4* src = reinterpret_cast<const uint4*>(X + (int64_t)b * gj.xb + (int64_t)t * gj.ldx);
                uint4* dst = reinterpret_cast<uint4*>(Xnon + ((int64_t)b * gj.T + dstrow) * (int64_t)gj.d);
                const float ss = copy_row_sumsq(src, dst, nvec, lane);
                if (lane == 0) {
                    float inv = 0.f;
                    if (!(ss <= 3.0e38f)) atomicOr(status, ST_NONFINITE);
                    else if (ss > 0.f) inv = 1.0f / sqrtf(ss);
                    else atomicAdd(status + 1, 1u);
                    gj.inv_norm[(int64_t)b * gj.T + t] = inv;
                    gj.non_tok[(int64_t)b * gj.T + dstrow] = t;
                }
            }
            continue;
        }
        const bool spec = b == 0 && i == g;
        const int32_t idx = spec ? first_idx : list[i];
        bool ok = idx >= 0 && idx < gj.T;
        if (ok && i > 0) ok = (spec ? first_prev : list[i - 1]) < idx;
        const int64_t prow = (int64_t)b * gj.T + i;
        if (!ok) {
            if (lane == 0) { atomicOr(status, ST_BAD_INDEX); gj.inv_rep[prow] = 0.f; }
            continue;
        }
        const uint4* src = reinterpret_cast<const uint4*>(X + (int64_t)b * gj.xb + (int64_t)idx * gj.ldx);
        uint4* dst = reinterpret_cast<uint4*>(Xrep + prow * (int64_t)gj.d);
        const float ss = copy_row_sumsq(src, dst, nvec, lane);
        if (lane == 0) {
            gj.inv_rep[prow] = (ss <= 3.0e38f && ss > 0.f) ? 1.0f / sqrtf(ss) : 0.f;
            gj.role[(int64_t)b * gj.T + idx] = i + 1;
        }
    }
    // the rows just written are read by TMA (async proxy) from other CTAs
    asm volatile("fence.proxy.async.global;" ::: "memory");
    __threadfence();
    __syncwarp();
    if (lane == 0) atomicAdd(counter, 1u);
}

}  // namespace tc
}  // namespace ada
