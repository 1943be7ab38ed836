// bf16 masked-Gram kernel for sm_100a: TMA -> shared memory -> tcgen05.mma -> TMEM,
// with the selection epilogue (1/(|a_i||b_j|) scaling, |.|, admissibility mask, row
// maximum) run straight out of TMEM, so that no Gram tile ever reaches HBM.
//
// Computes, per sequence, out[i] = max_j |a_i . b_j| * inv_a[i] * inv_b[j] over the
// admissible columns j (Definition 1; Algorithm 1 lines 3-4 and 7-8).  Both operands
// are row-major (K-major) bf16 matrices, so G = A B^T needs no transpose.
//
// One persistent CTA per SM, 192 threads:
//   warp 0      TMA producer: one lane issues cp.async.bulk.tensor loads of a 128 x 64
//               A box and a 256 x 64 B box per K block into a 4-stage ring
//               (128-byte swizzle, completion on an mbarrier)
//   warp 1      MMA issuer: one lane issues four tcgen05.mma (M=128, N<=256, K=16) per
//               K block; tcgen05.commit releases the ring stage, and after the last K
//               block hands the accumulator to the epilogue.  Owns the TMEM allocation
//               (512 columns = two 128 x 256 fp32 accumulators, so the epilogue of
//               tile i overlaps the main loop of tile i+1)
//   warps 2..5  epilogue: tcgen05.ld 32 lanes x 32 columns at a time (one accumulator
//               row per thread, so the row maximum is thread-local), then one
//               atomicMax per row and tile on the IEEE bit pattern (values are >= 0).
// Every wait is bounded: when a limit expires the CTA raises the context's TIMEOUT
// status, drains its own outstanding copies and MMAs (again bounded), frees its TMEM
// and returns.
#include <cuda.h>

#include "common.cuh"

namespace ada {

namespace {

constexpr int BM = 128;          // accumulator rows per tile (TMEM lanes)
constexpr int BN = 256;          // accumulator columns per tile
constexpr int BK = 64;           // bf16 elements per K block = one 128-byte swizzle row
constexpr int STAGES = 4;
constexpr int UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2;                 // 16 KiB
constexpr int B_BYTES = BN * BK * 2;                 // 32 KiB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int NUM_THREADS = 192;
constexpr int TMEM_COLS = 512;
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;   // 2 s

struct alignas(16) Shared {
    unsigned long long full[STAGES];
    unsigned long long empty[STAGES];
    unsigned long long tmem_full[2];
    unsigned long long tmem_empty[2];
    unsigned long long drain;
    unsigned tmem_base;
    int abort_flag;
    // per epilogue warp, so that staging needs no barrier across warps
    alignas(16) float col_scale[4][BN];
    alignas(16) int col_token[4][BN];
};
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + (int)sizeof(Shared) + 1024;   // +1024: alignment slack

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ unsigned smem_u32(const void* p) {
    return static_cast<unsigned>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
                 "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try(unsigned long long* bar, unsigned parity) {
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
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait.  Returns false when the CTA is aborting (this or another wait ran out).
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned parity,
                                          volatile int* abort_flag, int where) {
    if (mbar_try(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    unsigned polls = 0;
    while (true) {
        if (mbar_try(bar, parity)) return true;
        if (*abort_flag != 0) return false;
        if ((++polls & 63u) == 0 && global_ns() - t0 > WAIT_LIMIT_NS) {
            *abort_flag = where;
            return false;
        }
    }
}
__device__ __forceinline__ void tma_load_3d(const CUtensorMap* map, unsigned long long* bar,
                                            void* dst, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<unsigned long long>(map)), "r"(smem_u32(bar)),
          "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void tcgen05_fence_before() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tcgen05_fence_after() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void umma_commit(unsigned long long* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void umma_bf16(unsigned tmem_d, unsigned long long adesc,
                                          unsigned long long bdesc, unsigned idesc,
                                          unsigned accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tmem_ld32(unsigned taddr, float (&v)[32]) {
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

// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes wide and
// stored with the 128-byte swizzle: 8-row groups are 1024 bytes apart (stride byte offset),
// the leading byte offset is unused for swizzled K-major tiles, descriptor version 1.
__device__ __forceinline__ unsigned long long smem_desc_sw128(unsigned addr) {
    unsigned long long d = 0;
    d |= (unsigned long long)((addr & 0x3FFFFu) >> 4);        // start address, 16-byte units
    d |= (unsigned long long)1 << 16;                         // leading byte offset (ignored)
    d |= (unsigned long long)(1024 >> 4) << 32;               // stride byte offset
    d |= (unsigned long long)1 << 46;                         // descriptor version (sm_100)
    d |= (unsigned long long)2 << 61;                         // layout: 128-byte swizzle
    return d;
}
// Instruction descriptor: D = fp32, A = B = bf16, both K-major, M = 128, N = n.
__device__ __forceinline__ unsigned instr_desc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((unsigned)(n >> 3) << 17) | ((unsigned)(BM >> 4) << 24);
}

// ---------------------------------------------------------------- tile schedule
struct Tile {
    int b, row0, col0, n, m;
};

// Lower-triangular schedule for BN = 2*BM: row tiles 2p and 2p+1 both need p+1 column tiles.
__device__ __forceinline__ int tri_tiles(int n) {
    const int M = (n + BM - 1) / BM, P = M >> 1;
    return P * (P + 1) + ((M & 1) ? P + 1 : 0);
}
__device__ __forceinline__ bool decode_tile(const GramProblem& p, int id, Tile& t) {
    for (int b = 0; b < p.B; ++b) {
        const int n = p.n_dev != nullptr ? p.n_dev[b] : p.n_host;
        int cnt;
        if (p.tri) cnt = tri_tiles(n);
        else cnt = n > 0 ? ((p.rows + BM - 1) / BM) * ((n + BN - 1) / BN) : 0;
        if (id < cnt) {
            t.b = b;
            t.n = n;
            if (p.tri) {
                int P = (int)((sqrtf(4.0f * (float)id + 1.0f) - 1.0f) * 0.5f);
                while (P * (P + 1) > id) --P;
                while ((P + 1) * (P + 2) <= id) ++P;
                const int rem = id - P * (P + 1);
                const int mi = rem < P + 1 ? 2 * P : 2 * P + 1;
                const int nj = rem < P + 1 ? rem : rem - (P + 1);
                t.row0 = mi * BM;
                t.col0 = nj * BN;
                t.m = n;
            } else {
                const int nct = (n + BN - 1) / BN;
                t.row0 = (id / nct) * BM;
                t.col0 = (id % nct) * BN;
                t.m = p.rows;
            }
            return true;
        }
        id -= cnt;
    }
    return false;
}
// Columns the MMA must produce for a tile: up to the matrix edge, and for the triangular
// problem up to the last row of the tile; a multiple of 16 in [16, 256].
__device__ __forceinline__ int tile_ncols(const GramProblem& p, const Tile& t) {
    int nc = t.n - t.col0;
    if (p.tri) nc = min(nc, t.row0 + BM - t.col0);
    nc = min(nc, BN);
    return max(16, (nc + 15) & ~15);
}

// ---------------------------------------------------------------- the kernel
__global__ void __launch_bounds__(NUM_THREADS, 1)
k_gram_tc(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
          const GramProblem p, unsigned* __restrict__ status) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    Shared& sh = *reinterpret_cast<Shared*>(smem + STAGES * STAGE_BYTES);
    volatile int* abort_flag = &sh.abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kb = (p.d + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&sh.full[s], 1);
            mbar_init(&sh.empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&sh.tmem_full[a], 1);
            mbar_init(&sh.tmem_empty[a], 4);      // one arrival per epilogue warp
        }
        mbar_init(&sh.drain, 1);
        sh.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&sh.tmem_base)), "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const unsigned tmem_base = sh.tmem_base;

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            unsigned it = 0;      // running K-block counter over all of this CTA's tiles
            Tile t;
            bool ok = true;
            for (int id = blockIdx.x; ok && decode_tile(p, id, t); id += gridDim.x) {
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const unsigned ph = (it / STAGES) & 1u;
                    if (!mbar_wait(&sh.empty[s], ph ^ 1u, abort_flag, 1)) { ok = false; break; }
                    unsigned char* sa = smem + s * STAGE_BYTES;
                    mbar_expect_tx(&sh.full[s], STAGE_BYTES);
                    tma_load_3d(&map_a, &sh.full[s], sa, kb * BK, t.row0, t.b);
                    tma_load_3d(&map_b, &sh.full[s], sa + A_BYTES, kb * BK, t.col0, t.b);
                }
            }
            // drain: every copy this lane issued must have landed before the CTA may exit
            const unsigned issued = it;
            for (int s = 0; s < STAGES; ++s) {
                // number of fills issued to stage s
                const unsigned fills = issued / STAGES + ((issued % STAGES) > (unsigned)s ? 1u : 0u);
                if (fills == 0) continue;
                const unsigned ph = (fills - 1) & 1u;
                const unsigned long long t0 = global_ns();
                while (!mbar_try(&sh.full[s], ph)) {
                    if (global_ns() - t0 > WAIT_LIMIT_NS / 2) { *abort_flag = 7; break; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            unsigned it = 0, tile_it = 0;
            Tile t;
            bool ok = true;
            for (int id = blockIdx.x; ok && decode_tile(p, id, t); id += gridDim.x, ++tile_it) {
                const unsigned acc = tile_it & 1u, acc_ph = (tile_it >> 1) & 1u;
                if (!mbar_wait(&sh.tmem_empty[acc], acc_ph ^ 1u, abort_flag, 2)) { ok = false; break; }
                tcgen05_fence_after();
                const unsigned idesc = instr_desc(tile_ncols(p, t));
                const unsigned d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const unsigned ph = (it / STAGES) & 1u;
                    if (!mbar_wait(&sh.full[s], ph, abort_flag, 3)) { ok = false; break; }
                    tcgen05_fence_after();
                    const unsigned a_addr = smem_u32(smem + s * STAGE_BYTES);
                    const unsigned long long adesc = smem_desc_sw128(a_addr);
                    const unsigned long long bdesc = smem_desc_sw128(a_addr + A_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        // advancing K by 16 bf16 = 32 bytes = 2 descriptor address units
                        umma_bf16(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0);
                    }
                    umma_commit(&sh.empty[s]);          // stage reusable once these MMAs retire
                }
                if (ok) umma_commit(&sh.tmem_full[acc]);  // accumulator complete
            }
            // all MMAs issued by this thread must retire before TMEM is freed
            umma_commit(&sh.drain);
            const unsigned long long t0 = global_ns();
            while (!mbar_try(&sh.drain, 0)) {
                if (global_ns() - t0 > WAIT_LIMIT_NS / 2) { *abort_flag = 8; break; }
            }
        }
    } else {
        // ------------------------------------------------ epilogue (warps 2..5)
        const int quad = warp & 3;                    // TMEM lane quadrant this warp may read
        float* cs = sh.col_scale[warp - 2];
        int* ct = sh.col_token[warp - 2];
        unsigned tile_it = 0;
        Tile t;
        for (int id = blockIdx.x; decode_tile(p, id, t); id += gridDim.x, ++tile_it) {
            const unsigned acc = tile_it & 1u, acc_ph = (tile_it >> 1) & 1u;
            const int64_t o = (int64_t)t.b * p.cap;
            const int ncols = tile_ncols(p, t);
            const int ncols32 = (ncols + 31) & ~31;   // TMEM is read 32 columns at a time
            // stage this tile's column factors (0 for inadmissible columns); warp-private copy
            __syncwarp();
            for (int c = lane; c < ncols32; c += 32) {
                const int col = t.col0 + c;
                float f = 0.f;
                int tok = col;
                if (c < ncols && col < t.n) {
                    f = p.inv_b[o + col];
                    if (!p.tri) {
                        if (!(p.col_gate[o + col] < p.thr_bits)) f = 0.f;   // representative removed at line 5
                        if (p.causal) tok = p.col_token[o + col];
                    }
                }
                cs[c] = f;
                ct[c] = tok;
            }
            __syncwarp();
            // warp-uniform outcome of the bounded wait
            const bool got = mbar_wait(&sh.tmem_full[acc], acc_ph, abort_flag, 4);
            if (!__all_sync(0xffffffffu, got)) break;
            tcgen05_fence_after();
            const int row = t.row0 + quad * 32 + lane;
            const bool need_cmp = p.tri ? (t.col0 + ncols > t.row0) : (p.causal != 0);
            float mx = 0.f;
            for (int c0 = 0; c0 < ncols32; c0 += 32) {
                float v[32];
                tmem_ld32(tmem_base + ((unsigned)(quad * 32) << 16) + acc * BN + c0, v);
                if (!need_cmp) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        const float4 f = *reinterpret_cast<const float4*>(cs + c0 + j);
                        mx = fmaxf(mx, fabsf(v[j]) * f.x);
                        mx = fmaxf(mx, fabsf(v[j + 1]) * f.y);
                        mx = fmaxf(mx, fabsf(v[j + 2]) * f.z);
                        mx = fmaxf(mx, fabsf(v[j + 3]) * f.w);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const float x = fabsf(v[j]) * cs[c0 + j];
                        if (ct[c0 + j] < row) mx = fmaxf(mx, x);
                    }
                }
            }
            // accumulator consumed: hand it back to the MMA warp
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.tmem_empty[acc]);
            if (row < t.m) {
                const bool skip = !p.tri && p.row_role[o + row] != 0;   // inherited reps are not candidates
                if (!skip) {
                    mx *= p.inv_a[o + row];
                    if (mx > 0.f) atomicMax(p.out + o + row, __float_as_uint(mx));
                }
            }
        }
    }

    tcgen05_fence_before();
    __syncthreads();
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                     "r"(TMEM_COLS)
                     : "memory");
    }
    if (threadIdx.x == 0 && sh.abort_flag != 0) {
        atomicOr(status, ST_TIMEOUT);
        status[2] = (unsigned)sh.abort_flag;
    }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
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
bool make_map(CUtensorMap* map, const void* base, int d, int rows, int B, int64_t ld,
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

}  // namespace

bool gram_tc_available() { return encode_fn() != nullptr; }

cudaError_t launch_gram_tc(ada_ctx* ctx, const GramProblem& p, cudaStream_t s) {
    if (!ctx->tc_attr_set) {
        cudaError_t e = cudaFuncSetAttribute(k_gram_tc, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             SMEM_BYTES);
        if (e != cudaSuccess) return e;
        ctx->tc_attr_set = true;
    }
    const int n_cap = p.n_dev != nullptr ? p.cap : p.n_host;
    const int a_rows = p.tri ? n_cap : p.rows;
    if (n_cap <= 0 || a_rows <= 0) return cudaSuccess;
    CUtensorMap map_a, map_b;
    // rows beyond the matrices (and k beyond d) are zero-filled by the TMA unit
    if (!make_map(&map_a, p.A, p.d, p.tri ? p.cap : p.rows, p.B, p.lda, p.a_batch, BM) ||
        !make_map(&map_b, p.Bm, p.d, p.cap, p.B, p.ldb, p.b_batch, BN))
        return cudaErrorInvalidValue;
    prof_begin(ctx, p.tri ? K_GRAM_TC_TRI : K_GRAM_TC_CROSS, s);
    k_gram_tc<<<ctx->sm_count, NUM_THREADS, SMEM_BYTES, s>>>(map_a, map_b, p, ctx->status);
    prof_end(ctx, s);
    return cudaGetLastError();
}

}  // namespace ada
