// bf16 masked-Gram kernel for sm_100a: TMA -> shared memory -> tcgen05.mma -> TMEM,
// with the selection epilogue (1/(|a_i||b_j|) scaling, |.|, admissibility mask, row
// maximum) run straight out of TMEM, so that no Gram tile ever reaches HBM.
//
// Computes, per sequence, out[i] = max_j |a_i . b_j| * inv_a[i] * inv_b[j] over the
// admissible columns j (Definition 1; Algorithm 1 lines 3-4 and 7-8).  Both operands
// are row-major (K-major) bf16 matrices, so G = A B^T needs no transpose.
//
// One persistent CTA per SM.  Long-contraction shape, 14 warps:
//   warp 0      TMA producer: one lane issues cp.async.bulk.tensor loads of a 128 x 64
//               A box and up to four 64 x 64 B boxes per K block into a ring of 4 to 9
//               stages (fewer bytes per stage for narrow tiles, hence more K blocks in
//               flight; 128-byte swizzle, completion on an mbarrier)
//   warp 1      MMA issuer: one lane issues four tcgen05.mma (M=128, N<=256, K=16) per
//               K block; tcgen05.commit releases the ring stage, and after the last K
//               block hands the accumulator to the epilogue.  Owns the TMEM allocation
//               (512 columns = two 128 x 256 fp32 accumulators, so the epilogue of
//               tile i overlaps the main loop of tile i+1)
//   warps 2..5  epilogue: tcgen05.ld 32 lanes x 32 columns at a time (one accumulator
//               row per thread, so the row maximum is thread-local), then one
//               atomicMax per row and tile on the IEEE bit pattern (values are >= 0).
//   warps 6..13 optional row norms (Section 2.1): 1/||x_t|| of every row of X with plain
//               128-bit loads, overlapped with the main loops; the epilogues wait (bounded)
//               for them before they scale, so a long-K call needs no separate norm pass
// Short-contraction shape (d < 2048, no norm warps), 10 warps: warps 6..9 are a second
// epilogue set; see Shape below.
// Every wait is bounded: when a limit expires the CTA raises the context's TIMEOUT
// status, drains its own outstanding copies and MMAs (again bounded), frees its TMEM
// and returns.
#include "gram_tc_dev.cuh"


namespace ada {

using namespace tc;

namespace {

// The kernel comes in two shapes.  The long-contraction shape (14 warps, the last eight for the
// optional row norms) lives off its main loop: one epilogue set, a 216 KiB ring whose stage size
// follows each tile's width.  The short-contraction shape (d < 2048: one attention head, a small
// model width) lives off its epilogue, because a 128 x 256 fp32 accumulator takes about 2300
// cycles to read out of TMEM, more than such a tile's main loop: 10 warps, two epilogue sets that take
// alternate tiles (one accumulator each, so that one set's bookkeeping -- tile lookup, column
// factors, barrier, atomics -- overlaps the other's TMEM reads), a ring geometry fixed per
// segment (no drain between tiles of different width), one 256-row TMA box for a full-width
// right operand, a table of every sequence's length and first tile in shared memory (dozens of
// heads are dozens of sequences), and a 200 KiB ring to make room for all that.
template <bool SHORTK>
struct Shape {
    static constexpr int RING = SHORTK ? 200 * 1024 : RING_BYTES;
    static constexpr int PLAN_B = SHORTK ? 64 : 0;   // sequences whose tile ranges are kept in shared memory
    static constexpr int EPI_WARPS = SHORTK ? 8 : 4;
    static constexpr int THREADS = SHORTK ? 64 + 32 * 8 : NUM_THREADS;
};

// ---------------------------------------------------------------- work schedule
// A launch covers up to two problems ("segments"): a triangular one (Definition 1 on X, or
// Algorithm 1 lines 3-4 on the gathered representatives) and a cross one (lines 7-8).
// Their output tiles form one list, triangular tiles first, dealt round-robin to the
// persistent CTAs.  When both are present the cross epilogues need line 5's verdict on
// every column, i.e. the finished triangular segment: each epilogue warp bumps a global
// counter after publishing a triangular tile's maxima, and a cross epilogue waits (bounded)
// for the counter to reach 4 x (number of triangular tiles) before it stages its column
// factors.  The cross MAIN LOOPS do not wait, so the short r x r problem hides behind them.
// Triangular tiles precede cross tiles in every CTA's order and wait on nothing, and the
// launch is cooperative (all CTAs co-resident), so the wait always ends.
__device__ __forceinline__ int seq_n(const GramProblem& p, int b) {
    return p.n_dev != nullptr ? p.n_dev[b] : p.n_host;
}
// lower-triangular tile count for column tiles of width tw (64, 128 or 256): the 128-row
// tile mi needs the column tiles that start at or before its last row
__device__ __forceinline__ int tri_tiles(int n, int tw) {
    const int M = (n + BM - 1) / BM;
    if (tw == BM) return M * (M + 1) / 2;                // mi + 1 each
    if (tw == BM / 2) return M * (M + 1);                // 2 (mi + 1) each
    const int P = M >> 1;                                // row tiles 2P and 2P+1 both need P+1
    return P * (P + 1) + ((M & 1) ? P + 1 : 0);
}
// Stage geometry of the TMA ring for a tile of `ncols` columns: narrower tiles take fewer
// bytes per K block, so more K blocks fit in flight and the loop stays ahead of the
// load latency.
// bytes of one 64-element K block of a tile of `ncols` columns
__device__ __forceinline__ int sub_bytes(int ncols) {
    return A_BYTES + ((ncols + BOX_N - 1) / BOX_N) * BOX_BYTES;
}
// K blocks per ring stage: two where three such stages still fit the ring (tiles up to 128
// columns), so that the per-stage costs -- barrier round trips, fences, commit -- are paid
// once per 128 K elements; one for wider tiles
// (short contractions keep one: with a dozen K blocks the coarser pipeline costs more than
// it saves)
__device__ __forceinline__ int stage_ksub(int ncols, int d, int ring) {
    return (d >= 2048 && 3 * 2 * sub_bytes(ncols) <= ring) ? 2 : 1;
}
__device__ __forceinline__ int stage_count(int sbytes, int ring) {
    return min(MAX_STAGES, ring / sbytes);
}
// cross: columns are cut into nct equal tiles of width w (multiple of 16, <= 256).  `want` is
// the number of column tiles per row tile that would give every CTA one tile: a problem
// with few row tiles is cut finer (down to 64 columns), since a narrow tile moves fewer
// bytes per K block and finishes sooner, while a large one keeps 256-wide tiles.
__device__ __forceinline__ void cross_cols(int n, int want, int& nct, int& w) {
    const int lo = (n + BN - 1) / BN, hi = (n + BOX_N - 1) / BOX_N;
    nct = min(max(want, lo), hi);
    w = nct > 0 ? ((((n + nct - 1) / nct) + 15) & ~15) : 0;
}
// `par` below: column tile width (triangular segment) or wanted column tiles per row tile (cross)
// The tile ids a CTA takes from one segment ascend, so the search for a tile's sequence
// resumes at the sequence of the previous tile: `b` is that sequence, `base` the id of its
// first tile.  (With dozens of short sequences -- heads -- a search from sequence 0 for every
// tile would cost more than the tile's main loop.)
struct TileCursor {
    int b, base;
};
// tile `id` of segment p -> piece; false when id is past the segment's last tile
// s_n / s_first (shared memory, or NULL): length and first tile id of every sequence of the
// segment, s_first[B] = number of tiles; without them the lengths are read from global memory
// sequence by sequence.
__device__ __forceinline__ bool decode_tile(const GramProblem& p, int par, int id, Piece& t,
                                            TileCursor& cur, const int* s_n = nullptr,
                                            const int* s_first = nullptr) {
    const int tw = par;
    if (s_first != nullptr) {
        if (id >= s_first[p.B]) return false;
        int lo = cur.b;
        if (id >= s_first[lo + 1]) {                     // not the cursor's sequence: bisect above it
            int hi = p.B - 1;
            ++lo;
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (id >= s_first[mid + 1]) lo = mid + 1;
                else hi = mid;
            }
        }
        cur.b = lo;
        cur.base = s_first[lo];
    }
    for (; cur.b < p.B; ++cur.b) {
        const int b = cur.b;
        const int n = s_n != nullptr ? s_n[b] : seq_n(p, b);
        int cnt = 0, nct = 0, w = 0;
        if (n > 0) {
            if (p.tri) cnt = tri_tiles(n, tw);
            else {
                cross_cols(n, par, nct, w);
                cnt = ((p.rows + BM - 1) / BM) * nct;
            }
        }
        if (id - cur.base >= cnt) { cur.base += cnt; continue; }
        id -= cur.base;
        t.b = b;
        t.n = n;
        int nc;
        if (p.tri) {
            int mi, nj;
            if (tw == BM / 2) {                          // row tile mi holds tiles mi(mi+1) ... + 2mi+1
                mi = (int)((sqrtf(4.0f * (float)id + 1.0f) - 1.0f) * 0.5f);
                while (mi * (mi + 1) > id) --mi;
                while ((mi + 1) * (mi + 2) <= id) ++mi;
                nj = id - mi * (mi + 1);
            } else if (tw == BM) {                       // row tile mi holds tiles mi(mi+1)/2 ... + mi
                mi = (int)((sqrtf(8.0f * (float)id + 1.0f) - 1.0f) * 0.5f);
                while (mi * (mi + 1) / 2 > id) --mi;
                while ((mi + 1) * (mi + 2) / 2 <= id) ++mi;
                nj = id - mi * (mi + 1) / 2;
            } else {
                int P = (int)((sqrtf(4.0f * (float)id + 1.0f) - 1.0f) * 0.5f);
                while (P * (P + 1) > id) --P;
                while ((P + 1) * (P + 2) <= id) ++P;
                const int rem = id - P * (P + 1);
                mi = rem < P + 1 ? 2 * P : 2 * P + 1;
                nj = rem < P + 1 ? rem : rem - (P + 1);
            }
            t.row0 = mi * BM;
            t.col0 = nj * tw;
            t.m = n;
            nc = min(min(n - t.col0, t.row0 + BM - t.col0), tw);   // nothing right of the tile's last row
        } else {
            t.row0 = (id / nct) * BM;
            t.col0 = (id % nct) * w;
            t.m = p.rows;
            nc = min(n - t.col0, w);
        }
        t.ncols = max(16, (nc + 15) & ~15);                        // MMA N: multiple of 16
        return true;
    }
    return false;
}

// ---------------------------------------------------------------- the kernel
// Under ADA_CROSS_CAUSAL a cross tile whose first (lowest) column token is not below the
// tile's last row has no admissible (row, column) pair: every role skips it, so neither
// its loads nor its MMAs are issued.  Column tokens ascend with the column index.
__device__ __forceinline__ bool dead_tile(const GramProblem& p, const Piece& pc) {
    if (p.tri || !p.causal || p.col_token == nullptr) return false;
    return p.col_token[(int64_t)pc.b * p.cap + pc.col0] >= pc.row0 + BM;
}

// The first TAB tiles of every CTA are decoded once, by TAB threads in parallel while the
// kernel starts, into a table in shared memory: with a short contraction a tile's main loop
// is a few hundred cycles, less than the serial integer work of decoding it three times
// (producer, MMA issuer, epilogue).  Entry: x = row0 | ncols/16 << 24 | dead << 31, y = col0,
// z = n (0: no tile), w = sequence.  Tiles past the table are decoded on the fly.
constexpr int TAB = 80;
template <bool SHORTK>
struct alignas(16) SharedTc {
    unsigned long long full[MAX_STAGES];
    unsigned long long empty[MAX_STAGES];
    unsigned long long tmem_full[2];
    unsigned long long tmem_empty[2];
    unsigned long long drain;
    unsigned tmem_base;
    int abort_flag;
    int tiles0, tiles1, par0, par1;
    int wide0, wide1;           // widest tile of each segment (fixes the segment's ring geometry)
    uint4 tile_tab[TAB];
    int seq_len[2][Shape<SHORTK>::PLAN_B + 1];     // per segment: sequence lengths ...
    int seq_first[2][Shape<SHORTK>::PLAN_B + 1];   // ... and first tile ids (entry B: tile count)
    // per epilogue warp, so that staging needs no barrier across warps
    alignas(16) float col_scale[Shape<SHORTK>::EPI_WARPS][BN];
    alignas(16) int col_token[Shape<SHORTK>::EPI_WARPS][BN];
};
template <bool SHORTK>
constexpr int smem_tc_bytes() {
    return Shape<SHORTK>::RING + (int)sizeof(SharedTc<SHORTK>) + 1024;   // +1024: alignment slack
}
static_assert(smem_tc_bytes<false>() <= 227 * 1024 && smem_tc_bytes<true>() <= 227 * 1024,
              "shared memory budget");

// 0: no such tile, 1: tile in pc, 2: tile in pc but nothing to do (dead_tile)
__device__ __forceinline__ int next_tile(const uint4* tab, int it, const GramProblem& p, int par,
                                         int local_id, Piece& pc, TileCursor& cur,
                                         const int* s_n, const int* s_first) {
    if (it < TAB) {
        const uint4 e = tab[it];
        if (e.z == 0u) return 0;
        pc.row0 = (int)(e.x & 0xFFFFFFu);
        pc.ncols = (int)((e.x >> 24) & 31u) * 16;
        pc.col0 = (int)e.y;
        pc.n = (int)e.z;
        pc.b = (int)e.w;
        pc.m = p.tri ? pc.n : p.rows;
        return (e.x >> 31) ? 2 : 1;
    }
    if (!decode_tile(p, par, local_id, pc, cur, s_n, s_first)) return 0;
    return dead_tile(p, pc) ? 2 : 1;
}

struct GramMaps {
    // per segment: left operand (128-row boxes), right operand in 64-row and in 256-row boxes
    CUtensorMap a[2], b[2], bw[2];
};

template <bool SHORTK>
__global__ void __launch_bounds__(Shape<SHORTK>::THREADS, 1)
k_gram_tc(const __grid_constant__ GramMaps maps, const __grid_constant__ GramProblem seg0,
          const __grid_constant__ GramProblem seg1, const int nseg,
          const __grid_constant__ NormJob norms, unsigned* __restrict__ dep_ctr,
          unsigned* __restrict__ status) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    constexpr int RING = Shape<SHORTK>::RING;
    SharedTc<SHORTK>& sh = *reinterpret_cast<SharedTc<SHORTK>*>(smem + RING);
    volatile int* abort_flag = &sh.abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_STAGES; ++s) {
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
    // everything above is local to the CTA; from here on the predecessor's results are read
    grid_dep_wait();
    if (warp == 2) {
        // Work plan.  Everything per sequence -- its length, its tile counts -- is computed by
        // the lanes in parallel and reduced with shuffles: the lengths live in global memory, and
        // one thread walking dozens of sequences (heads) would hold the whole CTA back.
        const int G = (int)gridDim.x;
        int s256 = 0, s128 = 0, s64 = 0, rt0 = 0, rt1 = 0;
        for (int b = lane; b < seg0.B; b += 32) {
            const int n = seq_n(seg0, b);
            if (n <= 0) continue;
            if (seg0.tri) {
                s256 += tri_tiles(n, BN);
                s128 += tri_tiles(n, BM);
                s64 += tri_tiles(n, BM / 2);
            } else {
                rt0 += (seg0.rows + BM - 1) / BM;
            }
        }
        if (nseg > 1 && !seg1.tri)
            for (int b = lane; b < seg1.B; b += 32)
                if (seq_n(seg1, b) > 0) rt1 += (seg1.rows + BM - 1) / BM;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            s256 += __shfl_xor_sync(0xffffffffu, s256, o);
            s128 += __shfl_xor_sync(0xffffffffu, s128, o);
            s64 += __shfl_xor_sync(0xffffffffu, s64, o);
            rt0 += __shfl_xor_sync(0xffffffffu, rt0, o);
            rt1 += __shfl_xor_sync(0xffffffffu, rt1, o);
        }
        // a triangular problem too small to give every CTA a 256-wide tile is cut 128 or 64 wide
        // (narrower tiles move fewer bytes per K block and finish sooner) as long as that
        // still fits in one round of the grid; a cross problem gets as many column tiles per
        // row tile as fill the grid once
        int par0 = BN, t0 = s256;
        if (seg0.tri && 2 * t0 < G) { par0 = BM; t0 = s128; }
        if (seg0.tri && 2 * t0 < G) { par0 = BM / 2; t0 = s64; }
        if (!seg0.tri) par0 = rt0 > 0 ? max(1, G / rt0) : 1;
        const int par1 = (nseg > 1 && !seg1.tri) ? (rt1 > 0 ? max(1, G / rt1) : 1) : BN;
        // second pass: tile count and widest tile of each segment; with few enough sequences
        // also every sequence's length and first tile id, for the tile search
        int c0 = 0, c1 = 0, w0 = 16, w1 = 16;
        constexpr int PLAN_B = Shape<SHORTK>::PLAN_B;
        if constexpr (!SHORTK) {
            for (int b = lane; b < seg0.B; b += 32) {
                const int n = seq_n(seg0, b);
                if (n <= 0) continue;
                if (seg0.tri) {
                    c0 += tri_tiles(n, par0);
                } else {
                    int nct, w;
                    cross_cols(n, par0, nct, w);
                    c0 += ((seg0.rows + BM - 1) / BM) * nct;
                }
            }
            if (nseg > 1)
                for (int b = lane; b < seg1.B; b += 32) {
                    const int n = seq_n(seg1, b);
                    if (n <= 0) continue;
                    if (seg1.tri) {
                        c1 += tri_tiles(n, BN);
                    } else {
                        int nct, w;
                        cross_cols(n, par1, nct, w);
                        c1 += ((seg1.rows + BM - 1) / BM) * nct;
                    }
                }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                c0 += __shfl_xor_sync(0xffffffffu, c0, o);
                c1 += __shfl_xor_sync(0xffffffffu, c1, o);
            }
        } else {
            for (int sgi = 0; sgi < nseg; ++sgi) {
                const GramProblem& p = sgi ? seg1 : seg0;
                const int par = sgi ? par1 : par0;
                const bool keep = p.B <= PLAN_B;
                int run = 0, wide = 16;                      // tiles of the sequences before this round
                for (int b0 = 0; b0 < p.B; b0 += 32) {
                    const int b = b0 + lane;
                    int n = 0, cnt = 0;
                    if (b < p.B) {
                        n = max(seq_n(p, b), 0);
                        if (n > 0) {
                            if (p.tri) {
                                cnt = tri_tiles(n, par);
                                wide = max(wide, min(par, (n + 15) & ~15));
                            } else {
                                int nct, w;
                                cross_cols(n, par, nct, w);
                                cnt = ((p.rows + BM - 1) / BM) * nct;
                                wide = max(wide, w);
                            }
                        }
                    }
                    int incl = cnt;
    #pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const int v = __shfl_up_sync(0xffffffffu, incl, o);
                        if (lane >= o) incl += v;
                    }
                    if (keep && b < p.B) {
                        sh.seq_len[sgi][b] = n;
                        sh.seq_first[sgi][b] = run + incl - cnt;
                    }
                    run += __shfl_sync(0xffffffffu, incl, 31);
                }
    #pragma unroll
                for (int o = 16; o > 0; o >>= 1) wide = max(wide, __shfl_xor_sync(0xffffffffu, wide, o));
                if (keep && lane == 0) sh.seq_first[sgi][p.B] = run;
                if (sgi == 0) { c0 = run; w0 = wide; }
                else { c1 = run; w1 = wide; }
            }
        }
        if (lane == 0) {
            sh.par0 = par0;
            sh.tiles0 = c0;
            sh.wide0 = min(w0, BN);
            sh.par1 = nseg > 1 ? par1 : 1;
            sh.tiles1 = nseg > 1 ? c1 : 0;
            sh.wide1 = min(w1, BN);
        }
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const unsigned tmem_base = sh.tmem_base;
    const int tiles0 = sh.tiles0, total = sh.tiles0 + sh.tiles1, par0 = sh.par0, par1 = sh.par1;
    const int wide0 = sh.wide0, wide1 = sh.wide1;
    Piece pc;
    // per-segment sequence tables (NULL: too many sequences, or the long-contraction shape)
    const int* sn0 = seg0.B <= Shape<SHORTK>::PLAN_B ? sh.seq_len[0] : nullptr;
    const int* sf0 = seg0.B <= Shape<SHORTK>::PLAN_B ? sh.seq_first[0] : nullptr;
    const int* sn1 = seg1.B <= Shape<SHORTK>::PLAN_B ? sh.seq_len[1] : nullptr;
    const int* sf1 = seg1.B <= Shape<SHORTK>::PLAN_B ? sh.seq_first[1] : nullptr;
    if (threadIdx.x < TAB) {
        const int id = blockIdx.x + (int)threadIdx.x * (int)gridDim.x;
        uint4 e = make_uint4(0u, 0u, 0u, 0u);
        if (id < total) {
            const int sg = id < tiles0 ? 0 : 1;
            const GramProblem& p = sg ? seg1 : seg0;
            TileCursor c0 = {0, 0};
            if (decode_tile(p, sg ? par1 : par0, id - (sg ? tiles0 : 0), pc, c0, sg ? sn1 : sn0, sg ? sf1 : sf0))
                e = make_uint4((unsigned)pc.row0 | ((unsigned)(pc.ncols >> 4) << 24) |
                                   (dead_tile(p, pc) ? 0x80000000u : 0u),
                               (unsigned)pc.col0, (unsigned)pc.n, (unsigned)pc.b);
        }
        sh.tile_tab[threadIdx.x] = e;
    }
    __syncthreads();

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            unsigned fills = 0;      // bit s: parity of the number of fills of stage s
            unsigned used = 0;       // stages filled under the current geometry
            unsigned ever = 0;       // stages ever filled
            int cur_sb = 0, cur_nst = 0, s = 0;
            bool ok = true;
            TileCursor cur = {0, 0};
            int cur_sg = 0;
            int it = 0;
            for (int id = blockIdx.x; ok && id < total; id += gridDim.x, ++it) {
                const int sg = id < tiles0 ? 0 : 1;
                const GramProblem& p = sg ? seg1 : seg0;
                if (sg != cur_sg) { cur.b = 0; cur.base = 0; cur_sg = sg; }
                const int got_tile = next_tile(sh.tile_tab, it, p, sg ? par1 : par0,
                                               id - (sg ? tiles0 : 0), pc, cur, sg ? sn1 : sn0,
                                               sg ? sf1 : sf0);
                if (got_tile == 0) break;
                if (got_tile == 2) continue;      // causal cross tile with no admissible pair
                // ring geometry is fixed per segment by its widest tile, so that a narrower
                // (diagonal or last) tile needs no drain of the ring: it fills less of its stage
                const int wide = SHORTK ? (sg ? wide1 : wide0) : pc.ncols;
                const int ksub = stage_ksub(wide, p.d, RING);
                const int num_kb = (p.d + BK * ksub - 1) / (BK * ksub);
                const int nbox = (pc.ncols + BOX_N - 1) / BOX_N;
                const int subb = sub_bytes(wide);
                const int sb = ksub * subb;
                const unsigned tx = (unsigned)(ksub * sub_bytes(pc.ncols));
                if (sb != cur_sb) {
                    // new stage geometry: every stage of the old one must have been released
                    for (int q = 0; q < cur_nst && ok; ++q)
                        if ((used >> q) & 1u)
                            ok = mbar_wait(&sh.empty[q], ((fills >> q) & 1u) ^ 1u, abort_flag, 6);
                    if (!ok) break;
                    cur_sb = sb; cur_nst = stage_count(sb, RING); s = 0; used = 0;
                }
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(&sh.empty[s], ((fills >> s) & 1u) ^ 1u, abort_flag, 1)) { ok = false; break; }
                    unsigned char* sa = smem + s * sb;
                    mbar_expect_tx(&sh.full[s], tx);
                    for (int u = 0; u < ksub; ++u) {          // K blocks past d are zero-filled
                        unsigned char* su = sa + u * subb;
                        const int k0 = (kb * ksub + u) * BK;
                        tma_load_3d(&maps.a[sg], &sh.full[s], su, k0, pc.row0, pc.b);
                        if (SHORTK && nbox == BN / BOX_N) {   // full-width tile: one 256-row box
                            tma_load_3d(&maps.bw[sg], &sh.full[s], su + A_BYTES, k0, pc.col0, pc.b);
                        } else {
                            for (int j = 0; j < nbox; ++j)
                                tma_load_3d(&maps.b[sg], &sh.full[s], su + A_BYTES + j * BOX_BYTES, k0,
                                            pc.col0 + j * BOX_N, pc.b);
                        }
                    }
                    fills ^= 1u << s; used |= 1u << s; ever |= 1u << s;
                    s = (s + 1 == cur_nst) ? 0 : s + 1;
                }
            }
            // drain: every copy this lane issued must have landed before the CTA may exit
            for (int q = 0; q < MAX_STAGES; ++q) {
                if (!((ever >> q) & 1u)) continue;
                const unsigned ph = ((fills >> q) & 1u) ^ 1u;      // parity of the last fill's phase
                const unsigned long long t0 = global_ns();
                while (!mbar_try(&sh.full[q], ph)) {
                    if (global_ns() - t0 > WAIT_LIMIT_NS / 2) { *abort_flag = 7; break; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            unsigned uses = 0, tile_it = 0;   // bit s of `uses`: parity of the number of uses of stage s
            int cur_sb = 0, cur_nst = 0, s = 0;
            bool ok = true;
            TileCursor cur = {0, 0};
            int cur_sg = 0;
            int it = 0;
            for (int id = blockIdx.x; ok && id < total; id += gridDim.x, ++it) {
                const int sg = id < tiles0 ? 0 : 1;
                const GramProblem& p = sg ? seg1 : seg0;
                if (sg != cur_sg) { cur.b = 0; cur.base = 0; cur_sg = sg; }
                const int got_tile = next_tile(sh.tile_tab, it, p, sg ? par1 : par0,
                                               id - (sg ? tiles0 : 0), pc, cur, sg ? sn1 : sn0,
                                               sg ? sf1 : sf0);
                if (got_tile == 0) break;
                if (got_tile == 2) continue;      // causal cross tile with no admissible pair
                const int wide = SHORTK ? (sg ? wide1 : wide0) : pc.ncols;
                const int ksub = stage_ksub(wide, p.d, RING);
                const int num_kb = (p.d + BK * ksub - 1) / (BK * ksub);
                const int subb = sub_bytes(wide);
                const int sb = ksub * subb;
                if (sb != cur_sb) { cur_sb = sb; cur_nst = stage_count(sb, RING); s = 0; }
                const unsigned acc = tile_it & 1u, acc_ph = (tile_it >> 1) & 1u;
                ++tile_it;
                if (!mbar_wait(&sh.tmem_empty[acc], acc_ph ^ 1u, abort_flag, 2)) { ok = false; break; }
                tcgen05_fence_after();
                const unsigned idesc = instr_desc(pc.ncols);
                const unsigned d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(&sh.full[s], (uses >> s) & 1u, abort_flag, 3)) { ok = false; break; }
                    tcgen05_fence_after();
                    for (int u = 0; u < ksub; ++u) {
                        const unsigned a_addr = smem_u32(smem + s * sb + u * subb);
                        const unsigned long long adesc = smem_desc_sw128(a_addr);
                        const unsigned long long bdesc = smem_desc_sw128(a_addr + A_BYTES);
#pragma unroll
                        for (int k = 0; k < BK / UMMA_K; ++k) {
                            // advancing K by 16 bf16 = 32 bytes = 2 descriptor address units
                            umma_bf16(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | u | k) != 0);
                        }
                    }
                    umma_commit(&sh.empty[s]);          // stage reusable once these MMAs retire
                    uses ^= 1u << s;
                    s = (s + 1 == cur_nst) ? 0 : s + 1;
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
    } else if (warp < 2 + Shape<SHORTK>::EPI_WARPS) {
        // ------------------------------------------------ epilogue (warps 2..5, and 6..9 without norm warps)
        const int quad = warp & 3;                    // TMEM lane quadrant this warp may read
        const unsigned eset = (unsigned)(warp - 2) >> 2;   // which of the two sets
        float* cs = sh.col_scale[warp - 2];
        int* ct = sh.col_token[warp - 2];
        const unsigned dep_total = 4u * (unsigned)tiles0;
        bool dep_ok = !(nseg > 1 && tiles0 > 0);
        bool norm_ok = norms.X == nullptr;           // row norms computed by this launch's norm warps
        const unsigned norm_total = (unsigned)(gridDim.x * NORM_WARPS);      // cross epilogues must see segment 0 finished
        unsigned tile_it = 0;
        TileCursor cur = {0, 0};
            int cur_sg = 0;
        int it = 0;
        for (int id = blockIdx.x; id < total; id += gridDim.x, ++it) {
            const int sg = id < tiles0 ? 0 : 1;
            const GramProblem& p = sg ? seg1 : seg0;
            if (sg != cur_sg) { cur.b = 0; cur.base = 0; cur_sg = sg; }
            const int got_tile = next_tile(sh.tile_tab, it, p, sg ? par1 : par0,
                                           id - (sg ? tiles0 : 0), pc, cur, sg ? sn1 : sn0, sg ? sf1 : sf0);
            if (got_tile == 0) break;
            if (got_tile == 2) continue;          // causal cross tile with no admissible pair
            const unsigned acc = tile_it & 1u, acc_ph = (tile_it >> 1) & 1u;
            ++tile_it;
            if (SHORTK && acc != eset) continue;      // the other set's tile
            const int64_t o = (int64_t)pc.b * p.cap;
            const int ncols = pc.ncols;
            const int ncols32 = (ncols + 31) & ~31;   // TMEM is read 32 columns at a time
            if (sg == 1 && !dep_ok) {
                // every triangular tile of this launch first (line 5 before line 7)
                if (!wait_counter(dep_ctr, dep_total, lane, abort_flag, 5)) break;
                dep_ok = true;
            }
            if (p.wait_norm_b && !norm_ok) {
                if (!wait_counter(dep_ctr + 1, norm_total, lane, abort_flag, 9)) break;
                norm_ok = true;
            }
            // stage this tile's column factors (0 for inadmissible columns); warp-private copy
            __syncwarp();
            {
                // all of the tile's global loads are issued before the first is used: with a
                // short contraction the epilogue is the critical path, and eight dependent
                // round trips to L2 would be most of it
                float fb[BN / 32];
                unsigned gate[BN / 32] = {};
                int tk[BN / 32] = {};
                // (columns past the tile are clamped to its last one and discarded afterwards,
                // so that no load hangs on a data-dependent branch)
                const int last = pc.n - 1;
                const unsigned thr_b = (!p.tri && p.thr_seq != nullptr) ? p.thr_seq[pc.b] : p.thr_bits;
#pragma unroll
                for (int q = 0; q < BN / 32; ++q)
                    fb[q] = __ldcg(p.inv_b + o + min(pc.col0 + lane + 32 * q, last));
                if (!p.tri) {
                    // representative removed at line 5 (written earlier in this launch: read at L2)
#pragma unroll
                    for (int q = 0; q < BN / 32; ++q)
                        gate[q] = __ldcg(p.col_gate + o + min(pc.col0 + lane + 32 * q, last));
                }
                if (!p.tri && p.causal) {
#pragma unroll
                    for (int q = 0; q < BN / 32; ++q)
                        tk[q] = p.col_token[o + min(pc.col0 + lane + 32 * q, last)];
                }
#pragma unroll
                for (int q = 0; q < BN / 32; ++q) {
                    const int c = lane + 32 * q, col = pc.col0 + c;
                    const bool live = c < ncols && col < pc.n;
                    if (c < ncols32) {
                        cs[c] = (live && (p.tri || gate[q] < thr_b)) ? fb[q] : 0.f;
                        ct[c] = (live && !p.tri && p.causal) ? tk[q] : col;
                    }
                }
            }
            __syncwarp();
            // this thread's row: its role and inverse norm are fetched while the MMAs finish
            const int row = pc.row0 + quad * 32 + lane;
            const bool row_live = row < pc.m;
            const bool skip = row_live && !p.tri && p.row_role[o + row] != 0;   // inherited reps are not candidates
            const bool inv_early = !(p.wait_norm_a && !norm_ok);
            float inv_row = (row_live && inv_early) ? __ldcg(p.inv_a + o + row) : 0.f;
            // warp-uniform outcome of the bounded wait
            const bool got = mbar_wait(&sh.tmem_full[acc], acc_ph, abort_flag, 4);
            if (!__all_sync(0xffffffffu, got)) break;
            tcgen05_fence_after();
            const bool need_cmp = p.tri ? (pc.col0 + ncols > pc.row0) : (p.causal != 0);
            float mx4[2] = {0.f, 0.f};                    // independent partial maxima
            int arg = 0;                                  // nearest-representative mode: column of the maximum
            const bool want_arg = p.out_arg != nullptr;
            const unsigned tbase = tmem_base + ((unsigned)(quad * 32) << 16) + acc * BN;
            if (want_arg) {
                for (int c0 = 0; c0 < ncols32; c0 += 32) {
                    float v[32];
                    tmem_ld32(tbase + c0, v);
#pragma unroll
                    for (int j = 0; j < 32; ++j) {        // ascending columns, strict '>': lowest index on ties
                        const float x = fabsf(v[j]) * cs[c0 + j];
                        if (x > mx4[0]) { mx4[0] = x; arg = c0 + j; }
                    }
                }
            } else {
                auto consume = [&](const unsigned (&r)[32], int c0) {
                    if (!need_cmp) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            const float4 f = *reinterpret_cast<const float4*>(cs + c0 + j);
                            mx4[0] = fmaxf(mx4[0], fabsf(__uint_as_float(r[j])) * f.x);
                            mx4[1] = fmaxf(mx4[1], fabsf(__uint_as_float(r[j + 1])) * f.y);
                            mx4[0] = fmaxf(mx4[0], fabsf(__uint_as_float(r[j + 2])) * f.z);
                            mx4[1] = fmaxf(mx4[1], fabsf(__uint_as_float(r[j + 3])) * f.w);
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            const float4 f = *reinterpret_cast<const float4*>(cs + c0 + j);
                            const int4 t = *reinterpret_cast<const int4*>(ct + c0 + j);
                            if (t.x < row) mx4[0] = fmaxf(mx4[0], fabsf(__uint_as_float(r[j])) * f.x);
                            if (t.y < row) mx4[1] = fmaxf(mx4[1], fabsf(__uint_as_float(r[j + 1])) * f.y);
                            if (t.z < row) mx4[0] = fmaxf(mx4[0], fabsf(__uint_as_float(r[j + 2])) * f.z);
                            if (t.w < row) mx4[1] = fmaxf(mx4[1], fabsf(__uint_as_float(r[j + 3])) * f.w);
                        }
                    }
                };
                for (int c0 = 0; c0 < ncols32; c0 += 32) {
                    unsigned ra[32];
                    tmem_ld32_issue(tbase + c0, ra);
                    tmem_ld_wait(ra);
                    consume(ra, c0);
                }
            }
            float mx = fmaxf(mx4[0], mx4[1]);
            // accumulator consumed: hand it back to the MMA warp
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.tmem_empty[acc]);
            if (p.wait_norm_a && !norm_ok) {
                if (!wait_counter(dep_ctr + 1, norm_total, lane, abort_flag, 9)) break;
                norm_ok = true;
            }
            if (row_live) {
                if (!skip) {
                    if (!inv_early) inv_row = __ldcg(p.inv_a + o + row);
                    mx *= inv_row;
                    if (want_arg) {
                        const unsigned long long key =
                            ((unsigned long long)__float_as_uint(mx) << 32) |
                            (unsigned long long)(0xFFFFFFFFu - (unsigned)(pc.col0 + arg));
                        if (mx > 0.f) atomicMax(p.out_arg + o + row, key);
                    } else if (mx > 0.f) {
                        atomicMax(p.out + o + row, __float_as_uint(mx));
                    }
                }
            }
            if (sg == 0 && nseg > 1) {
                // publish: this warp's share of a triangular tile is in global memory
                __threadfence();
                __syncwarp();
                if (lane == 0) atomicAdd(dep_ctr, 1u);
            }
        }
    } else if (!SHORTK && norms.X != nullptr) {
        // ------------------------------------------------ row norms (warps 6 and up)
        norm_rows(norms, blockIdx.x * NORM_WARPS + (warp - 6), gridDim.x * NORM_WARPS, lane,
                  dep_ctr + 1, status);
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

}  // namespace

bool gram_tc_available() { return encode_fn() != nullptr; }

namespace {
// One warp waits on a counter that stays at zero; the limit expires and the status is raised.
__global__ void k_selftest_wait(const unsigned* counter, unsigned long long limit_ns,
                                unsigned* status) {
    grid_dep_wait();
    __shared__ int abort_flag;
    if (threadIdx.x == 0) abort_flag = 0;
    __syncwarp();
    const bool ok = wait_counter(counter, 1u, threadIdx.x & 31, &abort_flag, 11, limit_ns);
    if (!ok && threadIdx.x == 0) {
        atomicOr(status, ST_TIMEOUT);
        status[2] = (unsigned)abort_flag;
    }
}
}  // namespace

cudaError_t launch_selftest_wait(ada_ctx* ctx, int limit_ms, cudaStream_t s) {
    // tile_ctr[2] is never written by any kernel
    launch_k(ctx, k_selftest_wait, dim3(1), dim3(32), 0, s, ctx->tile_ctr + 2,
             (unsigned long long)limit_ms * 1000000ull, ctx->status);
    return cudaGetLastError();
}

// tri and/or cross may be NULL.  With both, the cross epilogues wait inside the kernel for the
// triangular segment (ctx->tile_ctr must be zero at launch) and the launch is cooperative.
cudaError_t launch_gram_tc(ada_ctx* ctx, const GramProblem* tri, const GramProblem* cross,
                           const NormJob* norms, cudaStream_t s) {
    if (!ctx->tc_attr_set) {
        cudaError_t e = cudaFuncSetAttribute(k_gram_tc<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             smem_tc_bytes<true>());
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(k_gram_tc<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 smem_tc_bytes<false>());
        if (e != cudaSuccess) return e;
        ctx->tc_attr_set = true;
    }
    GramMaps maps;
    memset(&maps, 0, sizeof(maps));
    GramProblem segs[2];
    memset(segs, 0, sizeof(segs));
    int nseg = 0;
    const GramProblem* in[2] = {tri, cross};
    for (int i = 0; i < 2; ++i) {
        const GramProblem* p = in[i];
        if (p == nullptr) continue;
        const int n_cap = p->n_dev != nullptr ? p->cap : p->n_host;
        const int a_rows = p->tri ? n_cap : p->rows;
        if (n_cap <= 0 || a_rows <= 0) continue;
        // rows beyond the matrices (and k beyond d) are zero-filled by the TMA unit
        if (!make_map(&maps.a[nseg], p->A, p->d, p->tri ? p->cap : p->rows, p->B, p->lda, p->a_batch, BM) ||
            !make_map(&maps.b[nseg], p->Bm, p->d, p->cap, p->B, p->ldb, p->b_batch, BOX_N) ||
            !make_map(&maps.bw[nseg], p->Bm, p->d, p->cap, p->B, p->ldb, p->b_batch, BN))
            return cudaErrorInvalidValue;
        segs[nseg++] = *p;
    }
    if (nseg == 0) return cudaSuccess;
    if (nseg == 1) { maps.a[1] = maps.a[0]; maps.b[1] = maps.b[0]; maps.bw[1] = maps.bw[0]; segs[1] = segs[0]; segs[1].B = 0; }
    NormJob nj;
    memset(&nj, 0, sizeof(nj));
    if (norms != nullptr) nj = *norms;
    const bool fused = nseg == 2;
    prof_begin(ctx, fused ? K_GRAM_TC_CASCADE : (segs[0].tri ? K_GRAM_TC_TRI : K_GRAM_TC_CROSS), s);
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(ctx->sm_count);
    // short contraction and no norm warps needed: the epilogue-bound shape
    const bool shortk = nj.X == nullptr && segs[0].d < 2048;
    cfg.blockDim = dim3(shortk ? Shape<true>::THREADS : Shape<false>::THREADS);
    cfg.dynamicSmemBytes = shortk ? smem_tc_bytes<true>() : smem_tc_bytes<false>();
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (fused && ctx->cooperative) {
        attr[na].id = cudaLaunchAttributeCooperative;
        attr[na].val.cooperative = 1;
        ++na;
    }
    if (ctx->dep_launch) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    cudaError_t e = shortk ? cudaLaunchKernelEx(&cfg, k_gram_tc<true>, maps, segs[0], segs[1], nseg, nj,
                                                ctx->tile_ctr, ctx->status)
                           : cudaLaunchKernelEx(&cfg, k_gram_tc<false>, maps, segs[0], segs[1], nseg, nj,
                                                ctx->tile_ctr, ctx->status);
    prof_end(ctx, s);
    return e;
}

}  // namespace ada
