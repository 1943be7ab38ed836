// bf16 masked-Gram kernel for sm_100a, two-CTA form: the CTAs of a cluster of two
// (one per SM of a TPC) share one 256-row output tile.  Each CTA loads its own 128 rows
// of the left operand but only HALF of the right operand's columns; the leader CTA
// issues tcgen05.mma.cta_group::2 (M = 256), which reads both halves from the two shared
// memories and writes each CTA's 128 x N accumulator into its own TMEM.  Per CTA and
// K block that is 16 KiB + N*64 bytes of TMA traffic instead of 16 KiB + N*128: the
// one-CTA kernel is bound by what one SM can pull out of L2, this one by the tensor pipe.
//
// Same contract as the one-CTA kernel (out[i] = max_j |a_i.b_j| inv_a[i] inv_b[j] over the
// admissible j; Definition 1, Algorithm 1 lines 3-4 and 7-8; the Gram never leaves TMEM),
// same tile list (triangular segment first, cross epilogues wait for it), same warp roles:
//   warp 0      TMA producer in BOTH CTAs (completion bytes of both land on the leader's
//               mbarrier; no multicast is used)
//   warp 1      leader: MMA issuer; releases ring stages and hands over accumulators with
//               tcgen05.commit multicast to both CTAs.  Both CTAs: TMEM allocation
//   warps 2..5  epilogue in both CTAs, each on its own 128 rows; the peer's epilogue
//               returns the accumulator by a remote arrive on the leader's mbarrier
//   warps 6..13 helpers.  Full selection: 1/||x_t|| of every row with plain loads, behind the
//               main loops.  Cascade step: first the gather of Algorithm 1 lines 1-2 (list
//               checked, role map, rows copied to Xrep with their inverse norms; loads of Xrep
//               and the epilogues wait for it), then warps 6..9 take the row norms of X out of
//               the left-operand tiles while those sit in shared memory (tiles of the first
//               column tile only; one thread per row), so X is read from memory exactly once
// The cross segment's row maxima are published WITHOUT the factor 1/||x_t|| (it commutes with
// the maximum; the compaction applies it), so no epilogue waits for a norm.  When one column
// tile covers all representatives the step is bound by streaming X once: the row tiles are
// then cut shorter than 128 rows per CTA so that every SM pair streams a share.
// Every wait is bounded; the two CTAs meet at a cluster barrier before either frees TMEM
// or exits.
#include "gram_tc_dev.cuh"

namespace ada {

using namespace tc;

// Time stamps for in-kernel timelines (development builds only: -DADA_TRACE).
#ifdef ADA_TRACE
__device__ unsigned long long g_trace[160 * 64];
#define TRACE(slot) do { g_trace[blockIdx.x * 64 + (slot)] = tc::global_ns(); } while (0)
#else
#define TRACE(slot) do { } while (0)
#endif

namespace {

constexpr int PM = 2 * BM;     // rows of a pair tile
// A ring stage holds KSUB consecutive 64-element K blocks (each its own 128-byte-swizzled
// sub-tile), so that the per-stage costs -- barrier round trips, fences, commit -- are paid
// once per 128 K elements and the MMA issue stays ahead of the tensor pipe.
constexpr int KSUB = 2;
constexpr int BKS = BK * KSUB; // K elements per stage

// ---------------------------------------------------------------- PTX, pair forms
__device__ __forceinline__ unsigned cluster_rank() {
    unsigned r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory location in CTA `rank` of this cluster
__device__ __forceinline__ unsigned map_to_cta(unsigned addr, unsigned rank) {
    unsigned r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_remote(unsigned cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr)
                 : "memory");
}
// TMA load whose completion bytes go to the LEADER's barrier: bit 24 of a shared::cluster
// address selects the CTA within the pair, clearing it names the even (leader) CTA.
__device__ __forceinline__ void tma_load_3d_pair(const CUtensorMap* map, unsigned long long* bar,
                                                 void* dst, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<unsigned long long>(map)),
          "r"(smem_u32(bar) & 0xFEFFFFFFu), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(unsigned tmem_d, unsigned long long adesc,
                                               unsigned long long bdesc, unsigned idesc,
                                               unsigned accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// commit: arrive on the barrier at this offset in BOTH CTAs once the MMAs issued so far retire
__device__ __forceinline__ void umma_commit_pair_both(unsigned long long* bar) {
    const unsigned short mask = 3;
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(smem_u32(bar)), "h"(mask)
        : "memory");
}
__device__ __forceinline__ void umma_commit_pair_local(unsigned long long* bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(smem_u32(bar))
                 : "memory");
}
// instruction descriptor of the pair MMA: M = 256
__device__ __forceinline__ unsigned instr_desc_pair(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((unsigned)(n >> 3) << 17) | ((unsigned)(PM >> 4) << 24);
}

// ---------------------------------------------------------------- tile list (256-row tiles)
__device__ __forceinline__ int seq_n(const GramProblem& p, int b) {
    int n = p.n_dev != nullptr ? p.n_dev[b] : p.n_host;
    if (p.n_clamp) n = min(max(n, 0), p.cap);
    return n;
}
__device__ __forceinline__ int tri_tiles(int n) {           // row pair P needs column tiles 0..P
    const int M = (n + PM - 1) / PM;
    return M * (M + 1) / 2;
}
// column tiles of a cross problem with n columns.  With in-launch norms (inv_out) a sequence
// without columns still gets one (empty) column tile: its rows have to be read for their norms.
__device__ __forceinline__ void cross_cols(const GramProblem& p, int n, int& nct, int& w) {
    nct = (n + BN - 1) / BN;
    if (nct == 0 && p.inv_out != nullptr && n == 0) nct = 1;
    w = nct > 0 ? max(32, (((n + nct - 1) / nct) + 31) & ~31) : 0;    // each CTA holds w/2 columns: keep w/2 a multiple of 16
}
// rows of the cross segment's left operand for a sequence with n inherited tokens: all of
// X, or only the tokens outside the inherited set when those were copied out (compact)
__device__ __forceinline__ int cross_rows(const GramProblem& p, int n, bool compact) {
    return compact ? p.rows - n : p.rows;
}
// hrows: rows of the left operand per CTA in cross tiles (128, or fewer in the streaming form)
__device__ __forceinline__ int seg_tiles(const GramProblem& p, int hrows, bool compact) {
    int total = 0;
    for (int b = 0; b < p.B; ++b) {
        const int n = seq_n(p, b);
        if (p.tri) { if (n > 0) total += tri_tiles(n); }
        else {
            int nct, w;
            cross_cols(p, n, nct, w);
            total += ((cross_rows(p, n, compact) + 2 * hrows - 1) / (2 * hrows)) * nct;
        }
    }
    return total;
}
__device__ __forceinline__ bool decode_tile(const GramProblem& p, int hrows, bool compact, int id, Piece& t) {
    for (int b = 0; b < p.B; ++b) {
        const int n = seq_n(p, b);
        int cnt = 0, nct = 0, w = 0;
        if (p.tri) cnt = n > 0 ? tri_tiles(n) : 0;
        else {
            cross_cols(p, n, nct, w);
            cnt = ((cross_rows(p, n, compact) + 2 * hrows - 1) / (2 * hrows)) * nct;
        }
        if (id >= cnt) { id -= cnt; continue; }
        t.b = b;
        t.n = n;
        int nc;
        if (p.tri) {
            int mi = (int)((sqrtf(8.0f * (float)id + 1.0f) - 1.0f) * 0.5f);
            while (mi * (mi + 1) / 2 > id) --mi;
            while ((mi + 1) * (mi + 2) / 2 <= id) ++mi;
            t.row0 = mi * PM;
            t.col0 = (id - mi * (mi + 1) / 2) * BN;
            t.m = n;
            nc = min(n - t.col0, BN);
        } else {
            t.row0 = (id / nct) * 2 * hrows;
            t.col0 = (id % nct) * w;
            t.m = cross_rows(p, n, compact);
            nc = min(n - t.col0, w);
        }
        t.ncols = max(32, (nc + 31) & ~31);
        return true;
    }
    return false;
}
// per-CTA stage: the CTA's rows of A (a_bytes per 64-element K block, a multiple of 1024) and
// ncols/2 rows of B (in 64-row boxes)
__device__ __forceinline__ int a_bytes_of(int hrows) { return (hrows * 128 + 1023) & ~1023; }
__device__ __forceinline__ int sub_bytes_pair(int a_bytes, int ncols) {
    return a_bytes + (((ncols >> 1) + BOX_N - 1) / BOX_N) * BOX_BYTES;
}
__device__ __forceinline__ int stage_count(int sbytes, int a_bytes) {
    // the MMA reads 128 rows of A whatever was loaded: keep what it reads past a shorter tile
    // inside the ring
    return min(MAX_STAGES, (RING_BYTES - (A_BYTES - a_bytes)) / sbytes);
}

// Row norms of the cross segment's left operand (inv_out).  When one column tile covers all
// columns every row tile is loaded exactly once and the launch is bound by streaming them: the
// norms are then taken from the tiles in shared memory (`from_smem`; the stage release waits for
// the readers, which costs nothing while the tensor pipe idles).  With several column tiles the
// main loops are bound by the tensor pipe and by what an SM can draw from L2, a stage release
// that waits for readers slows them, and the helper warps read the rows with plain loads
// instead (X then stays resident in L2 between the column tiles anyway).
__device__ __forceinline__ bool norm_duty(const GramProblem& p, const Piece& pc, bool from_smem) {
    return from_smem && !p.tri && p.inv_out != nullptr && pc.col0 == 0;
}
// Under ADA_CROSS_CAUSAL a cross tile whose first (lowest) column token is not below the
// tile's last row has no admissible (row, column) pair: every role skips it, so neither
// its loads nor its MMAs are issued.  Column tokens ascend with the column index.  (A tile
// that has to yield row norms is never skipped.)
__device__ __forceinline__ bool dead_tile(const GramProblem& p, const Piece& pc, int hrows, bool from_smem,
                                          bool compact) {
    if (p.tri || !p.causal || p.col_token == nullptr || pc.n <= 0 || norm_duty(p, pc, from_smem)) return false;
    if (compact) return false;     // rows are compacted there: a row index is not a token index
    return p.col_token[(int64_t)pc.b * p.cap + pc.col0] >= pc.row0 + 2 * hrows;
}

struct GramMaps {
    CUtensorMap a[2], b[2];
    CUtensorMap ah;          // left operand of the cross segment in boxes of hb_rows rows
    CUtensorMap an;          // the rows outside a large inherited set (Xnon), 128-row boxes
};

// ---------------------------------------------------------------- the kernel
struct alignas(16) SharedPair {
    unsigned long long full[MAX_STAGES];
    unsigned long long empty[MAX_STAGES];
    unsigned long long consumed[MAX_STAGES];   // MMAs of a norm-duty stage retired: its A tile may be read
    unsigned long long tmem_full[2];
    unsigned long long tmem_empty[2];
    unsigned long long drain;
    unsigned tmem_base;
    int abort_flag;
    int tiles0, tiles1, hrows, one_col_tile, compact;
    unsigned norm_cnt[MAX_STAGES];             // norm warps done with a stage
    // per epilogue warp, so that staging needs no barrier across warps
    alignas(16) float col_scale[4][BN];
    alignas(16) int col_token[4][BN];
};
constexpr int SMEM_PAIR_BYTES = RING_BYTES + (int)sizeof(SharedPair) + 1024;
static_assert(SMEM_PAIR_BYTES <= 227 * 1024, "shared memory budget");
constexpr int SMEM_NORM_WARPS = 4;             // warps 6..9 read the A tiles

__global__ void __launch_bounds__(NUM_THREADS, 1)
k_gram_tc2(const __grid_constant__ GramMaps maps, const __grid_constant__ GramProblem seg0,
           const __grid_constant__ GramProblem seg1, const int nseg,
           const __grid_constant__ NormJob norms, const __grid_constant__ GatherJob gather,
           unsigned* __restrict__ dep_ctr, unsigned* __restrict__ status) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    SharedPair& sh = *reinterpret_cast<SharedPair*>(smem + RING_BYTES);
    volatile int* abort_flag = &sh.abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const unsigned rank = cluster_rank();            // 0 = leader
    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_STAGES; ++s) {
            mbar_init(&sh.full[s], 1);
            mbar_init(&sh.empty[s], 1);
            mbar_init(&sh.consumed[s], 1);
            sh.norm_cnt[s] = 0u;
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&sh.tmem_full[a], 1);
            mbar_init(&sh.tmem_empty[a], 8);      // four epilogue warps in each CTA
        }
        mbar_init(&sh.drain, 1);
        sh.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&sh.tmem_base)), "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    // everything above is local to the CTA; from here on the predecessor's results are read
    grid_dep_wait();
    if (threadIdx.x == 0) TRACE(0);
    if (threadIdx.x == 64) {
        // streaming form: one column tile covers the columns of every sequence, so the launch is
        // one pass over the rows of A and shorter row tiles put every pair to work
        const GramProblem& cx = (nseg > 1) ? seg1 : seg0;
        int hrows = BM;
        bool one = !cx.tri;
        if (one)
            for (int b = 0; b < cx.B; ++b) one = one && seq_n(cx, b) <= BN;
        if (one && cx.hb_rows > 0 && cx.hb_rows < BM) hrows = cx.hb_rows;
        // a large inherited set (two fifths of the tokens or more, in every sequence) of a long
        // sequence: the rows outside it are copied out by the gather and the cross tiles run over
        // those only.  (Measured on the crossover sweep at r/T = 0.5: 1052 -> 699 us at T = 16384,
        // 250 -> 217 us at T = 8192, but 87 -> 97 us at T = 4096, where the copy costs more than
        // the saved tiles.)
        bool compact = !cx.tri && !one && gather.X != nullptr && gather.Xnon != nullptr && cx.rows >= gather.compact_min_rows;
        if (compact)
            for (int b = 0; b < cx.B; ++b) compact = compact && 5 * (int64_t)seq_n(cx, b) >= 2 * (int64_t)cx.rows;
        sh.hrows = hrows;
        sh.one_col_tile = one ? 1 : 0;
        sh.compact = compact ? 1 : 0;
        sh.tiles0 = seg_tiles(seg0, hrows, compact);
        sh.tiles1 = nseg > 1 ? seg_tiles(seg1, hrows, compact) : 0;
    }
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();          // the peer's barriers exist before anything signals them
    tcgen05_fence_after();
    const unsigned tmem_base = sh.tmem_base;
    const int tiles0 = sh.tiles0, total = sh.tiles0 + sh.tiles1;
    const int hrows = sh.hrows;                          // rows per CTA of a cross tile
    const bool smem_norms = sh.one_col_tile != 0;        // row norms out of the tiles in shared memory
    const bool compact = sh.compact != 0;                // cross tiles over the copied-out rows (Xnon)
    // the helper warps AND the epilogue warps (idle until the first tile is done) share the gather
    constexpr int GATHER_WARPS = NORM_WARPS + 4;
    const unsigned gather_total = (unsigned)(gridDim.x * GATHER_WARPS);
    const bool has_gather = gather.X != nullptr;
    Piece pc;
    if (threadIdx.x == 0) TRACE(1);

    if (warp == 0) {
        // ------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            unsigned fills = 0, used = 0, ever = 0;
            int cur_sb = 0, cur_nst = 0, s = 0;
            bool ok = true;
            // the right operand (and the triangle's left operand) is the gathered copy
            if (has_gather && total > 0) {
                ok = wait_counter_1(dep_ctr + 3, gather_total, abort_flag, 12);
                asm volatile("fence.proxy.async.global;" ::: "memory");
            }
            TRACE(3);
            for (int id = pair; ok && id < total; id += npairs) {
                const int sg = id < tiles0 ? 0 : 1;
                const GramProblem& p = sg ? seg1 : seg0;
                if (!decode_tile(p, hrows, compact, id - (sg ? tiles0 : 0), pc)) break;
                if (dead_tile(p, pc, hrows, smem_norms, compact)) continue;   // causal cross tile with no admissible pair
                const int num_kb = (p.d + BKS - 1) / BKS;
                const int half = pc.ncols >> 1;
                const int nbox = (half + BOX_N - 1) / BOX_N;
                const int arows = p.tri ? BM : hrows;
                const int a_bytes = a_bytes_of(arows);
                const int subb = sub_bytes_pair(a_bytes, pc.ncols);
                const int sb = KSUB * subb;
                const unsigned tx = (unsigned)(KSUB * (arows * 128 + nbox * BOX_BYTES));
                const CUtensorMap* amap = p.tri ? &maps.a[sg] : (compact ? &maps.an : (hrows != BM ? &maps.ah : &maps.a[sg]));
                if (sb != cur_sb) {
                    for (int q = 0; q < cur_nst && ok; ++q)
                        if ((used >> q) & 1u)
                            ok = mbar_wait(&sh.empty[q], ((fills >> q) & 1u) ^ 1u, abort_flag, 6);
                    if (!ok) break;
                    cur_sb = sb; cur_nst = stage_count(sb, a_bytes); s = 0; used = 0;
                }
                const int a_row = pc.row0 + (int)rank * arows;
                const int b_row = pc.col0 + (int)rank * half;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(&sh.empty[s], ((fills >> s) & 1u) ^ 1u, abort_flag, 1)) { ok = false; break; }
                    unsigned char* sa = smem + s * sb;
                    // the leader's barrier counts the bytes of both CTAs
                    if (rank == 0) mbar_expect_tx(&sh.full[s], 2u * tx);
                    // K blocks past d are zero-filled by the TMA unit
#pragma unroll
                    for (int u = 0; u < KSUB; ++u) {
                        unsigned char* su = sa + u * subb;
                        const int k0 = kb * BKS + u * BK;
                        tma_load_3d_pair(amap, &sh.full[s], su, k0, a_row, pc.b);
                        for (int j = 0; j < nbox; ++j)
                            tma_load_3d_pair(&maps.b[sg], &sh.full[s], su + a_bytes + j * BOX_BYTES, k0,
                                             b_row + j * BOX_N, pc.b);
                    }
                    fills ^= 1u << s; used |= 1u << s; ever |= 1u << s;
                    s = (s + 1 == cur_nst) ? 0 : s + 1;
                }
            }
            // drain: a stage's release (empty) implies its copy landed and was consumed
            for (int q = 0; q < MAX_STAGES; ++q) {
                if (!((ever >> q) & 1u)) continue;
                const unsigned ph = ((fills >> q) & 1u) ^ 1u;
                const unsigned long long t0 = global_ns();
                while (!mbar_try(&sh.empty[q], ph)) {
                    if (*abort_flag != 0 || global_ns() - t0 > WAIT_LIMIT_NS / 2) { *abort_flag = 7; break; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer (leader CTA only)
        if (lane == 0 && rank == 0) {
            unsigned uses = 0, tile_it = 0;
            int cur_sb = 0, cur_nst = 0, s = 0;
            bool ok = true;
            for (int id = pair; ok && id < total; id += npairs) {
                const int sg = id < tiles0 ? 0 : 1;
                const GramProblem& p = sg ? seg1 : seg0;
                if (!decode_tile(p, hrows, compact, id - (sg ? tiles0 : 0), pc)) break;
                if (dead_tile(p, pc, hrows, smem_norms, compact)) continue;   // causal cross tile with no admissible pair
                const int num_kb = (p.d + BKS - 1) / BKS;
                const int a_bytes = a_bytes_of(p.tri ? BM : hrows);
                const int subb = sub_bytes_pair(a_bytes, pc.ncols);
                const int sb = KSUB * subb;
                if (sb != cur_sb) { cur_sb = sb; cur_nst = stage_count(sb, a_bytes); s = 0; }
                const bool duty = norm_duty(p, pc, smem_norms);
                const unsigned acc = tile_it & 1u, acc_ph = (tile_it >> 1) & 1u;
                ++tile_it;
                if (!mbar_wait(&sh.tmem_empty[acc], acc_ph ^ 1u, abort_flag, 2)) { ok = false; break; }
                tcgen05_fence_after();
                const unsigned idesc = instr_desc_pair(pc.ncols);
                const unsigned d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(&sh.full[s], (uses >> s) & 1u, abort_flag, 3)) { ok = false; break; }
                    if (tile_it == 1 && kb == 0) TRACE(5);
                    tcgen05_fence_after();
#pragma unroll
                    for (int u = 0; u < KSUB; ++u) {
                        const unsigned a_addr = smem_u32(smem + s * sb + u * subb);
                        const unsigned long long adesc = smem_desc_sw128(a_addr);
                        const unsigned long long bdesc = smem_desc_sw128(a_addr + a_bytes);
#pragma unroll
                        for (int k = 0; k < BK / UMMA_K; ++k)
                            umma_bf16_pair(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | u | k) != 0);
                    }
                    // both producers may refill this stage -- after the norm warps have read the
                    // A tiles, where those yield the row norms
                    umma_commit_pair_both(duty ? &sh.consumed[s] : &sh.empty[s]);
                    uses ^= 1u << s;
                    s = (s + 1 == cur_nst) ? 0 : s + 1;
                }
                if (ok) umma_commit_pair_both(&sh.tmem_full[acc]);   // both epilogues may read
                TRACE(8 + 2 * (int)min(tile_it - 1, 8u));
            }
            TRACE(6);
            umma_commit_pair_local(&sh.drain);
            const unsigned long long t0 = global_ns();
            while (!mbar_try(&sh.drain, 0)) {
                if (global_ns() - t0 > WAIT_LIMIT_NS / 2) { *abort_flag = 8; break; }
            }
        }
    } else if (warp < 6) {
        // ------------------------------------------------ epilogue (warps 2..5, both CTAs)
        const int quad = warp & 3;
        float* cs = sh.col_scale[warp - 2];
        int* ct = sh.col_token[warp - 2];
        const unsigned dep_total = 8u * (unsigned)tiles0;
        bool dep_ok = !(nseg > 1 && tiles0 > 0);
        bool norm_ok = norms.X == nullptr;           // row norms computed by this launch's norm warps
        bool gather_ok = !has_gather;
        const unsigned norm_total = (unsigned)(gridDim.x * NORM_WARPS);
        if (has_gather)               // Algorithm 1 lines 1-2, shared with the helper warps
            gather_rows(gather, blockIdx.x * GATHER_WARPS + NORM_WARPS + (warp - 2), gridDim.x * GATHER_WARPS,
                        lane, dep_ctr + 3, status, compact);
        // the accumulator goes back to the leader's barrier
        const unsigned empty_addr[2] = {map_to_cta(smem_u32(&sh.tmem_empty[0]), 0),
                                        map_to_cta(smem_u32(&sh.tmem_empty[1]), 0)};
        unsigned tile_it = 0;
        for (int id = pair; id < total; id += npairs) {
            const int sg = id < tiles0 ? 0 : 1;
            const GramProblem& p = sg ? seg1 : seg0;
            if (!decode_tile(p, hrows, compact, id - (sg ? tiles0 : 0), pc)) break;
            if (dead_tile(p, pc, hrows, smem_norms, compact)) continue;   // causal cross tile with no admissible pair
            const unsigned acc = tile_it & 1u, acc_ph = (tile_it >> 1) & 1u;
            ++tile_it;
            const int64_t o = (int64_t)pc.b * p.cap;
            const int ncols = pc.ncols;
            if (!gather_ok) {
                // the gathered rows' inverse norms (column factors, and the triangle's row factors)
                if (!wait_counter(dep_ctr + 3, gather_total, lane, abort_flag, 13)) break;
                gather_ok = true;
            }
            if (sg == 1 && !dep_ok) {
                // every triangular tile of this launch first (line 5 before line 7)
                if (!wait_counter(dep_ctr, dep_total, lane, abort_flag, 5)) break;
                dep_ok = true;
                if (warp == 2 && lane == 0) TRACE(4);
            }
            if (p.wait_norm_b && !norm_ok) {
                if (!wait_counter(dep_ctr + 1, norm_total, lane, abort_flag, 9)) break;
                norm_ok = true;
            }
            __syncwarp();
            {
                // all of the tile's global loads are issued before the first is used (columns
                // past the tile are clamped to its last one and discarded afterwards, so that
                // no load hangs on a data-dependent branch): eight dependent round trips to L2
                // would otherwise sit on the path from a finished accumulator to its maxima
                float fb[BN / 32];
                unsigned gate[BN / 32] = {};
                int tk[BN / 32] = {};
                const int last = max(pc.n - 1, 0);
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
                    const bool live = col < pc.n;
                    if (c < ncols) {
                        cs[c] = (live && (p.tri || gate[q] < thr_b)) ? fb[q] : 0.f;
                        ct[c] = (live && !p.tri && p.causal) ? tk[q] : col;
                    }
                }
            }
            __syncwarp();
            // this thread's row: its role and inverse norm are fetched while the MMAs finish
            const int arows = p.tri ? BM : hrows;
            const int lrow = quad * 32 + lane;
            const int row_base = pc.row0 + (int)rank * arows;
            const int row = row_base + lrow;
            bool row_live = lrow < arows && row < pc.m;
            // the token this row belongs to: the row index itself, except over the copied-out rows
            // (an entry the gather did not write -- possible only with a rejected list -- is
            // never used as an index)
            int tokrow = row;
            if (compact && !p.tri && row_live) {
                tokrow = __ldcg(gather.non_tok + o + row);
                if ((unsigned)tokrow >= (unsigned)p.cap) { tokrow = row; row_live = false; }
            }
            const bool defer = !p.tri && p.defer_row != 0;   // the row's own factor is applied later
            // inherited reps are not candidates (with a deferred factor the compaction ignores them)
            const bool skip = row_live && !p.tri && !defer && p.row_role[o + row] != 0;
            const bool inv_early = !(p.wait_norm_a && !norm_ok);
            float inv_row = defer ? 1.0f : ((row_live && inv_early) ? __ldcg(p.inv_a + o + row) : 0.f);
            const bool got = mbar_wait(&sh.tmem_full[acc], acc_ph, abort_flag, 4);
            if (!__all_sync(0xffffffffu, got)) break;
            tcgen05_fence_after();
            const bool need_cmp = p.tri ? (pc.col0 + ncols > row_base) : (p.causal != 0);
            float mx = 0.f;
            // (a warp whose 32 rows lie past a short tile's rows still joins the aligned loads)
            for (int c0 = 0; c0 < ncols; c0 += 32) {
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
                        if (ct[c0 + j] < tokrow) mx = fmaxf(mx, x);
                    }
                }
            }
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(empty_addr[acc]);
            if (!defer && p.wait_norm_a && !norm_ok) {
                if (!wait_counter(dep_ctr + 1, norm_total, lane, abort_flag, 9)) break;
                norm_ok = true;
            }
            if (row_live) {
                if (!skip) {
                    if (!defer && !inv_early) inv_row = __ldcg(p.inv_a + o + row);
                    mx *= inv_row;
                    if (mx > 0.f) atomicMax(p.out + o + tokrow, __float_as_uint(mx));
                }
            }
            if (sg == 0 && nseg > 1) {
                __threadfence();
                __syncwarp();
                if (lane == 0) atomicAdd(dep_ctr, 1u);
            }
            if (warp == 2 && lane == 0) TRACE(9 + 2 * (int)min(tile_it - 1, 8u));
        }
    } else {
        // ------------------------------------------------ helper warps (6 and up)
        if (norms.X != nullptr)       // full selection: row norms with plain loads
            norm_rows(norms, blockIdx.x * NORM_WARPS + (warp - 6), gridDim.x * NORM_WARPS, lane,
                      dep_ctr + 1, status);
        if (has_gather)               // Algorithm 1 lines 1-2
            gather_rows(gather, blockIdx.x * GATHER_WARPS + (warp - 6), gridDim.x * GATHER_WARPS, lane,
                        dep_ctr + 3, status, compact);
        if (warp == 6 && lane == 0) TRACE(2);
        const GramProblem& cx = (nseg > 1) ? seg1 : seg0;
        if (!cx.tri && cx.inv_out != nullptr && !smem_norms && !compact) {
            // several column tiles: 1/||x_t|| of every row with plain loads, behind the main loops
            // (nothing in this launch waits for them: the row factor is applied by the compaction)
            NormJob nj;
            nj.X = cx.A; nj.ldx = cx.lda; nj.n_rows = (int64_t)cx.B * cx.rows; nj.d = cx.d;
            nj.inv_norm = cx.inv_out;
            nj.batch = cx.a_batch; nj.rows_per_seq = cx.rows;
            norm_rows(nj, blockIdx.x * NORM_WARPS + (warp - 6), gridDim.x * NORM_WARPS, lane,
                      dep_ctr + 1, status);
        } else if (warp < 6 + SMEM_NORM_WARPS && !cx.tri && cx.inv_out != nullptr) {
            // row norms of X out of the A tiles in shared memory: thread lrow owns row lrow of
            // the CTA's tile; this role follows the ring exactly as the producer fills it
            const int lrow = (warp - 6) * 32 + lane;
            unsigned cons = 0;
            int cur_sb = 0, cur_nst = 0, s = 0;
            bool ok = true;
            for (int id = pair; ok && id < total; id += npairs) {
                const int sg = id < tiles0 ? 0 : 1;
                const GramProblem& p = sg ? seg1 : seg0;
                if (!decode_tile(p, hrows, compact, id - (sg ? tiles0 : 0), pc)) break;
                if (dead_tile(p, pc, hrows, smem_norms, compact)) continue;
                const int num_kb = (p.d + BKS - 1) / BKS;
                const int arows = p.tri ? BM : hrows;
                const int a_bytes = a_bytes_of(arows);
                const int subb = sub_bytes_pair(a_bytes, pc.ncols);
                const int sb = KSUB * subb;
                if (sb != cur_sb) { cur_sb = sb; cur_nst = stage_count(sb, a_bytes); s = 0; }
                if (!norm_duty(p, pc, smem_norms)) { s = (s + num_kb) % cur_nst; continue; }
                float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
                for (int kb = 0; kb < num_kb; ++kb) {
                    int good = 1;
                    if (lane == 0) good = mbar_wait(&sh.consumed[s], (cons >> s) & 1u, abort_flag, 14) ? 1 : 0;
                    if (__shfl_sync(0xffffffffu, good, 0) == 0) { ok = false; break; }
                    if (lrow < arows) {
#pragma unroll
                        for (int u = 0; u < KSUB; ++u) {
                            // the 16-byte chunks of a row are permuted by the swizzle, which a sum
                            // of squares need not undo; lanes start at different chunks so that a
                            // warp's loads spread over all banks
                            const unsigned char* rowp = smem + s * sb + u * subb + lrow * 128;
                            uint4 x[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                x[j] = *reinterpret_cast<const uint4*>(rowp + (((j + lane) & 7) << 4));
                            s0 += sumsq_bf16x8(x[0]) + sumsq_bf16x8(x[4]);
                            s1 += sumsq_bf16x8(x[1]) + sumsq_bf16x8(x[5]);
                            s2 += sumsq_bf16x8(x[2]) + sumsq_bf16x8(x[6]);
                            s3 += sumsq_bf16x8(x[3]) + sumsq_bf16x8(x[7]);
                        }
                    }
                    __syncwarp();
                    // the last of the four warps releases the stage to the producer
                    if (lane == 0) {
                        if (atomicAdd(&sh.norm_cnt[s], 1u) == SMEM_NORM_WARPS - 1) {
                            sh.norm_cnt[s] = 0u;
                            mbar_arrive(&sh.empty[s]);
                        }
                    }
                    cons ^= 1u << s;
                    s = (s + 1 == cur_nst) ? 0 : s + 1;
                }
                if (!ok) break;
                const int row = pc.row0 + (int)rank * arows + lrow;
                if (lrow < arows && row < pc.m) {
                    const float ss = (s0 + s1) + (s2 + s3);
                    float inv = 0.f;
                    if (!(ss <= 3.0e38f)) atomicOr(status, ST_NONFINITE);
                    else if (ss > 0.f) inv = 1.0f / sqrtf(ss);
                    else atomicAdd(status + 1, 1u);
                    p.inv_out[(int64_t)pc.b * p.cap + row] = inv;
                }
                if (lrow == 0) TRACE(40);
            }
        }
    }

    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();          // neither CTA frees TMEM or exits while the other may still touch it
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                     "r"(TMEM_COLS)
                     : "memory");
    }
    if (threadIdx.x == 0 && sh.abort_flag != 0) {
        atomicOr(status, ST_TIMEOUT);
        status[2] = 100u + (unsigned)sh.abort_flag;
    }
    if (threadIdx.x == 0) TRACE(63);
}

}  // namespace

static cudaError_t ensure_tc2(ada_ctx* ctx) {
    if (ctx->tc2_attr_set) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(k_gram_tc2, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         SMEM_PAIR_BYTES);
    if (e != cudaSuccess) return e;
    // how many clusters of two fit on the device at once
    cudaLaunchConfig_t q;
    memset(&q, 0, sizeof(q));
    q.gridDim = dim3(2 * (ctx->sm_count / 2));
    q.blockDim = dim3(NUM_THREADS);
    q.dynamicSmemBytes = SMEM_PAIR_BYTES;
    cudaLaunchAttribute qa[1];
    qa[0].id = cudaLaunchAttributeClusterDimension;
    qa[0].val.clusterDim.x = 2; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
    q.attrs = qa; q.numAttrs = 1;
    int nclusters = 0;
    e = cudaOccupancyMaxActiveClusters(&nclusters, k_gram_tc2, &q);
    if (e != cudaSuccess || nclusters < 1) { cudaGetLastError(); return cudaErrorLaunchOutOfResources; }
    ctx->tc2_pairs = nclusters < ctx->sm_count / 2 ? nclusters : ctx->sm_count / 2;
    ctx->tc2_attr_set = true;
    return cudaSuccess;
}

// Rows of X per CTA for a cross-Gram whose columns fit one column tile (at most 256
// representatives per sequence): such a launch is one pass over X, so the row tiles are cut to
// give every SM pair but the ones that take the small triangular problems a share.  128 = the
// ordinary tile.  (0 if the kernel cannot be configured.)
int gram_tc2_hb_rows(ada_ctx* ctx, int B, int T) {
    if (ensure_tc2(ctx) != cudaSuccess) return 0;
    const int free_pairs = ctx->tc2_pairs - B;            // one triangular tile per sequence
    if (free_pairs < B) return BM;
    const int tiles_per_seq = free_pairs / B;
    int h = (T + 2 * tiles_per_seq - 1) / (2 * tiles_per_seq);
    if (h < 16) h = 16;
    return h >= BM ? BM : h;
}

// Pair-CTA launch.  tri and/or cross may be NULL; with both the cross epilogues wait in-kernel
// for the triangular segment (ctx->tile_ctr must be zero at launch).
cudaError_t launch_gram_tc2(ada_ctx* ctx, const GramProblem* tri, const GramProblem* cross,
                            const NormJob* norms, const GatherJob* gather, cudaStream_t s) {
    cudaError_t e0 = ensure_tc2(ctx);
    if (e0 != cudaSuccess) return e0;
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
        if (!make_map(&maps.a[nseg], p->A, p->d, p->tri ? p->cap : p->rows, p->B, p->lda, p->a_batch, BM) ||
            !make_map(&maps.b[nseg], p->Bm, p->d, p->cap, p->B, p->ldb, p->b_batch, BOX_N))
            return cudaErrorInvalidValue;
        if (!p->tri) {
            const int hb = (p->hb_rows > 0 && p->hb_rows < BM) ? p->hb_rows : BM;
            if (!make_map(&maps.ah, p->A, p->d, p->rows, p->B, p->lda, p->a_batch, hb))
                return cudaErrorInvalidValue;
        }
        segs[nseg++] = *p;
    }
    if (nseg == 0) return cudaSuccess;
    if (nseg == 1) { maps.a[1] = maps.a[0]; maps.b[1] = maps.b[0]; segs[1] = segs[0]; segs[1].B = 0; }
    if (segs[0].tri && nseg == 1) maps.ah = maps.a[0];
    maps.an = maps.ah;
    if (gather != nullptr && gather->Xnon != nullptr && cross != nullptr &&
        !make_map(&maps.an, gather->Xnon, cross->d, cross->rows, cross->B, cross->d, (int64_t)cross->cap * cross->d, BM))
        return cudaErrorInvalidValue;
    NormJob nj;
    memset(&nj, 0, sizeof(nj));
    if (norms != nullptr) nj = *norms;
    GatherJob gj;
    memset(&gj, 0, sizeof(gj));
    if (gather != nullptr) gj = *gather;
    const bool fused = nseg == 2;
    prof_begin(ctx, fused ? K_GRAM_TC_CASCADE : (segs[0].tri ? K_GRAM_TC_TRI : K_GRAM_TC_CROSS), s);
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(2 * ctx->tc2_pairs);
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = SMEM_PAIR_BYTES;
    cfg.stream = s;
    cudaLaunchAttribute attr[3];
    int na = 0;
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = 2; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = 1;
    ++na;
    // CTAs wait on results of other CTAs (triangle before cross epilogues, the gather before
    // everything): all of them have to be resident
    if ((fused || gj.X != nullptr) && ctx->cooperative) {
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
    cudaError_t e = cudaLaunchKernelEx(&cfg, k_gram_tc2, maps, segs[0], segs[1], nseg, nj, gj, ctx->tile_ctr,
                                       ctx->status);
    prof_end(ctx, s);
    return e;
}

}  // namespace ada

#ifdef ADA_TRACE
extern "C" int ada_trace_read(unsigned long long* host, int clear) {
    if (cudaMemcpyFromSymbol(host, ada::g_trace, sizeof(ada::g_trace)) != cudaSuccess) return 1;
    if (clear) {
        static unsigned long long zeros[160 * 64];
        if (cudaMemcpyToSymbol(ada::g_trace, zeros, sizeof(zeros)) != cudaSuccess) return 2;
    }
    return 0;
}
#endif
