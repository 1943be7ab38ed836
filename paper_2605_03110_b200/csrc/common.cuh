// Internal declarations shared by the translation units of libada.so.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include "../../include/ada.h"

namespace ada {

// bits of the device status word (status[0])
enum : unsigned {
    ST_BAD_INDEX = 1u << 0,  // inherited list not strictly ascending / out of [0,T)
    ST_BAD_COUNT = 1u << 1,  // a count outside [0,T]
    ST_NONFINITE = 1u << 2,  // NaN / Inf met while normalising
    ST_TIMEOUT = 1u << 3,    // a bounded wait in a kernel ran out
    ST_BAD_TAU = 1u << 4,    // a device-resident threshold state outside (0,1)
};
// status[1] counts zero-norm rows, status[2] records where a wait gave up.

enum KernelId {
    K_NORM_GATHER = 0,
    K_GRAM_FFMA_TRI,
    K_GRAM_FFMA_CROSS,
    K_GRAM_TC_TRI,
    K_GRAM_TC_CROSS,
    K_GRAM_TC_CASCADE,
    K_SPLIT,
    K_COMPACT_FULL,
    K_COMPACT_CASCADE,
    K_NEAREST_FINISH,
    K_COUNT
};

// One masked-Gram-with-row-maximum problem, batched over B sequences.
//   C(i,j) = a_i . b_j           a_i = row i of A, b_j = row j of Bm (both K-major)
//   v(i,j) = |C(i,j)| * inv_a[i] * inv_b[j]
//   out[i] = max over admissible j of v(i,j), combined with atomicMax on the
//            IEEE bit pattern (v >= 0, so unsigned order == float order)
// tri  : A == Bm, admissible j < i, i < n
// cross: rows i < T of X against columns j < n of the gathered representative
//        rows; admissible iff col_gate[j] < thr_bits (the representative is
//        valid) and, when causal, col_token[j] < i; rows with row_role[i] != 0
//        (inherited representatives) produce nothing.
struct GramProblem {
    const void* A;            // rows of the left operand
    const void* Bm;           // rows of the right operand
    int64_t lda, ldb;         // row strides in elements
    int64_t a_batch, b_batch; // batch strides in elements
    const float* inv_a;       // [B*cap]
    const float* inv_b;       // [B*cap]
    unsigned* out;            // [B*cap] gamma bit patterns (zero-initialised)
    const int32_t* n_dev;     // [B] device-resident column/row count, or NULL
    int n_host;               // used when n_dev == NULL
    int rows;                 // number of A rows (cross); ignored for tri
    int cap;                  // per-sequence capacity (= T) of the per-token arrays
    int d;                    // contraction length
    int B;
    int tri;                  // 1: lower-triangular self Gram, 0: cross
    // cross only
    const unsigned* col_gate; // [B*cap] gamma_rep bits by position
    unsigned thr_bits;        // bit pattern of (float)thr
    const unsigned* thr_seq;  // per-sequence bit patterns instead (adaptive threshold), or NULL
    const int32_t* col_token; // [B*cap] token index of each column (causal) or NULL
    const int32_t* row_role;  // [B*cap] 0 for non-representatives
    int causal;
    // set when inv_a / inv_b are produced inside the same launch (NormJob): the epilogue
    // waits for the norm warps before it reads them
    int wait_norm_a, wait_norm_b;
    // nearest-representative mode (cross only): instead of `out`, combine per row the packed
    // key (value bits << 32 | ~column) with a 64-bit atomicMax: largest value, lowest column
    unsigned long long* out_arg;
    // n_dev holds the caller's raw counts: clamp them to [0, cap] (nobody has sanitised them yet)
    int n_clamp;
    // pair kernel, cross only -----------------------------------------------------------------
    // out[] receives the row maximum WITHOUT the factor inv_a[i] (a positive factor common to the
    // row commutes with the maximum, rounding included); the compaction applies it.  No row
    // norm is then needed inside the launch.
    int defer_row;
    // 1/||a_i|| of every row of A, computed from the A tiles while they sit in shared memory (by
    // the tiles of the first column tile) and stored here; NULL: not wanted
    float* inv_out;
    // rows of A per CTA when a single column tile covers every sequence's columns (a cross-Gram
    // bound by streaming A once: shorter row tiles put every SM pair to work); 0 or 128: 128
    int hb_rows;
};

// Algorithm 1 lines 1-2 inside a pair-kernel launch: the inherited list is validated, scattered
// into the role map, and its rows of X are copied (raw) to Xrep with their inverse norms, by
// spare warps of every CTA before the first tile; loads of Xrep and the epilogues wait for it.
// X == NULL: nothing to do.
struct GatherJob {
    const void* X;            // bf16 rows
    int64_t ldx, xb;          // row / sequence strides of X in elements
    const int32_t* rep_in;    // [B*T]
    const int32_t* rep_in_cnt;// [B]
    int32_t* role;            // [B*T] position + 1 of inherited tokens
    int32_t* r_eff;           // [B] sanitised counts
    void* Xrep;               // [B*T][d]
    float* inv_rep;           // [B*T] by position
    int T, d, B;
    // line 6's row set as a matrix of its own, made when the inherited set is large (see
    // gather_rows): rows outside the set in token order, their token indices, 1/||x_t|| by token
    void* Xnon;               // [B*T][d], or NULL: never
    int32_t* non_tok;         // [B*T]
    float* inv_norm;          // [B*T]
    int compact_min_rows;     // sequences shorter than this never use it
};

// Row norms computed inside a tensor-core Gram launch by four extra warps per CTA
// (Section 2.1; Algorithm 1 line 1): inv_norm[row] = 1/||x_row|| for all n_rows rows of X.
// X == NULL: nothing to do.
struct NormJob {
    const void* X;
    int64_t ldx;
    int64_t n_rows;
    int d;
    float* inv_norm;
    // rows_per_seq > 0: row i is row (i % rows_per_seq) of sequence (i / rows_per_seq), which
    // starts `batch` elements after the previous one; 0: rows are ldx apart throughout
    int64_t batch;
    int rows_per_seq;
};

struct Profiler {
    bool on = false;
    static const int MAXREC = 4096;
    cudaEvent_t ev0[MAXREC], ev1[MAXREC];
    int kid[MAXREC];
    int n = 0, created = 0;
};

}  // namespace ada

struct ada_ctx {
    int device;
    int64_t maxB, maxT, maxd;
    ada_dtype dt;
    int es;
    ada_engine engine;
    int sm_count;
    bool tc_attr_set;
    bool cooperative;    // fused launches use the cooperative attribute
    bool dep_launch;     // kernels are launched with programmatic stream serialization
    int compact_min_rows;  // sequence length from which a large inherited set's complement is copied out
    bool tc2_attr_set;   // pair-CTA kernel configured
    int tc2_pairs;       // clusters of two that fit on the device at once
    // device workspace
    char* ws;            // one allocation
    float* inv_norm;     // [maxB*maxT] 1/||x_t||
    float* inv_rep;      // [maxB*maxT] 1/||x|| of gathered rows, by position
    unsigned* g_tok;     // [maxB*maxT] gamma (full) or gamma_cross, by token, bit patterns
    unsigned* g_rep;     // [maxB*maxT] gamma_rep by position, bit patterns
    int32_t* role;       // [maxB*maxT] 0 = not inherited, p+1 = position p in the inherited list
    int32_t* r_eff;      // [maxB] sanitised inherited counts
    float* thr_seq;      // [maxB] per-sequence (float)(1 - tau^2) of an adaptive step
    unsigned* status;    // [8]
    unsigned* tile_ctr;  // [8] dependency counter of the fused Gram launch
    unsigned long long* agg;  // [maxB][agg_stride] block counts published by the compaction
    unsigned* done_ctr;  // compaction blocks finished
    int agg_stride;
    unsigned long long* near_key;  // [maxB*maxT] packed (value, ~column) of the nearest representative
    void* Xrep;          // [maxB*maxT*maxd] gathered representative rows (raw values)
    void* Xnon;          // [maxB*maxT*maxd] bf16 contexts: the rows outside a large inherited set
    int32_t* non_tok;    // [maxB*maxT] their token indices
    // fp32 contexts: three-term bf16 splits laid out for one contraction of length 6d
    void *splitXA, *splitXB;   // [maxB*maxT][6 maxd] of X
    void *splitRA, *splitRB;   // same, of the gathered representative rows
    // gathered Q_R, K_R, V_R^T of the attention on the representative set (allocated on first use)
    char* attn_ws;
    size_t attn_ws_bytes;
    // staging for the *_host entry points (allocated on first use)
    char* stage;
    size_t stage_bytes;
    cudaStream_t host_stream;
    ada::Profiler prof;
};

namespace ada {

// Programmatic dependent launch.  Every kernel of the library starts with grid_dep_wait()
// -- before any early return, so that a grid never completes ahead of its predecessor -- and is
// launched with the stream-serialization attribute: its blocks may be placed on an SM, and run
// what precedes the wait (barrier set-up, TMEM allocation), as soon as the blocks of the kernel
// before it in the stream have left, instead of after that whole grid has drained; the wait
// returns once the predecessor has completed and its writes are visible.  Without the
// attribute the wait is a no-op.
#ifdef __CUDACC__
static __device__ __forceinline__ void grid_dep_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
// Lets the next kernel's blocks be placed now instead of when this block exits (they still wait,
// in their own grid_dep_wait, for this whole grid to complete).  Worth it in kernels that leave
// most SMs idle or whose blocks are short.
static __device__ __forceinline__ void grid_dep_launch_next() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
#endif
template <typename... KArgs, typename... Args>
cudaError_t launch_k(ada_ctx* ctx, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                     cudaStream_t s, Args&&... args) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = ctx->dep_launch ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// RAII-free launch bracket used by every launcher.
void prof_begin(ada_ctx* ctx, int kid, cudaStream_t s);
void prof_end(ada_ctx* ctx, cudaStream_t s);

// prep_kernels.cu
cudaError_t launch_norm_gather(ada_ctx* ctx, const void* X, int B, int T, int d, int64_t ldx,
                               int64_t xb, ada_dtype dt, float* inv_norm, void* Xhat, const int32_t* rep_in,
                               const int32_t* rep_in_cnt, int32_t* role, int32_t* r_eff, void* Xrep,
                               float* inv_rep, cudaStream_t s);
cudaError_t launch_split(ada_ctx* ctx, const void* X, int B, int T, int d, int64_t ldx, int64_t xb,
                         bool with_rep, cudaStream_t s);
cudaError_t launch_nearest_finish(ada_ctx* ctx, int B, int T, const int32_t* rep_idx,
                                  int32_t* nearest_idx, float* nearest_gamma, cudaStream_t s);
cudaError_t launch_compact_full(ada_ctx* ctx, int B, int T, float thr, int32_t* rep_idx,
                                int32_t* rep_cnt, float* gamma, cudaStream_t s);
// adaptive threshold (Section 8.1): tau_state != NULL makes the step use ctx->thr_seq and update
// tau_state / write the turnover of Eq. (6) once the counts are known
struct TauUpdate {
    double* tau_state;     // [B] device, in/out; NULL = fixed threshold
    float* turnover;       // [B] device, optional
    int update;            // 0: leave tau_state as it is
    double target, gain, tau_min, tau_max;
};
cudaError_t launch_tau_thr(ada_ctx* ctx, int B, const double* tau_state, cudaStream_t s);
// row_scale: the cross maxima in the scratch still lack the factor 1/||x_t|| (GramProblem::defer_row)
cudaError_t launch_compact_cascade(ada_ctx* ctx, int B, int T, float thr, int32_t* rep_out,
                                   int32_t* rep_out_cnt, int32_t* add_idx, int32_t* add_cnt,
                                   int32_t* rem_idx, int32_t* rem_cnt, float* gamma_rep,
                                   float* gamma_cross, const TauUpdate& tu, bool row_scale,
                                   cudaStream_t s);

// gram_ffma.cu
cudaError_t launch_gram_ffma(ada_ctx* ctx, const GramProblem& p, ada_dtype dt, cudaStream_t s);

// gram_tc.cu (bf16, tcgen05 + TMA)
cudaError_t launch_gram_tc(ada_ctx* ctx, const GramProblem* tri, const GramProblem* cross,
                           const NormJob* norms, cudaStream_t s);
bool gram_tc_available();
cudaError_t launch_selftest_wait(ada_ctx* ctx, int limit_ms, cudaStream_t s);

// attn_reps.cu (Eq. 2 on the representative rows, both contractions on tcgen05)
cudaError_t launch_attention_reps(ada_ctx* ctx, const void* Q, const void* K, const void* V, int T, int h,
                                  int d_h, int64_t ld, const int32_t* rep_idx, const int32_t* rep_cnt,
                                  const int32_t* nearest_idx, float* out, int64_t ldo, int causal,
                                  cudaStream_t s);

// gram_tc2.cu (bf16, tcgen05.cta_group::2: two CTAs per 256-row tile)
cudaError_t launch_gram_tc2(ada_ctx* ctx, const GramProblem* tri, const GramProblem* cross,
                            const NormJob* norms, const GatherJob* gather, cudaStream_t s);
// rows of the left operand per CTA for a cross-Gram that a single column tile covers
int gram_tc2_hb_rows(ada_ctx* ctx, int B, int T);

}  // namespace ada
