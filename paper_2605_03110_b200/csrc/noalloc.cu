// Full selection without any allocation: the scratch lives in a fixed device array that is
// part of the library image.
//
// Meant for callers that must not allocate device memory when they call in: a serving
// process that handed all of HBM to its own pool at start-up (a later cudaMalloc fails or
// fragments that pool), a latency-critical loop that cannot afford the device-wide
// synchronisation an allocation implies, or a plug-in whose host application forbids
// allocator calls.  Such callers cannot create an ada_ctx, whose workspace is one cudaMalloc.
#include <string.h>

#include <mutex>

#include "common.cuh"

using namespace ada;

namespace {

// gamma bit patterns [ADA_NOALLOC_MAX_T] | inverse norms [ADA_NOALLOC_MAX_T] | status words,
// counters and the compaction's 16 published block counts (256 bytes)
constexpr size_t kGammaBytes = (size_t)ADA_NOALLOC_MAX_T * 4;
constexpr size_t kInvBytes = (size_t)ADA_NOALLOC_MAX_T * 4;
constexpr size_t kTailBytes = 256;
constexpr size_t kScratchBytes = kGammaBytes + kInvBytes + kTailBytes;

// Held by every GPU that loads the library, from module load to process exit (about 128 KiB).
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 16;
struct PerDevice {
    std::once_flag once;
    ada_status setup_status;
    unsigned char* scratch;   // device address of g_noalloc_scratch on this device
    ada_ctx ctx;              // host-side bookkeeping only; owns no memory; written once, at set-up
};
PerDevice g_dev[kMaxDevices];

// One-time set-up for the current device (guarded: two host threads may make their first call
// at once).  In host code the array's name is only a handle: the address a kernel can use has
// to be asked for, with this device current.
ada_status setup_device(int device, PerDevice** out) {
    if (device < 0 || device >= kMaxDevices) return ADA_ERR_UNSUPPORTED;
    PerDevice& pd = g_dev[device];
    std::call_once(pd.once, [&pd, device]() {
        pd.setup_status = ADA_ERR_CUDA;
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return;
        }
        pd.scratch = static_cast<unsigned char*>(ptr);
        ada_ctx& c = pd.ctx;
        c.device = device;
        c.maxB = 1;
        c.maxT = ADA_NOALLOC_MAX_T;
        c.maxd = 0;
        c.dt = ADA_BF16;               // unused: the storage type travels as an argument
        c.es = 2;
        c.engine = ADA_ENGINE_AUTO;
        c.tc_attr_set = false;
        c.cooperative = true;
        c.dep_launch = false;          // plain stream order between this call's launches
        c.compact_min_rows = 0x7fffffff;
        c.tc2_attr_set = false;
        c.tc2_pairs = 0;
        c.ws = nullptr;
        c.attn_ws = nullptr;
        c.attn_ws_bytes = 0;
        c.stage = nullptr;
        c.stage_bytes = 0;
        c.host_stream = nullptr;
        if (cudaDeviceGetAttribute(&c.sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess)
            return;
        c.g_tok = reinterpret_cast<unsigned*>(pd.scratch);
        c.inv_norm = reinterpret_cast<float*>(pd.scratch + kGammaBytes);
        c.status = reinterpret_cast<unsigned*>(pd.scratch + kGammaBytes + kInvBytes);
        c.tile_ctr = c.status + 8;                                           // +32 bytes
        c.done_ctr = c.status + 16;                                          // +64 bytes
        c.agg = reinterpret_cast<unsigned long long*>(c.status + 32);        // +128 bytes: 16 words
        c.agg_stride = ADA_NOALLOC_MAX_T / 1024;
        c.g_rep = nullptr;
        c.inv_rep = nullptr;
        c.role = nullptr;
        c.r_eff = nullptr;
        c.thr_seq = nullptr;
        c.Xrep = nullptr;
        c.Xnon = nullptr;
        c.non_tok = nullptr;
        c.near_key = nullptr;
        c.splitXA = c.splitXB = c.splitRA = c.splitRB = nullptr;
        pd.setup_status = ADA_OK;
    });
    *out = &pd;
    return pd.setup_status;
}

}  // namespace

extern "C" ada_status ada_select_full_noalloc(const void* X, int64_t T, int64_t d, int64_t ldx,
                                              ada_dtype dt, double tau, int32_t* rep_idx,
                                              int32_t* rep_cnt, float* gamma, void* stream) {
    if (X == nullptr || rep_idx == nullptr || rep_cnt == nullptr) return ADA_ERR_INVALID_ARG;
    if (T < 1 || d < 1 || ldx < d || !(tau > 0.0 && tau < 1.0)) return ADA_ERR_INVALID_ARG;
    if (dt != ADA_F32 && dt != ADA_BF16) return ADA_ERR_INVALID_ARG;
    if (T > ADA_NOALLOC_MAX_T) return ADA_ERR_WORKSPACE;   // the fixed scratch holds ADA_NOALLOC_MAX_T tokens
    const int64_t es = dt == ADA_F32 ? 4 : 2;
    if ((reinterpret_cast<uintptr_t>(X) & 15u) != 0 || (ldx * es) % 16 != 0 || (d * es) % 16 != 0)
        return ADA_ERR_UNSUPPORTED;
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) return ADA_ERR_CUDA;
    PerDevice* pd = nullptr;
    ada_status st = setup_device(device, &pd);
    if (st != ADA_OK) return st;
    ada_ctx* ctx = &pd->ctx;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const float thr = (float)(1.0 - tau * tau);

    // The array keeps whatever the previous call (or a faulted one) left: clear the part
    // that must start at zero -- the gamma bit patterns and the status/counter words.
    if (cudaMemsetAsync(ctx->g_tok, 0, (size_t)T * 4, s) != cudaSuccess) return ADA_ERR_CUDA;
    if (cudaMemsetAsync(ctx->status, 0, kTailBytes, s) != cudaSuccess) return ADA_ERR_CUDA;
    if (launch_norm_gather(ctx, X, 1, (int)T, (int)d, ldx, T * ldx, dt, ctx->inv_norm, nullptr, nullptr,
                           nullptr, nullptr, nullptr, nullptr, nullptr, s) != cudaSuccess)
        return ADA_ERR_CUDA;
    GramProblem p;
    memset(&p, 0, sizeof(p));
    p.A = X; p.Bm = X;
    p.lda = ldx; p.ldb = ldx;
    p.a_batch = T * ldx; p.b_batch = T * ldx;
    p.inv_a = ctx->inv_norm; p.inv_b = ctx->inv_norm;
    p.out = ctx->g_tok;
    p.n_dev = nullptr; p.n_host = (int)T;
    p.rows = (int)T; p.cap = (int)T; p.d = (int)d; p.B = 1;
    p.tri = 1;
    cudaError_t e;
    if (dt == ADA_BF16 && gram_tc_available()) e = launch_gram_tc(ctx, &p, nullptr, nullptr, s);
    else e = launch_gram_ffma(ctx, p, dt, s);
    if (e != cudaSuccess) return ADA_ERR_CUDA;
    if (launch_compact_full(ctx, 1, (int)T, thr, rep_idx, rep_cnt, gamma, s) != cudaSuccess)
        return ADA_ERR_CUDA;
    return ADA_OK;
}
