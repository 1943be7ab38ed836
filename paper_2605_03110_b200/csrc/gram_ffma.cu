// fp32 FFMA masked-Gram kernel with the fused row-maximum epilogue.
//
// This is the FP32 path of the selection (Definition 1; Algorithm 1 lines 3-4
// and 7-8): products and sums are IEEE fp32 on the plain ALUs, so gamma agrees
// with an fp64 evaluation to ~1e-6.  It also accepts bf16 storage (widened
// exactly) as a slow cross-check of the tensor-core kernel.  The Gram tile
// lives in registers only; the epilogue applies 1/(|a_i||b_j|), |.|, the
// admissibility mask and the row maximum, and publishes one atomicMax per row
// and tile.
#include "common.cuh"

namespace ada {

namespace {

constexpr int BM = 64, BN = 64, BK = 16, LDS = BM + 4;

template <typename T>
__device__ __forceinline__ void load4(const T* p, float (&v)[4]);
template <>
__device__ __forceinline__ void load4<float>(const float* p, float (&v)[4]) {
    const float4 f = __ldg(reinterpret_cast<const float4*>(p));
    v[0] = f.x; v[1] = f.y; v[2] = f.z; v[3] = f.w;
}
template <>
__device__ __forceinline__ void load4<__nv_bfloat16>(const __nv_bfloat16* p, float (&v)[4]) {
    const uint2 u = __ldg(reinterpret_cast<const uint2*>(p));
    v[0] = __uint_as_float(u.x << 16); v[1] = __uint_as_float(u.x & 0xffff0000u);
    v[2] = __uint_as_float(u.y << 16); v[3] = __uint_as_float(u.y & 0xffff0000u);
}

template <typename T>
__global__ void __launch_bounds__(256)
k_gram_ffma(const GramProblem p) {
    grid_dep_wait();
    const int b = blockIdx.z;
    const int n = p.n_dev != nullptr ? p.n_dev[b] : p.n_host;   // columns (and rows when tri)
    const int m = p.tri ? n : p.rows;
    const int row0 = blockIdx.y * BM, col0 = blockIdx.x * BN;
    if (row0 >= m || col0 >= n) return;
    if (p.tri && col0 >= row0 + BM) return;                     // strictly above the diagonal

    __shared__ float As[BK][LDS];
    __shared__ float Bs[BK][LDS];

    const T* A = reinterpret_cast<const T*>(p.A) + (int64_t)b * p.a_batch;
    const T* Bm = reinterpret_cast<const T*>(p.Bm) + (int64_t)b * p.b_batch;
    const int tid = threadIdx.x;
    const int lr = tid >> 2;          // tile row loaded by this thread (0..63)
    const int lk = (tid & 3) * 4;     // first of its 4 k values
    const int ty = tid >> 4, tx = tid & 15;

    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    const bool a_ok = row0 + lr < m, b_ok = col0 + lr < n;
    const T* a_ptr = A + (int64_t)(row0 + lr) * p.lda + lk;
    const T* b_ptr = Bm + (int64_t)(col0 + lr) * p.ldb + lk;

    // software pipeline: the global loads of K block i+1 are in flight while block i is
    // multiplied out of shared memory
    float av[4] = {0.f, 0.f, 0.f, 0.f}, bv[4] = {0.f, 0.f, 0.f, 0.f};
    if (lk < p.d) {                   // d is a multiple of 4: a group of 4 is all in or all out
        if (a_ok) load4<T>(a_ptr, av);
        if (b_ok) load4<T>(b_ptr, bv);
    }
    for (int k0 = 0; k0 < p.d; k0 += BK) {
        __syncthreads();              // the previous block has been consumed
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            As[lk + i][lr] = av[i];
            Bs[lk + i][lr] = bv[i];
        }
        __syncthreads();
        const int kn = k0 + BK + lk;
#pragma unroll
        for (int i = 0; i < 4; ++i) av[i] = bv[i] = 0.f;
        if (kn < p.d) {
            if (a_ok) load4<T>(a_ptr + k0 + BK, av);
            if (b_ok) load4<T>(b_ptr + k0 + BK, bv);
        }
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            const float4 a4 = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            const float4 b4 = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
            const float a[4] = {a4.x, a4.y, a4.z, a4.w};
            const float bb[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], bb[j], acc[i][j]);
        }
    }

    // ---- epilogue: scale, |.|, mask, row maximum --------------------------------
    const int64_t o = (int64_t)b * p.cap;
    float cs[4];
    bool cok[4];
    int ctok[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int c = col0 + tx * 4 + j;
        cok[j] = c < n;
        cs[j] = 0.f;
        ctok[j] = c;
        if (cok[j]) {
            cs[j] = p.inv_b[o + c];
            if (!p.tri) {
                cok[j] = p.col_gate[o + c] < (p.thr_seq != nullptr ? p.thr_seq[b] : p.thr_bits);   // valid representative (line 5)
                if (p.causal) ctok[j] = p.col_token[o + c];
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = row0 + ty * 4 + i;
        float mx = 0.f;
        if (r < m) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const bool adm = cok[j] && ((p.tri || p.causal) ? ctok[j] < r : true);
                const float v = fabsf(acc[i][j]) * cs[j];
                if (adm) mx = fmaxf(mx, v);
            }
        }
        // the 16 threads sharing this row are 16 consecutive lanes
#pragma unroll
        for (int s = 8; s > 0; s >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, s));
        if (tx == 0 && r < m) {
            const bool skip = !p.tri && p.row_role[o + r] != 0;   // inherited reps are not candidates
            if (!skip) {
                mx *= p.inv_a[o + r];
                if (mx > 0.f) atomicMax(p.out + o + r, __float_as_uint(mx));
            }
        }
    }
}

}  // namespace

cudaError_t launch_gram_ffma(ada_ctx* ctx, const GramProblem& p, ada_dtype dt, cudaStream_t s) {
    const int n_cap = p.n_dev != nullptr ? p.cap : p.n_host;
    const int m_cap = p.tri ? n_cap : p.rows;
    if (n_cap <= 0 || m_cap <= 0) return cudaSuccess;
    dim3 grid((n_cap + BN - 1) / BN, (m_cap + BM - 1) / BM, p.B);
    prof_begin(ctx, p.tri ? K_GRAM_FFMA_TRI : K_GRAM_FFMA_CROSS, s);
    if (dt == ADA_F32) launch_k(ctx, k_gram_ffma<float>, grid, dim3(256), 0, s, p);
    else launch_k(ctx, k_gram_ffma<__nv_bfloat16>, grid, dim3(256), 0, s, p);
    prof_end(ctx, s);
    return cudaGetLastError();
}

}  // namespace ada
