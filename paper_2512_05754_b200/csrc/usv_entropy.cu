// Entropy-aware scheduler inputs (Sec. 3.4 of the USV paper).
//
//   key_marginal_kernel   Eq. 16: abar[b,j] = 1/(H N) sum_h sum_i A(h,i,j) for the block-masked
//                         attention of Eq. 5, d = 64 (d = 128 runs on the tensor cores,
//                         usv_entropy_tc.cu).  One CTA per (b, h, query block): S = Q K^T per
//                         selected key block on mma.sync, A = exp(S - lse_i) with the
//                         log-sum-exp the attention forward wrote, column sums over the 64
//                         rows, fp32 atomic adds into abar.
//   entropy_kernel        Eq. 17: h[b] = -(1/log N) sum_j abar log abar.
//   usv_allocate_sparsity Eq. 18-19 on the host: w = (1-h)^gamma, rho_l = clip(rho_bar w_l / mean w).
//
// This sits beside the hot path: a per-layer statistic the scheduler reads between steps.
#include <math.h>

#include "usv_entropy.cuh"
#include "usv_mma_sync.cuh"

namespace usv {

template <int D>
__global__ void __launch_bounds__(128) key_marginal_kernel(const MargArgs a) {
    dep_sync();
    constexpr int LD = MmaSmem<D>::LD;
    constexpr int TILE = MmaSmem<D>::TILE;
    constexpr int KT = D / 16;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __nv_bfloat16* Qs = reinterpret_cast<__nv_bfloat16*>(smem_raw);
    __nv_bfloat16* Ks = Qs + TILE;          // two K buffers
    __shared__ float cs[USV_BLOCK];         // column sums of the current tile

    const int I = blockIdx.x % a.NB;
    const int bh = blockIdx.x / a.NB;
    const int b = bh / a.H, h = bh % a.H;
    const int kh = a.k_per_head[h];
    const int N = a.N;
    const int32_t* sel = a.sel + ((int64_t)bh * a.NB + I) * a.kmax;
    const __nv_bfloat16* Q = a.q + b * a.sq.sb + h * a.sq.sh;
    const __nv_bfloat16* K = a.k + b * a.sk.sb + h * a.sk.sh;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tig = lane & 3;

    int t = 0;
    while (t < kh && sel[t] < 0) ++t;
    load_tile<D>(Qs, Q, a.sq.sn, I * USV_BLOCK, N);
    if (t < kh) load_tile<D>(Ks, K, a.sk.sn, sel[t] * USV_BLOCK, N);
    cp_async_commit();
    if (threadIdx.x < USV_BLOCK) cs[threadIdx.x] = 0.f;

    // this thread's two rows (g and g + 8 of its warp's 16) and their base-2 log-sum-exp
    const int row0 = I * USV_BLOCK + warp * 16 + g, row1 = row0 + 8;
    const float LOG2E = 1.4426950408889634f;
    const float l0 = row0 < N ? a.lse[(int64_t)bh * N + row0] * LOG2E : 0.f;
    const float l1 = row1 < N ? a.lse[(int64_t)bh * N + row1] * LOG2E : 0.f;
    const float c = a.scale_log2;

    uint32_t qf[KT][4];
    int buf = 0;
    bool first = true;
    while (t < kh) {
        const int J = sel[t];
        int tn = t + 1;
        while (tn < kh && sel[tn] < 0) ++tn;
        cp_async_wait_all();
        __syncthreads();   // tile t visible; the column sums of the tile before have been flushed
        if (tn < kh) load_tile<D>(Ks + (buf ^ 1) * TILE, K, a.sk.sn, sel[tn] * USV_BLOCK, N);
        cp_async_commit();
        if (first) {
            const __nv_bfloat16* qrow = Qs + (warp * 16 + g) * LD + 2 * tig;
#pragma unroll
            for (int kt = 0; kt < KT; ++kt) {
                qf[kt][0] = *reinterpret_cast<const uint32_t*>(qrow + kt * 16);
                qf[kt][1] = *reinterpret_cast<const uint32_t*>(qrow + 8 * LD + kt * 16);
                qf[kt][2] = *reinterpret_cast<const uint32_t*>(qrow + kt * 16 + 8);
                qf[kt][3] = *reinterpret_cast<const uint32_t*>(qrow + 8 * LD + kt * 16 + 8);
            }
            first = false;
        }
        const __nv_bfloat16* Kt = Ks + buf * TILE;
        const int nvalid = N - J * USV_BLOCK;   // keys of this block with index < N
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            float s[4] = {0.f, 0.f, 0.f, 0.f};
            const __nv_bfloat16* krow = Kt + (nt * 8 + g) * LD + 2 * tig;
#pragma unroll
            for (int kt = 0; kt < KT; ++kt) {
                const uint32_t b0 = *reinterpret_cast<const uint32_t*>(krow + kt * 16);
                const uint32_t b1 = *reinterpret_cast<const uint32_t*>(krow + kt * 16 + 8);
                mma_bf16_16816(s, qf[kt], b0, b1);
            }
            // attention weights of rows g, g+8 at columns col, col+1; rows / keys beyond N count nothing
            const int col = nt * 8 + 2 * tig;
            float c0 = 0.f, c1 = 0.f;
            if (row0 < N) { c0 += exp2f(fmaf(s[0], c, -l0)); c1 += exp2f(fmaf(s[1], c, -l0)); }
            if (row1 < N) { c0 += exp2f(fmaf(s[2], c, -l1)); c1 += exp2f(fmaf(s[3], c, -l1)); }
            if (col >= nvalid) c0 = 0.f;
            if (col + 1 >= nvalid) c1 = 0.f;
            // sum over the 8 row groups of the warp (lanes that share tig)
#pragma unroll
            for (int o = 4; o < 32; o <<= 1) {
                c0 += __shfl_xor_sync(0xffffffffu, c0, o);
                c1 += __shfl_xor_sync(0xffffffffu, c1, o);
            }
            if (g == 0) {
                atomicAdd(&cs[col], c0);
                atomicAdd(&cs[col + 1], c1);
            }
        }
        __syncthreads();
        if (threadIdx.x < USV_BLOCK) {
            const int j = J * USV_BLOCK + threadIdx.x;
            if (j < N) atomicAdd(a.marg + (int64_t)b * N + j, cs[threadIdx.x] * a.inv_hn);
            cs[threadIdx.x] = 0.f;
        }
        buf ^= 1;
        t = tn;
    }
    cp_async_wait_all();
}

// one CTA per batch element
__global__ void __launch_bounds__(1024) entropy_kernel(const float* __restrict__ marg, int N, float* __restrict__ h) {
    dep_sync();
    __shared__ float red[32];
    const float* m = marg + (int64_t)blockIdx.x * N;
    float s = 0.f;
    for (int j = threadIdx.x; j < N; j += 1024) {
        const float v = m[j];
        if (v > 0.f) s -= v * logf(v);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x < 32) {
        s = red[threadIdx.x];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (threadIdx.x == 0) h[blockIdx.x] = N > 1 ? s / logf((float)N) : 0.f;
    }
}

}  // namespace usv

extern "C" int usv_attn_entropy(int B, int H, int N, int d, const void* q, const usv_strides* sq,
                                const void* k, const usv_strides* sk, const int32_t* sel,
                                const int32_t* k_per_head, int kmax, const float* lse, float scale,
                                float* key_marginal, float* entropy, void* ws, void* stream) {
    using namespace usv;
    if (B <= 0 || H <= 0 || N <= 0) return fail(USV_ERR_INVALID_ARG, "attn_entropy: B,H,N must be positive");
    if (d != 64 && d != 128) return fail(USV_ERR_UNSUPPORTED, "attn_entropy: d=%d (need 64 or 128)", d);
    if (H > USV_MAX_HEADS) return fail(USV_ERR_UNSUPPORTED, "attn_entropy: H > %d", USV_MAX_HEADS);
    int rc;
    if ((rc = check_view("q", q, sq, d)) != USV_OK) return rc;
    if ((rc = check_view("k", k, sk, d)) != USV_OK) return rc;
    if (sel == nullptr || k_per_head == nullptr || lse == nullptr || key_marginal == nullptr || entropy == nullptr)
        return fail(USV_ERR_INVALID_ARG, "attn_entropy: null pointer");
    if (!(scale >= 0.f)) return fail(USV_ERR_INVALID_ARG, "attn_entropy: scale must be >= 0");
    const int NB = ceil_div(N, USV_BLOCK);
    MargArgs a;
    int kmx = 0;
    for (int h = 0; h < H; ++h) {
        if (k_per_head[h] < 1 || k_per_head[h] > NB)
            return fail(USV_ERR_INVALID_ARG, "attn_entropy: k_per_head[%d]=%d outside [1,%d]", h, k_per_head[h], NB);
        a.k_per_head[h] = k_per_head[h];
        kmx = k_per_head[h] > kmx ? k_per_head[h] : kmx;
    }
    if (kmax < kmx) return fail(USV_ERR_INVALID_ARG, "attn_entropy: kmax=%d < max k=%d", kmax, kmx);
    const int64_t grid = (int64_t)B * H * NB;
    if (grid > 2147483647LL) return fail(USV_ERR_UNSUPPORTED, "attn_entropy: too many query blocks");
    a.q = static_cast<const __nv_bfloat16*>(q);
    a.k = static_cast<const __nv_bfloat16*>(k);
    a.sq = *sq; a.sk = *sk;
    a.sel = sel; a.lse = lse; a.marg = key_marginal;
    a.status = static_cast<unsigned int*>(ws);
    a.B = B; a.H = H; a.N = N; a.NB = NB; a.kmax = kmax;
    const float sc = scale == 0.f ? 1.0f / sqrtf((float)d) : scale;
    a.scale_log2 = sc * 1.4426950408889634f;
    a.inv_hn = 1.0f / ((float)H * (float)N);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(key_marginal, 0, (size_t)B * N * sizeof(float), st);
    if (e != cudaSuccess) return fail(USV_ERR_CUDA, "attn_entropy: memset: %s", cudaGetErrorString(e));
    if (d == 128) {
        int rc2 = launch_marginal_tc(a, st);
        if (rc2 != USV_OK) return rc2;
    } else {
        const size_t smem = (size_t)3 * MmaSmem<64>::TILE * sizeof(__nv_bfloat16);
        cudaFuncSetAttribute(key_marginal_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        launch_dep(key_marginal_kernel<64>, dim3((unsigned)grid), dim3(128), smem, st, a);
    }
    if (d != 128) USV_CHECK_LAUNCH("key_marginal_kernel");
    launch_dep(entropy_kernel, dim3(B), dim3(1024), 0, st, key_marginal, N, entropy);
    USV_CHECK_LAUNCH("entropy_kernel");
    return USV_OK;
}

extern "C" int usv_allocate_sparsity(int L, const float* entropy, float gamma, float rho_bar, float rho_min,
                                     float rho_max, float* rho) {
    using namespace usv;
    if (L <= 0 || entropy == nullptr || rho == nullptr) return fail(USV_ERR_INVALID_ARG, "allocate_sparsity: bad L or null pointer");
    if (!(gamma >= 1.f)) return fail(USV_ERR_INVALID_ARG, "allocate_sparsity: gamma must be >= 1");
    if (!(rho_min <= rho_max)) return fail(USV_ERR_INVALID_ARG, "allocate_sparsity: rho_min > rho_max");
    double mean = 0.0;
    for (int l = 0; l < L; ++l) {
        if (!(entropy[l] >= 0.f && entropy[l] <= 1.f))
            return fail(USV_ERR_INVALID_ARG, "allocate_sparsity: entropy[%d]=%g outside [0,1]", l, (double)entropy[l]);
        mean += pow(1.0 - (double)entropy[l], (double)gamma);
    }
    mean /= (double)L;
    for (int l = 0; l < L; ++l) {
        // all layers at entropy 1 (mean 0): no layer is favoured, every one keeps the base ratio
        const double w = mean > 0.0 ? pow(1.0 - (double)entropy[l], (double)gamma) / mean : 1.0;
        const double r = (double)rho_bar * w;
        rho[l] = (float)(r < rho_min ? rho_min : (r > rho_max ? rho_max : r));
    }
    return USV_OK;
}
