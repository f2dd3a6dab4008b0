// Coarse stage of the key-block selection: block pooling (HBM stream) and block scores.
//
//   pool_kernel   : one CTA per (tensor, b, h, four blocks); 16-byte loads, the next block in
//                   flight while the current one is reduced (fp32 tree), mean over the VALID
//                   rows of a block.  At d = 128 it also writes the three bf16 planes
//                   (mean = hi + mid + lo) that the tensor-core score kernel multiplies, so the
//                   fp32 means are not read back for a separate split pass.
//   scores_kernel : fp32 CUDA-core NT GEMM per (b,h), 64x64 output tile, 4x4 per thread.
//                   Kept in fp32 (not bf16 tensor cores) because the result decides an integer
//                   (the top-k set) that is compared with an fp64 evaluation.
#include "usv_scores.cuh"

namespace usv {

struct PoolArgs {
    const __nv_bfloat16* x[2];
    int64_t sb[2], sh[2], sn[2];
    int N[2], NB[2];
    float* out[2];  // [B,H,NB,d]
    int H;
    // d = 128 with the tensor-core score kernel: bf16 planes [3][B*H][NB_pad][128] per tensor
    // (NULL: not wanted); rows NB .. NB_pad - 1 are written as zero
    __nv_bfloat16* planes[2];
    int NB_pad[2];
};

// D = head dim (64 or 128).  Threads: 128.  A row of D bf16 is D/8 uint4; TPR threads per row.
// A CTA pools POOL_SPAN consecutive blocks of one (tensor, b, h); the loads of the next block are
// issued before the current one is reduced, so that the CTA always has a block in flight.
constexpr int POOL_SPAN = 4;

template <int D>
__global__ void __launch_bounds__(128) pool_kernel(const PoolArgs a) {
    dep_sync();
    constexpr int TPR = D / 8;          // 16 (d=128) or 8 (d=64)
    constexpr int RPI = 128 / TPR;      // rows per iteration: 8 or 16
    constexpr int ITERS = USV_BLOCK / RPI;
    const int which = blockIdx.z;
    const int NB = a.NB[which];
    const int I0 = blockIdx.x * POOL_SPAN;
    if (I0 >= NB) return;
    const int I1 = min(I0 + POOL_SPAN, NB);
    const int bh = blockIdx.y;
    const int b = bh / a.H, h = bh % a.H;
    const int N = a.N[which];
    const int col = threadIdx.x % TPR, rg = threadIdx.x / TPR;
    const __nv_bfloat16* base =
        a.x[which] + b * a.sb[which] + h * a.sh[which] + (int64_t)col * 8;
    const int64_t sn = a.sn[which];
    __shared__ float red[2][RPI][D + 4];

    auto load_block = [&](int I, uint4* v) {
        const int row0 = I * USV_BLOCK;
        const int nvalid = min(USV_BLOCK, N - row0);
#pragma unroll
        for (int it = 0; it < ITERS; ++it) {
            const int r = it * RPI + rg;
            v[it] = make_uint4(0, 0, 0, 0);
            if (r < nvalid) v[it] = __ldg(reinterpret_cast<const uint4*>(base + (row0 + r) * sn));
        }
    };
    uint4 v[ITERS], vn[ITERS];
    load_block(I0, v);
    for (int I = I0; I < I1; ++I) {
        if (I + 1 < I1) load_block(I + 1, vn);
        float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
        for (int it = 0; it < ITERS; ++it) {
            float f[8];
            bf16x8_to_float(v[it], f);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] += f[e];
        }
        float (*rd)[D + 4] = red[(I - I0) & 1];   // two buffers: one barrier per block is enough
#pragma unroll
        for (int e = 0; e < 8; ++e) rd[rg][col * 8 + e] = acc[e];
        __syncthreads();
        if (threadIdx.x < D) {
            const int nvalid = min(USV_BLOCK, N - I * USV_BLOCK);
            float s = 0.f;
#pragma unroll
            for (int g = 0; g < RPI; ++g) s += rd[g][threadIdx.x];
            const float mean = s / (float)nvalid;
            a.out[which][((int64_t)bh * NB + I) * D + threadIdx.x] = mean;
            if (a.planes[which] != nullptr) {
                const int64_t plane = (int64_t)gridDim.y * a.NB_pad[which] * D;
                __nv_bfloat16* dst = a.planes[which] + ((int64_t)bh * a.NB_pad[which] + I) * D + threadIdx.x;
                float rem = mean;
#pragma unroll
                for (int p = 0; p < 3; ++p) {
                    const __nv_bfloat16 hp = __float2bfloat16_rn(rem);
                    dst[p * plane] = hp;
                    rem -= __bfloat162float(hp);
                }
            }
        }
#pragma unroll
        for (int it = 0; it < ITERS; ++it) v[it] = vn[it];
    }
    // the CTA that pooled the last block also clears the padding rows of the planes
    if (I1 == NB && a.planes[which] != nullptr && threadIdx.x < D) {
        const int64_t plane = (int64_t)gridDim.y * a.NB_pad[which] * D;
        for (int I = NB; I < a.NB_pad[which]; ++I) {
            __nv_bfloat16* dst = a.planes[which] + ((int64_t)bh * a.NB_pad[which] + I) * D + threadIdx.x;
#pragma unroll
            for (int p = 0; p < 3; ++p) dst[p * plane] = __float2bfloat16_rn(0.f);
        }
    }
}

// scores[bh, I, J] = scale * sum_e qbar[bh,I,e] * kbar[bh,J,e]
// CTA: 256 threads, 64x64 tile; smem tiles stored e-major so that the inner product reads
// float4 along the tile row/column.
__global__ void __launch_bounds__(256) scores_kernel(const float* __restrict__ qbar,
                                                     const float* __restrict__ kbar,
                                                     float* __restrict__ scores, int NBq, int NBk,
                                                     int d, float scale) {
    dep_sync();
    constexpr int TM = 64, TN = 64, TK = 32;
    __shared__ __align__(16) float As[TK][TM + 4];
    __shared__ __align__(16) float Bs[TK][TN + 4];
    const int bh = blockIdx.z;
    const int i0 = blockIdx.y * TM, j0 = blockIdx.x * TN;
    const float* A = qbar + (int64_t)bh * NBq * d;
    const float* Bm = kbar + (int64_t)bh * NBk * d;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < d; k0 += TK) {
        // 64 rows x 32 floats = 512 float4; 256 threads -> 2 each
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            const int idx = threadIdx.x + t * 256;
            const int r = idx / 8, c4 = idx % 8;
            float4 va = make_float4(0, 0, 0, 0), vb = va;
            if (i0 + r < NBq)
                va = *reinterpret_cast<const float4*>(A + (int64_t)(i0 + r) * d + k0 + c4 * 4);
            if (j0 + r < NBk)
                vb = *reinterpret_cast<const float4*>(Bm + (int64_t)(j0 + r) * d + k0 + c4 * 4);
            As[c4 * 4 + 0][r] = va.x; As[c4 * 4 + 1][r] = va.y;
            As[c4 * 4 + 2][r] = va.z; As[c4 * 4 + 3][r] = va.w;
            Bs[c4 * 4 + 0][r] = vb.x; Bs[c4 * 4 + 1][r] = vb.y;
            Bs[c4 * 4 + 2][r] = vb.z; Bs[c4 * 4 + 3][r] = vb.w;
        }
        __syncthreads();
#pragma unroll
        for (int e = 0; e < TK; ++e) {
            const float4 av = *reinterpret_cast<const float4*>(&As[e][ty * 4]);
            const float4 bv = *reinterpret_cast<const float4*>(&Bs[e][tx * 4]);
            const float ar[4] = {av.x, av.y, av.z, av.w};
            const float br[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(ar[i], br[j], acc[i][j]);
        }
        __syncthreads();
    }
    float* out = scores + (int64_t)bh * NBq * NBk;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int I = i0 + ty * 4 + i;
        if (I >= NBq) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int J = j0 + tx * 4 + j;
            if (J < NBk) out[(int64_t)I * NBk + J] = acc[i][j] * scale;
        }
    }
}

}  // namespace usv

extern "C" size_t usv_block_scores_workspace(int B, int H, int Nq, int Nk, int d) {
    if (B <= 0 || H <= 0 || Nq <= 0 || Nk <= 0 || d <= 0) return 0;
    const size_t nbq = usv::ceil_div(Nq, USV_BLOCK), nbk = usv::ceil_div(Nk, USV_BLOCK);
    // header, pooled means of q and k; at d = 128 also the bf16 planes of the tensor-core scores kernel
    return usv::WS_HEADER + usv::align_up((size_t)B * H * nbq * d * sizeof(float), 256) +
           usv::align_up((size_t)B * H * nbk * d * sizeof(float), 256) +
           (d == 128 ? usv::scores_tc_bytes(B * H, (int)nbq, (int)nbk) : 0);
}

extern "C" int usv_block_scores(int B, int H, int Nq, int Nk, int d, const void* q,
                                const usv_strides* sq, const void* k, const usv_strides* sk,
                                float* scores, void* ws, size_t ws_bytes, void* stream) {
    using namespace usv;
    if (B <= 0 || H <= 0 || Nq <= 0 || Nk <= 0)
        return fail(USV_ERR_INVALID_ARG, "block_scores: B,H,Nq,Nk must be positive");
    if (d != 64 && d != 128) return fail(USV_ERR_UNSUPPORTED, "block_scores: d=%d (need 64 or 128)", d);
    if ((int64_t)B * H > 65535) return fail(USV_ERR_UNSUPPORTED, "block_scores: B*H > 65535");
    int rc;
    if ((rc = check_view("q", q, sq, d)) != USV_OK) return rc;
    if ((rc = check_view("k", k, sk, d)) != USV_OK) return rc;
    if (scores == nullptr || ws == nullptr) return fail(USV_ERR_INVALID_ARG, "block_scores: null scores/ws");
    if (!aligned16(scores) || !aligned16(ws))
        return fail(USV_ERR_UNSUPPORTED, "block_scores: scores/ws not 16-byte aligned");
    if (ws_bytes < usv_block_scores_workspace(B, H, Nq, Nk, d))
        return fail(USV_ERR_WORKSPACE, "block_scores: workspace %zu < %zu", ws_bytes,
                    usv_block_scores_workspace(B, H, Nq, Nk, d));
    const int NBq = ceil_div(Nq, USV_BLOCK), NBk = ceil_div(Nk, USV_BLOCK);
    float* qbar = reinterpret_cast<float*>(static_cast<char*>(ws) + WS_HEADER);
    float* kbar = reinterpret_cast<float*>(static_cast<char*>(ws) + WS_HEADER +
                                           align_up((size_t)B * H * NBq * d * sizeof(float), 256));
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    PoolArgs a;
    a.x[0] = static_cast<const __nv_bfloat16*>(q);
    a.x[1] = static_cast<const __nv_bfloat16*>(k);
    a.sb[0] = sq->sb; a.sh[0] = sq->sh; a.sn[0] = sq->sn;
    a.sb[1] = sk->sb; a.sh[1] = sk->sh; a.sn[1] = sk->sn;
    a.N[0] = Nq; a.N[1] = Nk; a.NB[0] = NBq; a.NB[1] = NBk;
    a.out[0] = qbar; a.out[1] = kbar;
    a.H = H;
    a.planes[0] = a.planes[1] = nullptr;
    a.NB_pad[0] = a.NB_pad[1] = 0;
    void* tc_mem = reinterpret_cast<char*>(kbar) + align_up((size_t)B * H * NBk * d * sizeof(float), 256);
    if (d == 128) scores_tc_planes(tc_mem, B * H, NBq, NBk, &a.planes[0], &a.planes[1], &a.NB_pad[0], &a.NB_pad[1]);
    dim3 pg(ceil_div(NBq > NBk ? NBq : NBk, POOL_SPAN), B * H, 2);
    if (d == 128) launch_dep(pool_kernel<128>, dim3(pg), dim3(128), 0, st, a);
    else launch_dep(pool_kernel<64>, dim3(pg), dim3(128), 0, st, a);
    USV_CHECK_LAUNCH("pool_kernel");

    if (d == 128)
        return launch_scores_tc(scores, B * H, NBq, NBk, 1.0f / sqrtf((float)d), tc_mem,
                                static_cast<unsigned int*>(ws), st);
    dim3 sg(ceil_div(NBk, 64), ceil_div(NBq, 64), B * H);
    launch_dep(scores_kernel, dim3(sg), dim3(256), 0, st, qbar, kbar, scores, NBq, NBk, d, 1.0f / sqrtf((float)d));
    USV_CHECK_LAUNCH("scores_kernel");
    return USV_OK;
}

// ------------------------------------------------------------------------------------------
// Variant without caller scratch: the pooled means go to a fixed array inside the library image.
// For callers that may neither allocate device memory nor lend a buffer (allocator-frozen
// sections of a host framework, plugins that only receive tensors, fixed-budget loops).

namespace usv {

static __device__ __align__(256) unsigned char g_noalloc_scratch[USV_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
static void* g_noalloc_ptr[kMaxDevices] = {};  // device address of the array, per device

// In host code `g_noalloc_scratch` is only a handle for the runtime, not an address a kernel
// can use; the real per-device address has to be asked for once, with that device current.
static int noalloc_scratch(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(USV_ERR_CUDA, "block_scores_noalloc: cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices) return fail(USV_ERR_UNSUPPORTED, "block_scores_noalloc: device %d out of range", dev);
    void* p = __atomic_load_n(&g_noalloc_ptr[dev], __ATOMIC_ACQUIRE);
    if (p == nullptr) {
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess || p == nullptr)
            return fail(USV_ERR_CUDA, "block_scores_noalloc: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        __atomic_store_n(&g_noalloc_ptr[dev], p, __ATOMIC_RELEASE);  // same value from any thread
    }
    *out = p;
    return USV_OK;
}

}  // namespace usv

extern "C" int usv_block_scores_noalloc(int B, int H, int Nq, int Nk, int d, const void* q,
                                        const usv_strides* sq, const void* k,
                                        const usv_strides* sk, float* scores, void* stream) {
    using namespace usv;
    if (B <= 0 || H <= 0 || Nq <= 0 || Nk <= 0)
        return fail(USV_ERR_INVALID_ARG, "block_scores_noalloc: B,H,Nq,Nk must be positive");
    if (d != 64 && d != 128) return fail(USV_ERR_UNSUPPORTED, "block_scores_noalloc: d=%d (need 64 or 128)", d);
    if ((int64_t)B * H > 65535) return fail(USV_ERR_UNSUPPORTED, "block_scores_noalloc: B*H > 65535");
    int rc;
    if ((rc = check_view("q", q, sq, d)) != USV_OK) return rc;
    if ((rc = check_view("k", k, sk, d)) != USV_OK) return rc;
    if (scores == nullptr) return fail(USV_ERR_INVALID_ARG, "block_scores_noalloc: null scores");
    if (!aligned16(scores)) return fail(USV_ERR_UNSUPPORTED, "block_scores_noalloc: scores not 16-byte aligned");
    const size_t need = align_up((size_t)B * H * ceil_div(Nq, USV_BLOCK) * d * sizeof(float), 256) +
                        align_up((size_t)B * H * ceil_div(Nk, USV_BLOCK) * d * sizeof(float), 256);
    if (need > (size_t)USV_NOALLOC_SCRATCH_BYTES)
        return fail(USV_ERR_WORKSPACE,
                    "block_scores_noalloc: needs %zu bytes of scratch, the built-in array holds %u; "
                    "use usv_block_scores with a caller workspace for this size",
                    need, (unsigned)USV_NOALLOC_SCRATCH_BYTES);
    void* scratch = nullptr;
    if ((rc = noalloc_scratch(&scratch)) != USV_OK) return rc;

    const int NBq = ceil_div(Nq, USV_BLOCK), NBk = ceil_div(Nk, USV_BLOCK);
    float* qbar = static_cast<float*>(scratch);
    float* kbar = reinterpret_cast<float*>(static_cast<char*>(scratch) +
                                           align_up((size_t)B * H * NBq * d * sizeof(float), 256));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    PoolArgs a;
    a.x[0] = static_cast<const __nv_bfloat16*>(q);
    a.x[1] = static_cast<const __nv_bfloat16*>(k);
    a.sb[0] = sq->sb; a.sh[0] = sq->sh; a.sn[0] = sq->sn;
    a.sb[1] = sk->sb; a.sh[1] = sk->sh; a.sn[1] = sk->sn;
    a.N[0] = Nq; a.N[1] = Nk; a.NB[0] = NBq; a.NB[1] = NBk;
    a.out[0] = qbar; a.out[1] = kbar;
    a.H = H;
    a.planes[0] = a.planes[1] = nullptr;
    a.NB_pad[0] = a.NB_pad[1] = 0;
    dim3 pg(ceil_div(NBq > NBk ? NBq : NBk, POOL_SPAN), B * H, 2);
    if (d == 128) pool_kernel<128><<<pg, 128, 0, st>>>(a);
    else pool_kernel<64><<<pg, 128, 0, st>>>(a);
    USV_CHECK_LAUNCH("pool_kernel (noalloc)");
    dim3 sg(ceil_div(NBk, 64), ceil_div(NBq, 64), B * H);
    scores_kernel<<<sg, 256, 0, st>>>(qbar, kbar, scores, NBq, NBk, d, 1.0f / sqrtf((float)d));
    USV_CHECK_LAUNCH("scores_kernel (noalloc)");
    return USV_OK;
}
