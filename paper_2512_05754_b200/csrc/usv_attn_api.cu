// Entry point of the block-sparse attention forward: validation, head ordering, dispatch.
#include <algorithm>

#include "usv_attn.cuh"

extern "C" size_t usv_sparse_attn_workspace(int B, int H, int N, int d, int kmax) {
    (void)d;
    if (B <= 0 || H <= 0 || N <= 0) return 0;
    // header (status word, fallback counter), the fallback work list, the pairing plan
    const int NB = usv::ceil_div(N, USV_BLOCK);
    // sized for the worst case of every head keeping kmax blocks
    if (H > USV_MAX_HEADS) return 0;
    int32_t kk[USV_MAX_HEADS];
    for (int h = 0; h < H; ++h) kk[h] = kmax < 1 ? 1 : (kmax > NB ? NB : kmax);
    return usv::WS_HEADER + usv::align_up((size_t)B * H * NB * sizeof(int), 256) + usv::pair_plan_bytes(B, H, NB, kk);
}

static int sparse_attn_impl(int B, int H, int N, int d, const void* q, const usv_strides* sq,
                            const void* k, const usv_strides* sk, const void* v,
                            const usv_strides* sv, const int32_t* sel,
                            const int32_t* k_per_head, int kmax, void* o,
                            const usv_strides* so, float* o_f32, float* lse, float scale,
                            int impl, void* ws, size_t ws_bytes, void* stream, int N_full,
                            const int32_t* unmerge_off, const int32_t* unmerge_idx, void* y) {
    using namespace usv;
    if (y != nullptr) {
        if (unmerge_off == nullptr || unmerge_idx == nullptr)
            return fail(USV_ERR_INVALID_ARG, "sparse_attn_unmerge: null unmerge map");
        if (N_full < N) return fail(USV_ERR_INVALID_ARG, "sparse_attn_unmerge: N_full=%d < N=%d", N_full, N);
        if (d != 128 || impl != 0)
            return fail(USV_ERR_UNSUPPORTED, "sparse_attn_unmerge: the fused unmerge needs d = 128 and impl 0");
        if (!aligned16(y)) return fail(USV_ERR_UNSUPPORTED, "sparse_attn_unmerge: y not 16-byte aligned");
    }
    if (B <= 0 || H <= 0 || N <= 0) return fail(USV_ERR_INVALID_ARG, "sparse_attn: B,H,N must be positive");
    if (d != 64 && d != 128) return fail(USV_ERR_UNSUPPORTED, "sparse_attn: d=%d (need 64 or 128)", d);
    if (H > USV_MAX_HEADS) return fail(USV_ERR_UNSUPPORTED, "sparse_attn: H > %d", USV_MAX_HEADS);
    int rc;
    if ((rc = check_view("q", q, sq, d)) != USV_OK) return rc;
    if ((rc = check_view("k", k, sk, d)) != USV_OK) return rc;
    if ((rc = check_view("v", v, sv, d)) != USV_OK) return rc;
    if ((rc = check_view("o", o, so, d)) != USV_OK) return rc;
    if (sel == nullptr || k_per_head == nullptr) return fail(USV_ERR_INVALID_ARG, "sparse_attn: null sel/k_per_head");
    if (o_f32 != nullptr && !aligned16(o_f32)) return fail(USV_ERR_UNSUPPORTED, "sparse_attn: o_f32 misaligned");
    if (!(scale >= 0.f)) return fail(USV_ERR_INVALID_ARG, "sparse_attn: scale must be >= 0");
    if (impl != 0 && impl != 1) return fail(USV_ERR_INVALID_ARG, "sparse_attn: impl must be 0 or 1");
    if (ws == nullptr) return fail(USV_ERR_INVALID_ARG, "sparse_attn: null workspace");
    if (ws_bytes < usv_sparse_attn_workspace(B, H, N, d, kmax))
        return fail(USV_ERR_WORKSPACE, "sparse_attn: workspace %zu < %zu", ws_bytes,
                    usv_sparse_attn_workspace(B, H, N, d, kmax));
    const int NB = ceil_div(N, USV_BLOCK);
    AttnArgs a;
    int kmx = 0;
    for (int h = 0; h < H; ++h) {
        if (k_per_head[h] < 1 || k_per_head[h] > NB)
            return fail(USV_ERR_INVALID_ARG, "sparse_attn: k_per_head[%d]=%d outside [1,%d]", h,
                        k_per_head[h], NB);
        a.k_per_head[h] = k_per_head[h];
        a.head_order[h] = h;
        kmx = std::max(kmx, k_per_head[h]);
    }
    if (kmax < kmx) return fail(USV_ERR_INVALID_ARG, "sparse_attn: kmax=%d < max k=%d", kmax, kmx);
    std::stable_sort(a.head_order, a.head_order + H,
                     [&](int x, int y) { return k_per_head[x] > k_per_head[y]; });
    a.q = static_cast<const __nv_bfloat16*>(q);
    a.k = static_cast<const __nv_bfloat16*>(k);
    a.v = static_cast<const __nv_bfloat16*>(v);
    a.o = static_cast<__nv_bfloat16*>(o);
    a.sq = *sq; a.sk = *sk; a.sv = *sv; a.so = *so;
    a.sel = sel;
    a.o_f32 = o_f32;
    a.lse = lse;
    a.status = static_cast<unsigned int*>(ws);
    a.fallback_count = reinterpret_cast<int*>(static_cast<char*>(ws) + 4);
    a.work_counter = reinterpret_cast<int*>(static_cast<char*>(ws) + 8);
    a.fallback_list = reinterpret_cast<int*>(static_cast<char*>(ws) + WS_HEADER);
    void* plan_mem = static_cast<char*>(ws) + WS_HEADER + align_up((size_t)B * H * NB * sizeof(int), 256);
    a.pairs = nullptr;
    a.lists = nullptr;
    a.list_batch = 0;
    a.work_list = nullptr;
    a.work_count = nullptr;
    a.unmerge_off = unmerge_off;
    a.unmerge_idx = unmerge_idx;
    a.y = static_cast<__nv_bfloat16*>(y);
    a.N_full = N_full;
    a.B = B; a.H = H; a.N = N; a.NB = NB; a.kmax = kmax;
    const float sc = scale == 0.f ? 1.0f / sqrtf((float)d) : scale;
    a.scale_log2 = sc * 1.4426950408889634f;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the status word (word 0) is sticky; everything behind it starts at zero (the pairing-plan
    // kernel does that itself: a memset between two kernels costs them their overlapped launch)
    if (impl == 0 && attn_pair_supported(a, d)) {
        int rc2 = launch_pair_plan(a, plan_mem, st);
        if (rc2 != USV_OK) return rc2;
        rc2 = launch_attn_pair(a, d, st);
        if (rc2 != USV_OK) return rc2;
        // exact recomputation of the (normally zero) query blocks the fast kernel reported
        a.work_list = a.fallback_list;
        a.work_count = a.fallback_count;
        rc2 = launch_attn_mma(a, d, st);
        if (rc2 != USV_OK || y == nullptr) return rc2;
        return launch_scatter_fallbacks(a, d, st);
    }
    if (y != nullptr) return fail(USV_ERR_UNSUPPORTED, "sparse_attn_unmerge: sequence too long for the tcgen05 kernel");
    cudaError_t e = cudaMemsetAsync(static_cast<char*>(ws) + 4, 0, WS_HEADER - 4, st);
    if (e != cudaSuccess) return fail(USV_ERR_CUDA, "sparse_attn: memset: %s", cudaGetErrorString(e));
    return launch_attn_mma(a, d, st);
}

extern "C" int usv_sparse_attn_fwd(int B, int H, int N, int d, const void* q, const usv_strides* sq,
                                   const void* k, const usv_strides* sk, const void* v,
                                   const usv_strides* sv, const int32_t* sel,
                                   const int32_t* k_per_head, int kmax, void* o,
                                   const usv_strides* so, float* o_f32, float* lse, float scale,
                                   int impl, void* ws, size_t ws_bytes, void* stream) {
    return sparse_attn_impl(B, H, N, d, q, sq, k, sk, v, sv, sel, k_per_head, kmax, o, so, o_f32, lse, scale, impl, ws,
                            ws_bytes, stream, 0, nullptr, nullptr, nullptr);
}

extern "C" int usv_sparse_attn_fwd_unmerge(int B, int H, int N, int d, const void* q, const usv_strides* sq,
                                           const void* k, const usv_strides* sk, const void* v,
                                           const usv_strides* sv, const int32_t* sel,
                                           const int32_t* k_per_head, int kmax, void* o,
                                           const usv_strides* so, float* o_f32, float* lse, float scale,
                                           void* ws, size_t ws_bytes, int N_full, const int32_t* unmerge_off,
                                           const int32_t* unmerge_idx, void* y, void* stream) {
    if (y == nullptr) return usv::fail(USV_ERR_INVALID_ARG, "sparse_attn_unmerge: null y");
    return sparse_attn_impl(B, H, N, d, q, sq, k, sk, v, sv, sel, k_per_head, kmax, o, so, o_f32, lse, scale, 0, ws,
                            ws_bytes, stream, N_full, unmerge_off, unmerge_idx, y);
}
