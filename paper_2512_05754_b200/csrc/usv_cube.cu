// Local 3D cubes (overview figure of the paper, Fig. 2: the tokens are grouped into small 3D
// cubes, and attention inside the own cube runs beside the long-range top-k selection of cubes).
//
//   cube_order_kernel      token order in which the tokens of one cube are consecutive, so that a
//                          64-token block of the attention path is a 4 x 4 x 4 cube: closed-form
//                          position of every raster token, written as the permutation and its
//                          inverse.  The permutation is applied to [B,N,C] tensors with
//                          usv_token_unmerge (a row gather).
//   force_own_block_kernel the local branch as part of the selection: the score of (query block I,
//                          key block I) is raised to +inf, so that the top-k selection that
//                          follows always keeps a query block's own cube (or lowered to -inf, so
//                          that it never does: the long-range branch of the two-branch form).
//   combine_kernel         the two-branch form: local-cube output and long-range output, computed
//                          apart over disjoint key sets, fused with the softmax mass of each branch
//                          (one warp per query row, HBM stream).
#include "usv_common.cuh"

namespace usv {

// Position of raster token n in the cube order.  Cubes in raster order of their cube
// coordinates, tokens of a cube in raster order of their offsets; a cube cut by the edge of
// the grid holds fewer tokens, nothing is padded.  Everything before token (t,y,x):
//   whole slabs of cubes before its slab, whole rows of cubes before its row inside the slab,
//   whole cubes before its cube inside that row, then its rank inside its own (possibly cut) cube.
__global__ void __launch_bounds__(256) cube_order_kernel(int T, int Hh, int W, int ct, int ch, int cw,
                                                         int32_t* __restrict__ perm, int32_t* __restrict__ inv) {
    dep_sync();
    const int n = blockIdx.x * 256 + threadIdx.x;
    if (n >= T * Hh * W) return;
    const int x = n % W, y = (n / W) % Hh, t = n / (W * Hh);
    const int t0 = t / ct * ct, y0 = y / ch * ch, x0 = x / cw * cw;   // origin of the token's cube
    const int et = min(ct, T - t0), eh = min(ch, Hh - y0), ew = min(cw, W - x0);   // its extent
    const int pos = t0 * Hh * W               // slabs before
                    + et * y0 * W             // cube rows before, inside the slab
                    + et * eh * x0            // cubes before, inside the cube row
                    + ((t - t0) * eh + (y - y0)) * ew + (x - x0);
    perm[pos] = n;
    if (inv != nullptr) inv[n] = pos;
}

__global__ void __launch_bounds__(256) force_own_block_kernel(float* __restrict__ scores, int NBq, int NBk,
                                                              int64_t total, uint32_t value_bits) {
    dep_sync();
    const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;   // (b, h, I) flattened
    if (i >= total) return;
    const int I = (int)(i % NBq);
    if (I < NBk) scores[i * NBk + I] = __uint_as_float(value_bits);
}

struct CombineArgs {
    const void *o1, *o2;
    usv_strides s1, s2, so;
    const float *lse1, *lse2;
    __nv_bfloat16* o;
    float* o_f32;      // optional [B,H,N,D]
    float* lse;        // optional [B,H,N]
    int H, N;
    int64_t rows;
};

// o = (e^lse1 o1 + e^lse2 o2) / (e^lse1 + e^lse2), one warp per (b, h, n) row, D / 32 elements per lane.
template <int D, bool F32IN>
__global__ void __launch_bounds__(256) combine_kernel(const CombineArgs a) {
    dep_sync();
    constexpr int EPL = D / 32;   // 4 or 2
    const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (row >= a.rows) return;
    const int lane = threadIdx.x & 31;
    const int n = (int)(row % a.N);
    const int h = (int)((row / a.N) % a.H);
    const int64_t b = row / ((int64_t)a.N * a.H);
    const float l1 = a.lse1[row], l2 = a.lse2[row];
    const float m = fmaxf(l1, l2);
    const float ms = m == -INFINITY ? 0.f : m;
    const float w1 = expf(l1 - ms), w2 = expf(l2 - ms);
    const float tot = w1 + w2;
    const float inv = tot > 0.f ? 1.0f / tot : 0.f;
    float x1[EPL], x2[EPL];
    const int64_t off1 = b * a.s1.sb + h * a.s1.sh + (int64_t)n * a.s1.sn + lane * EPL;
    const int64_t off2 = b * a.s2.sb + h * a.s2.sh + (int64_t)n * a.s2.sn + lane * EPL;
    if (F32IN) {
        const float* p1 = static_cast<const float*>(a.o1) + off1;
        const float* p2 = static_cast<const float*>(a.o2) + off2;
        if (EPL == 4) {
            const float4 v1 = *reinterpret_cast<const float4*>(p1), v2 = *reinterpret_cast<const float4*>(p2);
            x1[0] = v1.x; x1[1] = v1.y; x1[EPL - 2] = v1.z; x1[EPL - 1] = v1.w;
            x2[0] = v2.x; x2[1] = v2.y; x2[EPL - 2] = v2.z; x2[EPL - 1] = v2.w;
        } else {
            const float2 v1 = *reinterpret_cast<const float2*>(p1), v2 = *reinterpret_cast<const float2*>(p2);
            x1[0] = v1.x; x1[1] = v1.y;
            x2[0] = v2.x; x2[1] = v2.y;
        }
    } else {
        const __nv_bfloat16* p1 = static_cast<const __nv_bfloat16*>(a.o1) + off1;
        const __nv_bfloat16* p2 = static_cast<const __nv_bfloat16*>(a.o2) + off2;
#pragma unroll
        for (int e = 0; e < EPL; e += 2) {
            const uint32_t u1 = *reinterpret_cast<const uint32_t*>(p1 + e);
            const uint32_t u2 = *reinterpret_cast<const uint32_t*>(p2 + e);
            x1[e] = __uint_as_float(u1 << 16); x1[e + 1] = __uint_as_float(u1 & 0xffff0000u);
            x2[e] = __uint_as_float(u2 << 16); x2[e + 1] = __uint_as_float(u2 & 0xffff0000u);
        }
    }
    float y[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
        // a branch without keys (weight 0) must not leak a NaN or an infinity of its (undefined) output
        const float t1 = w1 > 0.f ? w1 * x1[e] : 0.f;
        const float t2 = w2 > 0.f ? w2 * x2[e] : 0.f;
        y[e] = (t1 + t2) * inv;
    }
    __nv_bfloat16* po = a.o + b * a.so.sb + h * a.so.sh + (int64_t)n * a.so.sn + lane * EPL;
#pragma unroll
    for (int e = 0; e < EPL; e += 2) *reinterpret_cast<uint32_t*>(po + e) = pack_bf16x2(y[e], y[e + 1]);
    if (a.o_f32 != nullptr) {
        float* pf = a.o_f32 + row * D + lane * EPL;
#pragma unroll
        for (int e = 0; e < EPL; ++e) pf[e] = y[e];
    }
    if (a.lse != nullptr && lane == 0) a.lse[row] = tot > 0.f ? ms + logf(tot) : -INFINITY;
}

}  // namespace usv

using namespace usv;

extern "C" int usv_cube_order(int T, int Hh, int W, int ct, int ch, int cw, int32_t* perm, int32_t* inv,
                              void* stream) {
    if (T <= 0 || Hh <= 0 || W <= 0 || ct <= 0 || ch <= 0 || cw <= 0)
        return fail(USV_ERR_INVALID_ARG, "cube_order: grid %dx%dx%d / cube %dx%dx%d must be positive", T, Hh, W, ct,
                    ch, cw);
    if ((int64_t)T * Hh * W > 2147483647LL) return fail(USV_ERR_UNSUPPORTED, "cube_order: more than 2^31-1 tokens");
    if (perm == nullptr) return fail(USV_ERR_INVALID_ARG, "cube_order: null pointer");
    const int N = T * Hh * W;
    launch_dep(cube_order_kernel, dim3(ceil_div(N, 256)), dim3(256), 0, static_cast<cudaStream_t>(stream), T, Hh, W, ct, ch, cw, perm, inv);
    USV_CHECK_LAUNCH("cube_order_kernel");
    return USV_OK;
}

static int set_own_block(const char* who, int B, int H, int NBq, int NBk, float* scores, uint32_t bits, void* stream) {
    if (B <= 0 || H <= 0 || NBq <= 0 || NBk <= 0)
        return fail(USV_ERR_INVALID_ARG, "%s: need B,H,NBq,NBk > 0", who);
    if (scores == nullptr) return fail(USV_ERR_INVALID_ARG, "%s: null pointer", who);
    const int64_t total = (int64_t)B * H * NBq;
    if ((total + 255) / 256 > 2147483647LL) return fail(USV_ERR_UNSUPPORTED, "%s: too many rows", who);
    launch_dep(force_own_block_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, static_cast<cudaStream_t>(stream), 
        scores, NBq, NBk, total, bits);
    USV_CHECK_LAUNCH("force_own_block_kernel");
    return USV_OK;
}

extern "C" int usv_force_own_block(int B, int H, int NBq, int NBk, float* scores, void* stream) {
    return set_own_block("force_own_block", B, H, NBq, NBk, scores, 0x7f800000u, stream);
}

extern "C" int usv_exclude_own_block(int B, int H, int NBq, int NBk, float* scores, void* stream) {
    return set_own_block("exclude_own_block", B, H, NBq, NBk, scores, 0xff800000u, stream);
}

extern "C" int usv_attn_combine(int B, int H, int N, int d, const void* o1, const usv_strides* s1,
                                const float* lse1, const void* o2, const usv_strides* s2, const float* lse2,
                                int inputs_f32, void* o, const usv_strides* so, float* o_f32, float* lse,
                                void* stream) {
    if (B <= 0 || H <= 0 || N <= 0) return fail(USV_ERR_INVALID_ARG, "attn_combine: B,H,N must be positive");
    if (d != 64 && d != 128) return fail(USV_ERR_UNSUPPORTED, "attn_combine: d=%d (need 64 or 128)", d);
    if (inputs_f32 != 0 && inputs_f32 != 1) return fail(USV_ERR_INVALID_ARG, "attn_combine: inputs_f32 must be 0 or 1");
    int rc;
    if ((rc = check_view("o1", o1, s1, d)) != USV_OK) return rc;
    if ((rc = check_view("o2", o2, s2, d)) != USV_OK) return rc;
    if ((rc = check_view("o", o, so, d)) != USV_OK) return rc;
    if (lse1 == nullptr || lse2 == nullptr) return fail(USV_ERR_INVALID_ARG, "attn_combine: null lse");
    CombineArgs a;
    a.o1 = o1; a.o2 = o2; a.s1 = *s1; a.s2 = *s2; a.so = *so;
    a.lse1 = lse1; a.lse2 = lse2;
    a.o = static_cast<__nv_bfloat16*>(o);
    a.o_f32 = o_f32; a.lse = lse;
    a.H = H; a.N = N;
    a.rows = (int64_t)B * H * N;
    const int64_t blocks = (a.rows + 7) / 8;
    if (blocks > 2147483647LL) return fail(USV_ERR_UNSUPPORTED, "attn_combine: too many rows");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (d == 128) {
        if (inputs_f32) launch_dep((combine_kernel<128, true>), dim3((unsigned)blocks), dim3(256), 0, st, a);
        else launch_dep((combine_kernel<128, false>), dim3((unsigned)blocks), dim3(256), 0, st, a);
    } else {
        if (inputs_f32) launch_dep((combine_kernel<64, true>), dim3((unsigned)blocks), dim3(256), 0, st, a);
        else launch_dep((combine_kernel<64, false>), dim3((unsigned)blocks), dim3(256), 0, st, a);
    }
    USV_CHECK_LAUNCH("combine_kernel");
    return USV_OK;
}
