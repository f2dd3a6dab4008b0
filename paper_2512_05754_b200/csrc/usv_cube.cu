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
//                          follows always keeps a query block's own cube.
#include "usv_common.cuh"

namespace usv {

// Position of raster token n in the cube order.  Cubes in raster order of their cube
// coordinates, tokens of a cube in raster order of their offsets; a cube cut by the edge of
// the grid holds fewer tokens, nothing is padded.  Everything before token (t,y,x):
//   whole slabs of cubes before its slab, whole rows of cubes before its row inside the slab,
//   whole cubes before its cube inside that row, then its rank inside its own (possibly cut) cube.
__global__ void __launch_bounds__(256) cube_order_kernel(int T, int Hh, int W, int ct, int ch, int cw,
                                                         int32_t* __restrict__ perm, int32_t* __restrict__ inv) {
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
                                                              int64_t total) {
    const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;   // (b, h, I) flattened
    if (i >= total) return;
    const int I = (int)(i % NBq);
    if (I < NBk) scores[i * NBk + I] = __int_as_float(0x7f800000);
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
    cube_order_kernel<<<ceil_div(N, 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(T, Hh, W, ct, ch, cw, perm, inv);
    USV_CHECK_LAUNCH("cube_order_kernel");
    return USV_OK;
}

extern "C" int usv_force_own_block(int B, int H, int NBq, int NBk, float* scores, void* stream) {
    if (B <= 0 || H <= 0 || NBq <= 0 || NBk <= 0)
        return fail(USV_ERR_INVALID_ARG, "force_own_block: need B,H,NBq,NBk > 0");
    if (scores == nullptr) return fail(USV_ERR_INVALID_ARG, "force_own_block: null pointer");
    const int64_t total = (int64_t)B * H * NBq;
    if ((total + 255) / 256 > 2147483647LL) return fail(USV_ERR_UNSUPPORTED, "force_own_block: too many rows");
    force_own_block_kernel<<<(unsigned)((total + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        scores, NBq, NBk, total);
    USV_CHECK_LAUNCH("force_own_block_kernel");
    return USV_OK;
}
