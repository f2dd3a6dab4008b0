// Block-sparse attention forward, legacy tensor-core path (mma.sync m16n8k16, bf16).
//
// Kept as an on-device cross-check of the tcgen05 kernel and as the fallback for shapes the
// tcgen05 kernel does not cover.  One CTA (4 warps) per (b, h, query block); each warp owns 16
// query rows.  Selected K/V blocks stream through a double-buffered cp.async pipeline; S = QK^T
// and O += PV run on mma.sync with the softmax kept in registers (fp32, base-2 exponentials).
#include "usv_mma_sync.cuh"

namespace usv {

template <int D>
__device__ __forceinline__ void attn_mma_block(const AttnArgs& a, const int work, unsigned char* smem_raw) {
    constexpr int LD = MmaSmem<D>::LD;
    constexpr int TILE = MmaSmem<D>::TILE;
    constexpr int KT = D / 16;  // k-steps of QK^T
    constexpr int NT = D / 8;   // n-tiles of the output
    __nv_bfloat16* Qs = reinterpret_cast<__nv_bfloat16*>(smem_raw);
    __nv_bfloat16* Ks = Qs + TILE;
    __nv_bfloat16* Vs = Ks + 2 * TILE;

    const int I = work % a.NB;
    const int bh_ord = work / a.NB;
    const int b = bh_ord / a.H;
    const int h = a.head_order[bh_ord % a.H];
    const int kh = a.k_per_head[h];
    const int N = a.N;
    const int32_t* sel = a.sel + (((int64_t)b * a.H + h) * a.NB + I) * a.kmax;

    const __nv_bfloat16* Q = a.q + b * a.sq.sb + h * a.sq.sh;
    const __nv_bfloat16* K = a.k + b * a.sk.sb + h * a.sk.sh;
    const __nv_bfloat16* V = a.v + b * a.sv.sb + h * a.sv.sh;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tig = lane & 3;

    // first valid entry of the selection
    int t = 0;
    while (t < kh && sel[t] < 0) ++t;

    load_tile<D>(Qs, Q, a.sq.sn, I * USV_BLOCK, N);
    if (t < kh) {
        load_tile<D>(Ks, K, a.sk.sn, sel[t] * USV_BLOCK, N);
        load_tile<D>(Vs, V, a.sv.sn, sel[t] * USV_BLOCK, N);
    }
    cp_async_commit();

    uint32_t qf[KT][4];
    float o[NT][4];
#pragma unroll
    for (int n = 0; n < NT; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
    float m[2] = {-INFINITY, -INFINITY};  // running max of the scaled (base-2) logits, rows g, g+8
    float l[2] = {0.f, 0.f};              // this thread's share of the running denominators
    // The same sums taken over the bf16-rounded weights that feed the P.V product: normalising
    // by them makes the applied weights sum to one exactly, so the rounding of a dominant
    // weight cancels instead of scaling the whole row.
    float lr[2] = {0.f, 0.f};
    const float c = a.scale_log2;

    int buf = 0;
    bool first = true;
    while (t < kh) {
        const int J = sel[t];
        int tn = t + 1;
        while (tn < kh && sel[tn] < 0) ++tn;

        cp_async_wait_all();
        __syncthreads();  // tile t is visible; every warp has left the tile of the step before
        if (tn < kh) {
            load_tile<D>(Ks + (buf ^ 1) * TILE, K, a.sk.sn, sel[tn] * USV_BLOCK, N);
            load_tile<D>(Vs + (buf ^ 1) * TILE, V, a.sv.sn, sel[tn] * USV_BLOCK, N);
        }
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
        const __nv_bfloat16* Vt = Vs + buf * TILE;

        float s[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
            const __nv_bfloat16* krow = Kt + (nt * 8 + g) * LD + 2 * tig;
#pragma unroll
            for (int kt = 0; kt < KT; ++kt) {
                const uint32_t b0 = *reinterpret_cast<const uint32_t*>(krow + kt * 16);
                const uint32_t b1 = *reinterpret_cast<const uint32_t*>(krow + kt * 16 + 8);
                mma_bf16_16816(s[nt], qf[kt], b0, b1);
            }
        }
        const int nvalid = N - J * USV_BLOCK;  // keys of this block with index < N
        if (nvalid < USV_BLOCK) {
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                const int col = nt * 8 + 2 * tig;
                if (col >= nvalid) s[nt][0] = s[nt][2] = -INFINITY;
                if (col + 1 >= nvalid) s[nt][1] = s[nt][3] = -INFINITY;
            }
        }
        // online softmax (rows g -> elements 0,1; row g+8 -> elements 2,3)
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            mx[0] = fmaxf(mx[0], fmaxf(s[nt][0], s[nt][1]));
            mx[1] = fmaxf(mx[1], fmaxf(s[nt][2], s[nt][3]));
        }
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
        }
        float alpha[2], mnew[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            mnew[r] = fmaxf(m[r], mx[r] * c);
            const float ms = mnew[r] == -INFINITY ? 0.f : mnew[r];
            alpha[r] = exp2f(m[r] - ms);
            m[r] = mnew[r];
            mnew[r] = ms;
            l[r] *= alpha[r];
            lr[r] *= alpha[r];
        }
        uint32_t pf[4][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const float p0 = exp2f(fmaf(s[nt][0], c, -mnew[0]));
            const float p1 = exp2f(fmaf(s[nt][1], c, -mnew[0]));
            const float p2 = exp2f(fmaf(s[nt][2], c, -mnew[1]));
            const float p3 = exp2f(fmaf(s[nt][3], c, -mnew[1]));
            l[0] += p0 + p1;
            l[1] += p2 + p3;
            const uint32_t w01 = pack_bf16x2(p0, p1), w23 = pack_bf16x2(p2, p3);
            lr[0] += __uint_as_float(w01 << 16) + __uint_as_float(w01 & 0xffff0000u);
            lr[1] += __uint_as_float(w23 << 16) + __uint_as_float(w23 & 0xffff0000u);
            pf[nt >> 1][(nt & 1) * 2 + 0] = w01;
            pf[nt >> 1][(nt & 1) * 2 + 1] = w23;
        }
#pragma unroll
        for (int n = 0; n < NT; ++n) {
            o[n][0] *= alpha[0];
            o[n][1] *= alpha[0];
            o[n][2] *= alpha[1];
            o[n][3] *= alpha[1];
        }
        // O += P V
#pragma unroll
        for (int kt = 0; kt < 4; ++kt) {
            const __nv_bfloat16* vrow = Vt + (kt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * LD +
                                        (lane >> 4) * 8;
#pragma unroll
            for (int n2 = 0; n2 < NT / 2; ++n2) {
                uint32_t bfr[4];
                ldmatrix_x4_trans(bfr, vrow + n2 * 16);
                mma_bf16_16816(o[2 * n2], pf[kt], bfr[0], bfr[1]);
                mma_bf16_16816(o[2 * n2 + 1], pf[kt], bfr[2], bfr[3]);
            }
        }
        buf ^= 1;
        t = tn;
    }
    cp_async_wait_all();

    // finish the denominators across the quad, normalise, store
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        l[r] += __shfl_xor_sync(0xffffffffu, l[r], 1);
        l[r] += __shfl_xor_sync(0xffffffffu, l[r], 2);
        lr[r] += __shfl_xor_sync(0xffffffffu, lr[r], 1);
        lr[r] += __shfl_xor_sync(0xffffffffu, lr[r], 2);
    }
    const float inv[2] = {lr[0] > 0.f ? 1.f / lr[0] : 0.f, lr[1] > 0.f ? 1.f / lr[1] : 0.f};
    const int row_g[2] = {I * USV_BLOCK + warp * 16 + g, I * USV_BLOCK + warp * 16 + g + 8};

    if (a.lse != nullptr && tig == 0) {
#pragma unroll
        for (int r = 0; r < 2; ++r)
            if (row_g[r] < N)
                a.lse[((int64_t)b * a.H + h) * N + row_g[r]] =
                    l[r] > 0.f ? (m[r] + log2f(l[r])) * 0.69314718055994531f : 0.f;
    }
    if (a.o_f32 != nullptr) {
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            if (row_g[r] >= N) continue;
            float* dst = a.o_f32 + (((int64_t)b * a.H + h) * N + row_g[r]) * D + 2 * tig;
#pragma unroll
            for (int n = 0; n < NT; ++n)
                *reinterpret_cast<float2*>(dst + n * 8) =
                    make_float2(o[n][2 * r] * inv[r], o[n][2 * r + 1] * inv[r]);
        }
    }
    // bf16 output through this warp's own rows of the (now idle) Q tile for 16-byte stores
    __syncthreads();  // all warps are done reading Q fragments and K/V tiles
    __nv_bfloat16* stage = Qs + (warp * 16) * LD;
#pragma unroll
    for (int n = 0; n < NT; ++n) {
        *reinterpret_cast<uint32_t*>(stage + g * LD + n * 8 + 2 * tig) =
            pack_bf16x2(o[n][0] * inv[0], o[n][1] * inv[0]);
        *reinterpret_cast<uint32_t*>(stage + (g + 8) * LD + n * 8 + 2 * tig) =
            pack_bf16x2(o[n][2] * inv[1], o[n][3] * inv[1]);
    }
    __syncwarp();
    __nv_bfloat16* O = a.o + b * a.so.sb + h * a.so.sh;
    constexpr int VPR = D / 8;
    for (int idx = lane; idx < 16 * VPR; idx += 32) {
        const int r = idx / VPR, cc = idx % VPR;
        const int row = I * USV_BLOCK + warp * 16 + r;
        if (row < N)
            *reinterpret_cast<uint4*>(O + (int64_t)row * a.so.sn + cc * 8) =
                *reinterpret_cast<const uint4*>(stage + r * LD + cc * 8);
    }
}

// One CTA per query block, or (list mode) a fixed grid whose CTAs walk a device-side work list.
template <int D>
__global__ void __launch_bounds__(128) attn_mma_kernel(const AttnArgs a) {
    dep_sync();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    if (a.work_list == nullptr) {
        attn_mma_block<D>(a, blockIdx.x, smem_raw);
        return;
    }
    const int n = *a.work_count;
    for (int i = blockIdx.x; i < n; i += gridDim.x) {
        attn_mma_block<D>(a, a.work_list[i], smem_raw);
        __syncthreads();
    }
}

int launch_attn_mma(const AttnArgs& a, int d, cudaStream_t st) {
    int64_t grid = (int64_t)a.B * a.H * a.NB;
    if (grid > 2147483647LL) return fail(USV_ERR_UNSUPPORTED, "sparse_attn: too many query blocks");
    if (a.work_list != nullptr && grid > 296) grid = 296;
    if (d == 128) {
        cudaFuncSetAttribute(attn_mma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)MmaSmem<128>::BYTES);
        launch_dep(attn_mma_kernel<128>, dim3((unsigned)grid), dim3(128), MmaSmem<128>::BYTES, st, a);
    } else {
        cudaFuncSetAttribute(attn_mma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)MmaSmem<64>::BYTES);
        launch_dep(attn_mma_kernel<64>, dim3((unsigned)grid), dim3(128), MmaSmem<64>::BYTES, st, a);
    }
    USV_CHECK_LAUNCH("attn_mma_kernel");
    return USV_OK;
}

}  // namespace usv
