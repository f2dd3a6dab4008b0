// Block scores on the tensor cores: scores[bh, I, J] = scale * <qbar[bh,I,:], kbar[bh,J,:]>, d = 128.
//
// The scores decide integers (the top-k sets) and are an fp32 output of the ABI, so the fp32
// pooled means are split into THREE bf16 planes x = hi + mid + lo (24 significant bits) and a
// product is accumulated in fp32 from the six plane pairs that matter,
//     hi.hi + hi.mid + mid.hi + mid.mid + hi.lo + lo.hi        (dropped terms are <= 2^-24),
// i.e. 6 x 8 tcgen05.mma (M = N = 128, K = 16) per 128 x 128 tile: fp32-grade results at tensor
// speed.  Same skeleton as the merge matcher (usv_match_tc.cu): the 128 query-block rows of a
// CTA sit in TMEM as A operands, key-block rows stream through shared memory by TMA (2 stages),
// warp 4 = producer, warp 5 = MMA issuer, warps 0-3 read the fp32 tile out of TMEM (two buffers)
// and store it through a per-warp shared-memory transpose so that global stores are row-contiguous.
#include "usv_tcgen05.cuh"

namespace usv {

namespace sc {

using namespace t5;

constexpr int DM = 128;
constexpr int NPL = 3;                                  // bf16 planes per operand
constexpr int STAGES = 2;
constexpr uint32_t PLANE_BYTES = 128 * DM * 2;          // 32 KB: [d-half][128 rows][128 B]
constexpr uint32_t STAGE_BYTES = NPL * PLANE_BYTES;
constexpr uint32_t SM_B = 0;
constexpr uint32_t SM_T = SM_B + STAGES * STAGE_BYTES;  // float[4 warps][32][33] transpose buffers
constexpr uint32_t SM_BAR = SM_T + 4 * 32 * 33 * 4;
enum { B_AFULL = 0, B_BFULL = 1, B_BEMPTY = B_BFULL + STAGES, B_DFULL = B_BEMPTY + STAGES, B_DFREE = B_DFULL + 2,
       B_COUNT = B_DFREE + 2 };
constexpr uint32_t SM_MISC = SM_BAR + 8 * 16;
constexpr uint32_t SM_TOTAL = SM_MISC + 64;
constexpr size_t SMEM_BYTES = SM_TOTAL + 1024;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t TA = 0, TD = NPL * 64;               // A planes at 0, 64, 128; D buffers at 192 and 320

struct Args {
    int BH, NBq, NBk, NBq_pad, NBk_pad;
    __nv_bfloat16 *a_pl, *b_pl;         // [NPL][BH][NB_pad][128]
    float* scores;                      // [BH][NBq][NBk]
    float scale;
    unsigned int* status;
};

struct Maps {
    CUtensorMap b[NPL];
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}

__global__ void __launch_bounds__(192, 1)
scores_tc_kernel(const Args m, const __grid_constant__ Maps maps) {
    dep_launch();   // the set-up below touches shared and tensor memory only; dep_wait() follows it
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* sm = smem_raw + (base - raw);
    auto bar = [&](int i) { return base + SM_BAR + 8u * i; };
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(sm + SM_MISC);
    volatile int* s_abort = reinterpret_cast<volatile int*>(sm + SM_MISC + 4);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bh = blockIdx.y;
    const int i0 = blockIdx.x * 128;
    // key-block tiles [t_lo, t_hi) of this CTA: the column range is split over blockIdx.z so that
    // short problems still fill the GPU
    const int t_all = m.NBk_pad / 128;
    const int t_per = (t_all + gridDim.z - 1) / gridDim.z;
    const int t_lo = min(t_all, (int)blockIdx.z * t_per);
    const int T = min(t_all, t_lo + t_per) - t_lo;

    if (threadIdx.x == 0) {
        mbar_init(bar(B_AFULL), 4);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar(B_BFULL + s), 1);
            mbar_init(bar(B_BEMPTY + s), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(B_DFULL + s), 1);
            mbar_init(bar(B_DFREE + s), 4);
        }
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 5) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(base + SM_MISC), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_before();
    __syncthreads();
    fence_after();
    dep_wait();
    const uint32_t tmem = *s_tmem;

    if (warp == 4) {
        // ===== TMA producer: the three planes of 128 key-block rows per stage =====
        const int row0 = bh * m.NBk_pad;
        for (int t = 0; t < T; ++t) {
            const int s = t % STAGES;
            const uint32_t ph = (t / STAGES) & 1;
            if (!mbar_wait(bar(B_BEMPTY + s), ph ^ 1, s_abort, m.status, 0x10000)) break;
            const uint32_t dst = base + SM_B + s * STAGE_BYTES;
            if (elect_one()) {
                mbar_expect_tx(bar(B_BFULL + s), STAGE_BYTES);
#pragma unroll
                for (int p = 0; p < NPL; ++p) {
                    tma_load_2d(dst + p * PLANE_BYTES, &maps.b[p], bar(B_BFULL + s), 0, row0 + (t_lo + t) * 128);
                    tma_load_2d(dst + p * PLANE_BYTES + 16384, &maps.b[p], bar(B_BFULL + s), 64, row0 + (t_lo + t) * 128);
                }
            }
            __syncwarp();
        }
    } else if (warp == 5) {
        // ===== MMA issuer =====
        constexpr uint32_t IDESC = instr_desc(128, 128, 0, 0);   // A (TMEM) x B (K-major)
        const uint64_t bdesc0 = smem_desc(base + SM_B, 16, 1024);
        bool ok = mbar_wait(bar(B_AFULL), 0, s_abort, m.status, 0x20000);
        for (int t = 0; ok && t < T; ++t) {
            const int s = t % STAGES;
            const uint32_t ph = (t / STAGES) & 1;
            const int buf = t & 1;
            if (!mbar_wait(bar(B_BFULL + s), ph, s_abort, m.status, 0x40000)) break;
            if (t >= 2 && !mbar_wait(bar(B_DFREE + buf), ((t - 2) >> 1) & 1, s_abort, m.status, 0x80000)) break;
            fence_after();
            const uint64_t bst = bdesc0 + ((s * STAGE_BYTES) >> 4);
            const uint32_t d = tmem + TD + buf * 128;
            if (elect_one()) {
                // plane pairs (A, B): hi.hi, hi.mid, mid.hi, mid.mid, hi.lo, lo.hi
                constexpr int PA[6] = {0, 0, 1, 1, 0, 2};
                constexpr int PB[6] = {0, 1, 0, 1, 2, 0};
#pragma unroll
                for (int pass = 0; pass < 6; ++pass) {
                    const uint32_t ta = tmem + TA + PA[pass] * 64;
                    const uint64_t bd = bst + ((PB[pass] * PLANE_BYTES) >> 4);
#pragma unroll
                    for (int ks = 0; ks < DM / 16; ++ks)
                        umma_ts(d, ta + ks * 8, bd + (((ks >> 2) * 16384 + (ks & 3) * 32) >> 4), IDESC,
                                (pass > 0 || ks > 0));
                }
                umma_commit(bar(B_BEMPTY + s));
                umma_commit(bar(B_DFULL + buf));
            }
            __syncwarp();
        }
    } else {
        // ===== one thread per query-block row: A planes -> TMEM, then tiles TMEM -> global =====
        const int r = threadIdx.x;          // 0..127 = TMEM lane
        const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
        {
            const int64_t row = (int64_t)bh * m.NBq_pad + i0 + r;    // padded: always in range
            const int64_t plane = (int64_t)m.BH * m.NBq_pad * DM;
#pragma unroll
            for (int p = 0; p < NPL; ++p) {
                const uint4* src = reinterpret_cast<const uint4*>(m.a_pl + p * plane + row * DM);
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4) {
                    uint32_t q[16];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint4 v = __ldg(src + c4 * 4 + i);
                        q[4 * i] = v.x; q[4 * i + 1] = v.y; q[4 * i + 2] = v.z; q[4 * i + 3] = v.w;
                    }
                    tmem_st16(lane_base + TA + p * 64 + c4 * 16, q);
                }
            }
            tmem_wait_st();
            fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(B_AFULL));
        }
        float* tbuf = reinterpret_cast<float*>(sm + SM_T) + warp * (32 * 33);
        float* out = m.scores + ((int64_t)bh * m.NBq + i0 + warp * 32) * m.NBk;   // first row of this warp
        const int nrows = min(32, m.NBq - (i0 + warp * 32));                       // rows of this warp that exist
        for (int t = 0; t < T; ++t) {
            const int buf = t & 1;
            if (!mbar_wait(bar(B_DFULL + buf), (t >> 1) & 1, s_abort, m.status, 0x100000)) break;
            fence_after();
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                uint32_t sr[32];
                tmem_ld32(lane_base + TD + buf * 128 + ch * 32, sr);
                tmem_wait_ld();
                if (ch == 3) {
                    // the tile is in registers: hand the buffer back
                    fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(B_DFREE + buf));
                }
                // transpose through shared memory: lane = row -> lane = column
#pragma unroll
                for (int j = 0; j < 32; ++j) tbuf[lane * 33 + j] = __uint_as_float(sr[j]) * m.scale;
                __syncwarp();
                const int col = (t_lo + t) * 128 + ch * 32 + lane;
                if (col < m.NBk)
                    for (int rr = 0; rr < nrows; ++rr) out[(int64_t)rr * m.NBk + col] = tbuf[rr * 33 + lane];
                __syncwarp();
            }
        }
    }

    fence_before();
    __syncthreads();
    if (*s_abort) {
        const unsigned long long t0 = gtime();
        while (gtime() - t0 < 2000000ull) { }
        __syncthreads();
    }
    if (warp == 5) {
        fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
}

static int make_rows_map(CUtensorMap* map, const void* ptr, int64_t rows) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return fail(USV_ERR_CUDA, "block_scores: cuTensorMapEncodeTiled not available");
    cuuint64_t dims[2] = {(cuuint64_t)DM, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)DM * 2};
    cuuint32_t box[2] = {64, 128};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(USV_ERR_CUDA, "block_scores: cuTensorMapEncodeTiled failed with %d", (int)r);
    return USV_OK;
}

}  // namespace sc

static inline int pad128(int n) { return (n + 127) / 128 * 128; }

// bytes of the bf16 planes (256-byte aligned total)
size_t scores_tc_bytes(int BH, int NBq, int NBk) {
    return align_up((size_t)BH * ((size_t)pad128(NBq) + pad128(NBk)) * sc::DM * sc::NPL * sizeof(__nv_bfloat16), 256);
}

void scores_tc_planes(void* mem, int BH, int NBq, int NBk, __nv_bfloat16** a_pl, __nv_bfloat16** b_pl,
                      int* NBq_pad, int* NBk_pad) {
    *NBq_pad = pad128(NBq);
    *NBk_pad = pad128(NBk);
    *a_pl = static_cast<__nv_bfloat16*>(mem);
    *b_pl = *a_pl + (size_t)sc::NPL * BH * *NBq_pad * sc::DM;
}

int launch_scores_tc(float* scores, int BH, int NBq, int NBk, float scale, void* mem, unsigned int* status,
                     cudaStream_t st) {
    sc::Args m;
    m.BH = BH; m.NBq = NBq; m.NBk = NBk;
    m.scores = scores; m.scale = scale;
    m.status = status;
    scores_tc_planes(mem, BH, NBq, NBk, &m.a_pl, &m.b_pl, &m.NBq_pad, &m.NBk_pad);
    cudaError_t e;
    sc::Maps maps;
    const int64_t brows = (int64_t)BH * m.NBk_pad;
    for (int p = 0; p < sc::NPL; ++p) {
        int rc = sc::make_rows_map(&maps.b[p], m.b_pl + (size_t)p * brows * sc::DM, brows);
        if (rc != USV_OK) return rc;
    }
    e = cudaFuncSetAttribute(sc::scores_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sc::SMEM_BYTES);
    if (e != cudaSuccess) return fail(USV_ERR_CUDA, "block_scores: smem attribute: %s", cudaGetErrorString(e));
    const int ctas = (m.NBq_pad / 128) * BH, t_all = m.NBk_pad / 128;
    // One CTA per SM is resident: split the key-block tiles over blockIdx.z only as far as the
    // grid still fits one wave (148 SMs), so that no CTA pays its set-up for a single tile twice.
    int nz = 148 / ctas;
    nz = nz < 1 ? 1 : (nz > t_all ? t_all : nz);
    nz = (t_all + (t_all + nz - 1) / nz - 1) / ((t_all + nz - 1) / nz);   // slices that hold at least one tile
    dim3 grid(m.NBq_pad / 128, BH, nz);
    launch_dep(sc::scores_tc_kernel, dim3(grid), dim3(192), sc::SMEM_BYTES, st, m, maps);
    USV_CHECK_LAUNCH("scores_tc_kernel");
    return USV_OK;
}

}  // namespace usv
