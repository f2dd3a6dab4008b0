// Bipartite matching of token merge (Sec. 3.3, Eq. 8-9) on the tensor cores: for every source
// token the destination with the largest cosine, ties to the lowest destination.
//
// The cosines decide an integer (the arg-max) that is compared with an fp64 evaluation, so plain
// bf16 operands (2^-9 relative) are not enough.  Each fp32 unit descriptor x is split into
// hi = bf16(x) and lo = bf16(x - hi), and a cosine is accumulated in fp32 from three products,
//     <hi_a, hi_b> + <hi_a, lo_b> + <lo_a, hi_b>          (the dropped lo.lo term is ~2^-18),
// i.e. 3 x 8 tcgen05.mma (M = 128 sources, N = 128 destinations, K = 16) per 128 x 128 tile:
// an absolute error of a few 1e-6, two orders below the 1e-3 near-tie band.  The reported
// confidence u is afterwards recomputed in fp32 for the chosen destination only.
//
//   split_kernel     fp32 descriptors -> compact bf16 hi/lo rows, sources (by rank) and
//                    destinations (by ordinal) apart, zero-padded to multiples of 128 rows
//   match_tc_kernel  one CTA per 128 sources: their hi/lo rows sit in TMEM as A operands, the
//                    destination rows stream through shared memory (TMA, 2 stages); warp 4 =
//                    TMA producer, warp 5 = MMA issuer, warps 0-3 = one thread per source row
//                    reading the 128 x 128 cosine tile out of TMEM (two buffers) for a running
//                    arg-max in ascending destination order
//   rescore_kernel   u = <m_a, m_j*> in fp32
#include "usv_match.cuh"
#include "usv_tcgen05.cuh"

namespace usv {

namespace mt {

using namespace t5;

constexpr int DM = 128;
constexpr int STAGES = 2;
constexpr uint32_t HALF_BYTES = 128 * DM * 2;           // 32 KB: hi (or lo) rows of a tile, [d-half][128 rows][128 B]
constexpr uint32_t STAGE_BYTES = 2 * HALF_BYTES;        // hi then lo
constexpr uint32_t SM_B = 0;
constexpr uint32_t SM_BAR = SM_B + STAGES * STAGE_BYTES;
enum { B_AFULL = 0, B_BFULL = 1, B_BEMPTY = B_BFULL + STAGES, B_DFULL = B_BEMPTY + STAGES, B_DFREE = B_DFULL + 2,
       B_COUNT = B_DFREE + 2 };
constexpr uint32_t SM_MISC = SM_BAR + 8 * 16;
constexpr uint32_t SM_TOTAL = SM_MISC + 64;
constexpr size_t SMEM_BYTES = SM_TOTAL + 1024;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t TA_HI = 0, TA_LO = 64, TD = 128;     // D buffers at 128 and 256

// hi and lo are separate planes, so that one 2-D tensor map (128 x rows) covers each
__global__ void __launch_bounds__(256)
split_kernel(const float* __restrict__ mhat, MatchTcArgs m) {
    // one warp per output row (4 floats per lane)
    const int64_t gw = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    const int64_t rows_a = (int64_t)m.B * m.nA_pad, rows_b = (int64_t)m.B * m.nB_pad;
    if (gw >= rows_a + rows_b) return;
    const bool is_b = gw >= rows_a;
    const int64_t rr = is_b ? gw - rows_a : gw;
    const int pad = is_b ? m.nB_pad : m.nA_pad, cnt = is_b ? m.p.nB : m.nA;
    const int b = (int)(rr / pad), i = (int)(rr % pad);
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i < cnt) {
        const int tok = is_b ? m.p.dst_token(i) : m.src_idx[i];
        v = *reinterpret_cast<const float4*>(mhat + ((int64_t)b * m.N + tok) * DM + lane * 4);
    }
    const float x[4] = {v.x, v.y, v.z, v.w};
    __nv_bfloat16 hi[4], lo[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        hi[e] = __float2bfloat16_rn(x[e]);
        lo[e] = __float2bfloat16_rn(x[e] - __bfloat162float(hi[e]));
    }
    __nv_bfloat16* ph = (is_b ? m.b_hi : m.a_hi) + rr * DM + lane * 4;
    __nv_bfloat16* pl = (is_b ? m.b_lo : m.a_lo) + rr * DM + lane * 4;
    *reinterpret_cast<uint2*>(ph) = *reinterpret_cast<const uint2*>(hi);
    *reinterpret_cast<uint2*>(pl) = *reinterpret_cast<const uint2*>(lo);
}

struct Maps {
    CUtensorMap b_hi, b_lo;
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}

__global__ void __launch_bounds__(224, 1)
match_tc_kernel(const MatchTcArgs m, const __grid_constant__ Maps maps) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* sm = smem_raw + (base - raw);
    auto bar = [&](int i) { return base + SM_BAR + 8u * i; };
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(sm + SM_MISC);
    volatile int* s_abort = reinterpret_cast<volatile int*>(sm + SM_MISC + 4);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.y;
    const int a0 = blockIdx.x * 128;
    const int T = m.nB_pad / 128;   // destination tiles

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
    const uint32_t tmem = *s_tmem;

    if (warp == 4) {
        // ===== TMA producer: destination rows, hi plane then lo plane =====
        const int row0 = b * m.nB_pad;
        for (int t = 0; t < T; ++t) {
            const int s = t % STAGES;
            const uint32_t ph = (t / STAGES) & 1;
            if (!mbar_wait(bar(B_BEMPTY + s), ph ^ 1, s_abort, m.status, 0x10000)) break;
            const uint32_t dst = base + SM_B + s * STAGE_BYTES;
            if (elect_one()) {
                mbar_expect_tx(bar(B_BFULL + s), STAGE_BYTES);
                tma_load_2d(dst, &maps.b_hi, bar(B_BFULL + s), 0, row0 + t * 128);
                tma_load_2d(dst + 16384, &maps.b_hi, bar(B_BFULL + s), 64, row0 + t * 128);
                tma_load_2d(dst + 32768, &maps.b_lo, bar(B_BFULL + s), 0, row0 + t * 128);
                tma_load_2d(dst + 49152, &maps.b_lo, bar(B_BFULL + s), 64, row0 + t * 128);
            }
            __syncwarp();
        }
    } else if (warp == 5 || warp == 6) {
        // ===== two MMA issuers: warp 5 takes the even tiles, warp 6 the odd ones (each tile has its
        // own B stage and D buffer), so that one warp's barrier waits fall under the other's MMAs =====
        constexpr uint32_t IDESC = instr_desc(128, 128, 0, 0);   // A (TMEM) x B (K-major)
        const uint64_t bdesc0 = smem_desc(base + SM_B, 16, 1024);
        bool ok = mbar_wait(bar(B_AFULL), 0, s_abort, m.status, 0x20000);
        for (int t = warp - 5; ok && t < T; t += 2) {
            const int s = t % STAGES;
            const uint32_t ph = (t / STAGES) & 1;
            const int buf = t & 1;
            if (!mbar_wait(bar(B_BFULL + s), ph, s_abort, m.status, 0x40000)) break;
            if (t >= 2 && !mbar_wait(bar(B_DFREE + buf), ((t - 2) >> 1) & 1, s_abort, m.status, 0x80000)) break;
            fence_after();
            const uint64_t bhi = bdesc0 + ((s * STAGE_BYTES) >> 4);
            const uint64_t blo = bhi + (HALF_BYTES >> 4);
            const uint32_t d = tmem + TD + buf * 128;
            if (elect_one()) {
#pragma unroll
                for (int pass = 0; pass < 3; ++pass) {
                    const uint32_t ta = tmem + (pass == 2 ? TA_LO : TA_HI);
                    const uint64_t bd = pass == 1 ? blo : bhi;
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
        // ===== one thread per source row: A rows -> TMEM, then the running arg-max =====
        const int r = threadIdx.x;          // 0..127 = TMEM lane
        const int a = a0 + r;
        const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
        {
            const int64_t row = (int64_t)b * m.nA_pad + a;    // padded: always in range
            const uint4* ph = reinterpret_cast<const uint4*>(m.a_hi + row * DM);
            const uint4* pl = reinterpret_cast<const uint4*>(m.a_lo + row * DM);
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
                uint32_t q[16];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint4 v = __ldg(ph + c4 * 4 + i);
                    q[4 * i] = v.x; q[4 * i + 1] = v.y; q[4 * i + 2] = v.z; q[4 * i + 3] = v.w;
                }
                tmem_st16(lane_base + TA_HI + c4 * 16, q);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint4 v = __ldg(pl + c4 * 4 + i);
                    q[4 * i] = v.x; q[4 * i + 1] = v.y; q[4 * i + 2] = v.z; q[4 * i + 3] = v.w;
                }
                tmem_st16(lane_base + TA_LO + c4 * 16, q);
            }
            tmem_wait_st();
            fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(B_AFULL));
        }
        float best = -INFINITY;
        int bi = 0;
        bool ok = true;
        for (int t = 0; t < T; ++t) {
            const int buf = t & 1;
            if (!mbar_wait(bar(B_DFULL + buf), (t >> 1) & 1, s_abort, m.status, 0x100000)) { ok = false; break; }
            fence_after();
            const int nvalid = m.p.nB - t * 128;   // destinations of this tile that exist
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
                // The chunk's maximum first, on four independent chains (a running compare over
                // all 32 would be one long dependent chain); only a chunk that beats the best so far
                // is searched for where.  Ascending destination order and strict improvement: equal
                // cosines keep the lowest destination.
                if (nvalid < 128) {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (ch * 32 + j >= nvalid) sr[j] = 0xff800000u;   // -inf: a destination that does not exist
                }
                float c0 = __uint_as_float(sr[0]), c1 = __uint_as_float(sr[1]), c2 = __uint_as_float(sr[2]),
                      c3 = __uint_as_float(sr[3]);
#pragma unroll
                for (int j = 4; j < 32; j += 4) {
                    c0 = fmaxf(c0, __uint_as_float(sr[j]));
                    c1 = fmaxf(c1, __uint_as_float(sr[j + 1]));
                    c2 = fmaxf(c2, __uint_as_float(sr[j + 2]));
                    c3 = fmaxf(c3, __uint_as_float(sr[j + 3]));
                }
                const float cm = fmaxf(fmaxf(c0, c1), fmaxf(c2, c3));
                if (cm > best) {
                    best = cm;
                    int jj = 31;
#pragma unroll
                    for (int j = 30; j >= 0; --j)
                        if (__uint_as_float(sr[j]) == cm) jj = j;
                    bi = t * 128 + ch * 32 + jj;
                }
            }
        }
        if (ok && a < m.nA) {
            m.jstar_s[(int64_t)b * m.nA + a] = m.p.dst_token(bi);
            m.u_s[(int64_t)b * m.nA + a] = best;
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

// u = <m_a, m_j*(a)> in fp32, one warp per source
__global__ void __launch_bounds__(256)
rescore_kernel(const float* __restrict__ mhat, MatchTcArgs m) {
    const int64_t gw = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (gw >= (int64_t)m.B * m.nA) return;
    const int b = (int)(gw / m.nA), a = (int)(gw % m.nA);
    const float* M = mhat + (int64_t)b * m.N * DM;
    const float4 x = *reinterpret_cast<const float4*>(M + (int64_t)m.src_idx[a] * DM + lane * 4);
    const float4 y = *reinterpret_cast<const float4*>(M + (int64_t)m.jstar_s[gw] * DM + lane * 4);
    float acc = fmaf(x.x, y.x, fmaf(x.y, y.y, fmaf(x.z, y.z, x.w * y.w)));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) m.u_s[gw] = acc;
}

static int make_rows_map(CUtensorMap* map, const void* ptr, int64_t rows, const char* name) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return fail(USV_ERR_CUDA, "token_merge: cuTensorMapEncodeTiled not available");
    cuuint64_t dims[2] = {(cuuint64_t)DM, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)DM * 2};
    cuuint32_t box[2] = {64, 128};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(USV_ERR_CUDA, "token_merge: cuTensorMapEncodeTiled(%s) failed with %d", name, (int)r);
    return USV_OK;
}

}  // namespace mt

static inline int pad128(int n) { return (n + 127) / 128 * 128; }

size_t match_tc_bytes(int B, int N) {
    // sources + destinations = N rows, each side padded to 128: at most N + 254 rows; hi + lo planes
    return align_up((size_t)B * ((size_t)N + 256) * mt::DM * 2 * sizeof(__nv_bfloat16), 256);
}

int launch_match_tc(const float* mhat, const Part& p, int B, int N, int nA, const int32_t* src_idx,
                    int32_t* jstar_s, float* u_s, void* mem, unsigned int* status, cudaStream_t st) {
    MatchTcArgs m;
    m.p = p; m.B = B; m.N = N; m.nA = nA;
    m.nA_pad = pad128(nA); m.nB_pad = pad128(p.nB);
    m.src_idx = src_idx; m.jstar_s = jstar_s; m.u_s = u_s; m.status = status;
    __nv_bfloat16* base = static_cast<__nv_bfloat16*>(mem);
    const size_t na = (size_t)B * m.nA_pad * mt::DM, nb = (size_t)B * m.nB_pad * mt::DM;
    m.a_hi = base; m.a_lo = base + na; m.b_hi = base + 2 * na; m.b_lo = base + 2 * na + nb;
    const int64_t rows = (int64_t)B * (m.nA_pad + m.nB_pad);
    mt::split_kernel<<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(mhat, m);
    USV_CHECK_LAUNCH("split_kernel");
    mt::Maps maps;
    int rc;
    if ((rc = mt::make_rows_map(&maps.b_hi, m.b_hi, (int64_t)B * m.nB_pad, "b_hi")) != USV_OK) return rc;
    if ((rc = mt::make_rows_map(&maps.b_lo, m.b_lo, (int64_t)B * m.nB_pad, "b_lo")) != USV_OK) return rc;
    cudaError_t e = cudaFuncSetAttribute(mt::match_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)mt::SMEM_BYTES);
    if (e != cudaSuccess) return fail(USV_ERR_CUDA, "token_merge: smem attribute: %s", cudaGetErrorString(e));
    dim3 grid(m.nA_pad / 128, B);
    mt::match_tc_kernel<<<grid, 224, mt::SMEM_BYTES, st>>>(m, maps);
    USV_CHECK_LAUNCH("match_tc_kernel");
    const int64_t srcs = (int64_t)B * nA;
    mt::rescore_kernel<<<(unsigned)((srcs + 7) / 8), 256, 0, st>>>(mhat, m);
    USV_CHECK_LAUNCH("rescore_kernel");
    return USV_OK;
}

}  // namespace usv
