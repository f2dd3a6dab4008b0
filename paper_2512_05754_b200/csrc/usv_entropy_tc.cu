// Key marginal of the block-masked attention (Sec. 3.4, Eq. 16) on the 5th-generation tensor
// cores, d = 128.
//
//     abar[b,j] = 1/(H N) sum_h sum_i A(h,i,j),   A(h,i,j) = exp(scale <q_i,k_j> - lse_i)
//
// with lse_i the log-sum-exp the attention forward wrote.  Only the logits are needed, and the
// sum runs over the queries, so the product is taken transposed: one CTA per (b, h, query block)
// walks the block's selected key blocks two at a time and computes
//
//     S^T[128 keys x 64 queries] = K_tile . Q^T      tcgen05.mma, A = K tile in smem, B = Q in smem
//
// into one of four 64-column TMEM buffers.  Keys live on TMEM lanes: thread r of the four
// consumer warps owns key r of the tile, exponentiates its 64 logits against the queries'
// log-sum-exp (held in registers) and adds the sum to abar with one atomic per key and tile.
// A CTA needs 82 KB of shared memory and 256 TMEM columns, so two share an SM and fill each
// other's gaps.  Warp 4 is the TMA producer, warp 5 the MMA issuer and TMEM owner.  All waits
// are bounded; a role that gives up raises the CTA's abort flag and the others follow.
#include "usv_entropy.cuh"
#include "usv_tcgen05.cuh"

namespace usv {

namespace et {

using namespace t5;

constexpr int D = 128;
constexpr int KT = 2 * USV_BLOCK;               // keys per tile = two key blocks
constexpr int KSTAGES = 2;                      // two CTAs share an SM and cover each other's waits
constexpr int NBUF = 4;                         // S^T buffers of 64 columns
constexpr uint32_t TILE_BYTES = KT * D * 2;     // 32 KB: [d-half][128 keys][128 B]
constexpr uint32_t Q_BYTES = USV_BLOCK * D * 2; // 16 KB: [d-half][64 queries][128 B]
constexpr uint32_t SM_Q = 0;
constexpr uint32_t SM_K = SM_Q + Q_BYTES;
constexpr uint32_t SM_BAR = SM_K + KSTAGES * TILE_BYTES;
enum { B_QFULL = 0, B_KFULL, B_KEMPTY = B_KFULL + KSTAGES, B_SFULL = B_KEMPTY + KSTAGES,
       B_SFREE = B_SFULL + NBUF, B_COUNT = B_SFREE + NBUF };
constexpr uint32_t SM_MISC = SM_BAR + 8 * 16;   // tmem base, abort flag
constexpr uint32_t SM_TOTAL = SM_MISC + 64;
constexpr size_t SMEM_BYTES = SM_TOTAL + 1024;  // + slack for 1024-byte alignment
static_assert(B_COUNT <= 16, "barrier area");
static_assert(2 * SMEM_BYTES <= 232448, "two CTAs per SM");

constexpr uint32_t TMEM_COLS = 256;
constexpr int NCONS = 128;                      // consumer threads
constexpr int NTHREADS = NCONS + 64;
constexpr int W_TMA = NCONS / 32, W_MMA = NCONS / 32 + 1;

struct Maps {
    CUtensorMap q, k;
};

__global__ void __launch_bounds__(NTHREADS, 2)
marginal_tc_kernel(const MargArgs a, const __grid_constant__ Maps maps) {
    dep_launch();   // the set-up below touches shared and tensor memory only; dep_wait() follows it
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* sm = smem_raw + (base - raw);
    auto bar = [&](int i) { return base + SM_BAR + 8u * i; };
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(sm + SM_MISC);
    volatile int* s_abort = reinterpret_cast<volatile int*>(sm + SM_MISC + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int N = a.N;
    const int I = blockIdx.x % a.NB;
    const int bh = blockIdx.x / a.NB;
    const int b = bh / a.H, h = bh % a.H;
    const int kh = a.k_per_head[h];
    const int T = (kh + 1) >> 1;   // tiles of two list entries
    const int32_t* sel = a.sel + ((int64_t)bh * a.NB + I) * a.kmax;

    if (threadIdx.x < B_COUNT) {
        const int i = threadIdx.x;
        mbar_init(bar(i), (i >= B_SFREE && i < B_SFREE + NBUF) ? NCONS / 32 : 1);
        if (i == 0) *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == W_MMA) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(base + SM_MISC), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_before();
    __syncthreads();
    fence_after();
    dep_wait();
    const uint32_t tmem = *s_tmem;

    if (warp == W_TMA) {
        // ===== producer: the query block once, then the key tiles =================================
        if (elect_one()) {
            mbar_expect_tx(bar(B_QFULL), Q_BYTES);
            tma_load_4d(base + SM_Q, &maps.q, bar(B_QFULL), 0, I * USV_BLOCK, h, b);
            tma_load_4d(base + SM_Q + 8192, &maps.q, bar(B_QFULL), 64, I * USV_BLOCK, h, b);
        }
        __syncwarp();
        int n0 = T > 0 ? sel[0] : -1, n1 = (T > 0 && 1 < kh) ? sel[1] : -1;   // entries of the next tile, fetched ahead
        for (int t = 0; t < T; ++t) {
            const int s = t % KSTAGES;
            const uint32_t ph = (t / KSTAGES) & 1;
            // an entry may be -1 (no block): any finite tile will do, its keys are not counted
            const int e0 = n0, e1 = n1;
            n0 = (2 * t + 2 < kh) ? sel[2 * t + 2] : -1;
            n1 = (2 * t + 3 < kh) ? sel[2 * t + 3] : -1;
            const int J0 = e0 >= 0 ? e0 : 0, J1 = e1 >= 0 ? e1 : J0;
            if (!mbar_wait(bar(B_KEMPTY + s), ph ^ 1, s_abort, a.status, 0x1000000u)) break;
            const uint32_t dst = base + SM_K + s * TILE_BYTES;
            if (elect_one()) {
                mbar_expect_tx(bar(B_KFULL + s), TILE_BYTES);
                tma_load_4d(dst, &maps.k, bar(B_KFULL + s), 0, J0 * USV_BLOCK, h, b);
                tma_load_4d(dst + 8192, &maps.k, bar(B_KFULL + s), 0, J1 * USV_BLOCK, h, b);
                tma_load_4d(dst + 16384, &maps.k, bar(B_KFULL + s), 64, J0 * USV_BLOCK, h, b);
                tma_load_4d(dst + 24576, &maps.k, bar(B_KFULL + s), 64, J1 * USV_BLOCK, h, b);
            }
            __syncwarp();
        }
    } else if (warp == W_MMA) {
        // ===== MMA issuer ==========================================================================
        constexpr uint32_t IDESC = instr_desc(128, USV_BLOCK, 0, 0);    // K tile (K-major) x Q (K-major)
        const uint64_t kdesc0 = smem_desc(base + SM_K, 16, 1024);
        const uint64_t qdesc0 = smem_desc(base + SM_Q, 16, 1024);
        bool ok = mbar_wait(bar(B_QFULL), 0, s_abort, a.status, 0x2000000u);
        for (int t = 0; ok && t < T; ++t) {
            const int s = t % KSTAGES;
            const int bf = t % NBUF;
            if (!mbar_wait(bar(B_KFULL + s), (t / KSTAGES) & 1, s_abort, a.status, 0x4000000u)) break;
            if (t >= NBUF && !mbar_wait(bar(B_SFREE + bf), ((t / NBUF) - 1) & 1, s_abort, a.status, 0x8000000u)) break;
            fence_after();
            const uint64_t kdesc = kdesc0 + ((s * TILE_BYTES) >> 4);
            if (elect_one()) {
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks)
                    umma_ss(tmem + bf * 64, kdesc + (((ks >> 2) * 16384 + (ks & 3) * 32) >> 4),
                            qdesc0 + (((ks >> 2) * 8192 + (ks & 3) * 32) >> 4), IDESC, ks > 0);
                umma_commit(bar(B_SFULL + bf));
                umma_commit(bar(B_KEMPTY + s));
            }
            __syncwarp();
        }
    } else {
        // ===== consumers: thread r <-> TMEM lane r <-> key r of the tile ===========================
        const int r = threadIdx.x;
        const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
        const float c = a.scale_log2;
        // minus the base-2 log-sum-exp of the block's 64 queries; a query at or beyond N counts nothing
        float nl2[USV_BLOCK];
#pragma unroll
        for (int qi = 0; qi < USV_BLOCK; ++qi) {
            const int row = I * USV_BLOCK + qi;
            nl2[qi] = row < N ? -a.lse[(int64_t)bh * N + row] * 1.4426950408889634f : -INFINITY;
        }
        float* marg = a.marg + (int64_t)b * N;
        for (int t = 0; t < T; ++t) {
            const int bf = t % NBUF;
            const int e = (2 * t + (r >> 6) < kh) ? sel[2 * t + (r >> 6)] : -1;   // this key's block
            if (!mbar_wait(bar(B_SFULL + bf), (t / NBUF) & 1, s_abort, a.status, 0x10000000u)) break;
            fence_after();
            uint32_t s0[32], s1[32];
            tmem_ld32(lane_base + bf * 64, s0);
            tmem_ld32(lane_base + bf * 64 + 32, s1);
            tmem_wait_ld();
            fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(B_SFREE + bf));   // the logits are in registers
            float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
            for (int qi = 0; qi < 32; ++qi) {
                acc0 += ex2(fmaf(__uint_as_float(s0[qi]), c, nl2[qi]));
                acc1 += ex2(fmaf(__uint_as_float(s1[qi]), c, nl2[32 + qi]));
            }
            const int j = e * USV_BLOCK + (r & 63);
            if (e >= 0 && j < N) atomicAdd(marg + j, (acc0 + acc1) * a.inv_hn);
        }
    }

    // ---- teardown
    fence_before();
    __syncthreads();
    if (*s_abort) {
        // give copies and MMAs that may still be in flight time to land before the CTA's
        // shared memory and TMEM are handed back
        const unsigned long long t0 = gtime();
        while (gtime() - t0 < 2000000ull) { }
        __syncthreads();
    }
    if (warp == W_MMA) {
        fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
}

}  // namespace et

int launch_marginal_tc(const MargArgs& a, cudaStream_t st) {
    et::Maps maps;
    int rc;
    if ((rc = t5::make_bhnd_map(&maps.q, a.q, a.sq, a.B, a.H, a.N, et::D, "q")) != USV_OK) return rc;
    if ((rc = t5::make_bhnd_map(&maps.k, a.k, a.sk, a.B, a.H, a.N, et::D, "k")) != USV_OK) return rc;
    const int64_t grid = (int64_t)a.B * a.H * a.NB;
    cudaError_t e = cudaFuncSetAttribute(et::marginal_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)et::SMEM_BYTES);
    if (e != cudaSuccess) return fail(USV_ERR_CUDA, "attn_entropy: smem attribute: %s", cudaGetErrorString(e));
    launch_dep(et::marginal_tc_kernel, dim3((unsigned)grid), dim3(et::NTHREADS), et::SMEM_BYTES, st, a, maps);
    USV_CHECK_LAUNCH("marginal_tc_kernel");
    return USV_OK;
}

}  // namespace usv
