// Pairing plan of the block-sparse attention kernel.
//
// The tcgen05 kernel computes two query blocks per CTA over the UNION of their key-block lists,
// so it pays for every key block only one of the two selected.  Which blocks are paired is free:
// this file chooses, per (batch, head), a pairing with large list overlaps.
//
//   pair_overlap_kernel   overlap |sel(I) & sel(J)| for every J within PLAN_WINDOW blocks of I
//                         (bitmaps of the selection rows in shared memory, popcounts)
//   pair_match_kernel     PLAN_ROUNDS rounds of "mutual best unmatched neighbour" matching, then
//                         the blocks still single are paired in index order; output = the pairs
//                         (IA < IB, or IB = -1 for an odd block out), ordered by IA
//
// The result only affects speed: any pairing gives the same attention output.
#include "usv_attn.cuh"

namespace usv {

namespace plan {

constexpr int CH = 64;                 // query blocks per CTA of the overlap kernel
constexpr int W = PLAN_WINDOW;         // neighbours on each side
constexpr int ROUNDS = 5;

__global__ void __launch_bounds__(512)
pair_overlap_kernel(const AttnArgs a, uint16_t* __restrict__ ov) {
    extern __shared__ uint32_t bm[];   // [rows][nwords | 1]: odd row pitch, conflict-free column reads
    const int NB = a.NB;
    const int nwords = (NB + 31) >> 5;
    const int pitch = nwords | 1;
    const int bh = blockIdx.y;
    const int b = bh / a.H, h = bh % a.H;
    const int kh = a.k_per_head[h];
    if (kh >= NB) return;              // every list is the full set: pairing is arbitrary
    const int I0 = blockIdx.x * CH;
    const int lo = max(0, I0 - W), hi = min(NB, I0 + CH + W);   // rows held: [lo, hi)
    const int rows = hi - lo;
    for (int i = threadIdx.x; i < rows * pitch; i += blockDim.x) bm[i] = 0u;
    __syncthreads();
    const int32_t* sel = a.sel + ((int64_t)b * a.H + h) * NB * a.kmax;
    const int total = rows * kh;
    for (int i0 = threadIdx.x; i0 < total; i0 += 4 * blockDim.x) {
        int J[4], R[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {          // four independent loads in flight
            const int i = i0 + u * blockDim.x;
            R[u] = i < total ? i / kh : -1;
            J[u] = i < total ? sel[(int64_t)(lo + R[u]) * a.kmax + (i - R[u] * kh)] : -1;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (J[u] >= 0 && J[u] < NB) atomicOr(&bm[R[u] * pitch + (J[u] >> 5)], 1u << (J[u] & 31));
    }
    __syncthreads();
    const int nI = min(CH, NB - I0);
    uint16_t* out = ov + (((int64_t)b * a.H + h) * NB + I0) * (2 * W);
    for (int i = threadIdx.x; i < nI * 2 * W; i += blockDim.x) {
        const int ii = i / (2 * W), jj = i % (2 * W);
        const int I = I0 + ii;
        const int J = I - W + jj + (jj >= W ? 1 : 0);   // the 2W neighbours, I itself skipped
        int cnt = 0;
        if (J >= 0 && J < NB) {
            const uint32_t* x = bm + (I - lo) * pitch;
            const uint32_t* y = bm + (J - lo) * pitch;
            for (int w = 0; w < nwords; ++w) cnt += __popc(x[w] & y[w]);
        }
        out[i] = (uint16_t)min(cnt, 65535);
    }
}

// One CTA per (b, h).  partner/best live in shared memory (NB <= 4096).
__global__ void __launch_bounds__(1024)
pair_match_kernel(const AttnArgs a, const uint16_t* __restrict__ ov, int2* __restrict__ pairs) {
    __shared__ int16_t partner[4096];
    __shared__ int16_t best[4096];
    __shared__ int chunk_cnt[129];
    const int NB = a.NB;
    const int NP = (NB + 1) >> 1;
    const int bh = blockIdx.x;
    const int h = bh % a.H;
    int2* out = pairs + (int64_t)bh * NP;
    if (a.k_per_head[h] >= NB) {
        for (int p = threadIdx.x; p < NP; p += blockDim.x)
            out[p] = make_int2(2 * p, 2 * p + 1 < NB ? 2 * p + 1 : -1);
        return;
    }
    const uint16_t* o = ov + (int64_t)bh * NB * (2 * W);
    for (int i = threadIdx.x; i < NB; i += blockDim.x) partner[i] = -1;
    __syncthreads();
    // Two threads per query block (even lane: lower half of the window, odd lane: upper half).
    // The overlaps of a block never change, only who is still free.  Up to 512 blocks, each
    // thread keeps its 64 overlaps in registers across the rounds; beyond, they are re-read.
    static_assert(W == 64, "register staging below assumes a 64-block half window");
    const int half = threadIdx.x & 1;
    auto load_row = [&](int i, uint4* rv) {
        const uint4* row = reinterpret_cast<const uint4*>(o + (int64_t)i * (2 * W) + half * W);
#pragma unroll
        for (int u = 0; u < 8; ++u) rv[u] = __ldg(row + u);
    };
    auto find_best = [&](int i, const uint4* rv) {
        int bj = -1, bo = -1;
        if (i < NB && partner[i] < 0) {
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const uint32_t wv[4] = {rv[u].x, rv[u].y, rv[u].z, rv[u].w};
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int j = i - W + half * W + u * 8 + e + half;   // upper half skips i itself
                    const int v = (wv[e >> 1] >> ((e & 1) * 16)) & 0xffff;
                    if (j >= 0 && j < NB && partner[j] < 0 && v > bo) { bo = v; bj = j; }
                }
            }
        }
        // combine the two halves: larger overlap wins, ties go to the lower block (even lane)
        const int oo = __shfl_xor_sync(0xffffffffu, bo, 1);
        const int oj = __shfl_xor_sync(0xffffffffu, bj, 1);
        if (half == 0) {
            if (oo > bo) bj = oj;
            if (i < NB) best[i] = (int16_t)bj;
        }
    };
    auto mutual = [&]() {
        __syncthreads();
        for (int i = threadIdx.x; i < NB; i += blockDim.x) {
            const int j = best[i];
            if (j > i && best[j] == i) { partner[i] = (int16_t)j; partner[j] = (int16_t)i; }
        }
        __syncthreads();
    };
    if (NB <= 512) {
        const int i = threadIdx.x >> 1;
        uint4 rv[8];
        if (i < NB) load_row(i, rv);
        for (int r = 0; r < ROUNDS; ++r) {
            find_best(i, rv);
            mutual();
        }
    } else {
        for (int r = 0; r < ROUNDS; ++r) {
            for (int i0 = 0; i0 < NB; i0 += 512) {
                const int i = i0 + (threadIdx.x >> 1);
                uint4 rv[8];
                if (i < NB) load_row(i, rv);
                find_best(i, rv);
            }
            mutual();
        }
    }
    // blocks still single are paired in index order: ordered compaction in chunks of 32
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nchunks = (NB + 31) >> 5;
    for (int c = warp; c < nchunks; c += 32) {
        const int i = c * 32 + lane;
        const unsigned m = __ballot_sync(0xffffffffu, i < NB && partner[i] < 0);
        if (lane == 0) chunk_cnt[c] = __popc(m);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;
        for (int c = 0; c < nchunks; ++c) { const int n = chunk_cnt[c]; chunk_cnt[c] = run; run += n; }
        chunk_cnt[128] = run;
    }
    __syncthreads();
    for (int c = warp; c < nchunks; c += 32) {
        const int i = c * 32 + lane;
        const bool single = i < NB && partner[i] < 0;
        const unsigned m = __ballot_sync(0xffffffffu, single);
        if (single) best[chunk_cnt[c] + __popc(m & ((1u << lane) - 1u))] = (int16_t)i;   // rank -> index
    }
    __syncthreads();
    const int nsingle = chunk_cnt[128];
    for (int q = threadIdx.x; 2 * q + 1 < nsingle; q += blockDim.x) {
        const int x = best[2 * q], y = best[2 * q + 1];
        partner[x] = (int16_t)y;
        partner[y] = (int16_t)x;
    }
    __syncthreads();
    // pairs ordered by their lower block: ordered compaction of "I is the lower block of its pair"
    for (int c = warp; c < nchunks; c += 32) {
        const int i = c * 32 + lane;
        const unsigned m = __ballot_sync(0xffffffffu, i < NB && (partner[i] < 0 || partner[i] > i));
        if (lane == 0) chunk_cnt[c] = __popc(m);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;
        for (int c = 0; c < nchunks; ++c) { const int n = chunk_cnt[c]; chunk_cnt[c] = run; run += n; }
    }
    __syncthreads();
    for (int c = warp; c < nchunks; c += 32) {
        const int i = c * 32 + lane;
        const bool lower = i < NB && (partner[i] < 0 || partner[i] > i);
        const unsigned m = __ballot_sync(0xffffffffu, lower);
        if (lower) out[chunk_cnt[c] + __popc(m & ((1u << lane) - 1u))] = make_int2(i, partner[i]);
    }
}

}  // namespace plan

size_t pair_plan_bytes(int B, int H, int NB) {
    const size_t np = (size_t)(NB + 1) / 2;
    return align_up((size_t)B * H * np * sizeof(int2), 256) +
           align_up((size_t)B * H * NB * 2 * PLAN_WINDOW * sizeof(uint16_t), 256);
}

// pairs = first part of `mem`, overlaps = second part; mem holds pair_plan_bytes(B, H, NB).
int launch_pair_plan(const AttnArgs& a, void* mem, cudaStream_t st) {
    const size_t np = (size_t)(a.NB + 1) / 2;
    int2* pairs = static_cast<int2*>(mem);
    uint16_t* ov = reinterpret_cast<uint16_t*>(static_cast<char*>(mem) +
                                               align_up((size_t)a.B * a.H * np * sizeof(int2), 256));
    const int nwords = (a.NB + 31) >> 5;
    const size_t smem = (size_t)(plan::CH + 2 * plan::W) * (nwords | 1) * sizeof(uint32_t);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(plan::pair_overlap_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return fail(USV_ERR_CUDA, "sparse_attn: plan smem attribute: %s", cudaGetErrorString(e));
    }
    dim3 grid((a.NB + plan::CH - 1) / plan::CH, a.B * a.H);
    plan::pair_overlap_kernel<<<grid, 512, smem, st>>>(a, ov);
    USV_CHECK_LAUNCH("pair_overlap_kernel");
    plan::pair_match_kernel<<<a.B * a.H, 1024, 0, st>>>(a, ov, pairs);
    USV_CHECK_LAUNCH("pair_match_kernel");
    return USV_OK;
}

}  // namespace usv
