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
//   pair_list_kernel      ascending union of the two selection rows of every pair, each entry
//                         flagged with the side(s) that selected it (one warp per pair)
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
    __shared__ uint32_t freebits[128 + 6];
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
    for (int w = threadIdx.x; w < 128 + 6; w += blockDim.x) {
        const int first = (w - 3) * 32;               // block of bit 0 of this word
        freebits[w] = (w < 3 || first >= NB) ? 0u : (NB - first >= 32 ? 0xffffffffu : (1u << (NB - first)) - 1u);
    }
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
    // free[]: one bit per block, set while the block is unmatched; 3 zero words of padding on
    // each side so that a 64-bit window may hang over either end
    auto window = [&](int j0) -> unsigned long long {
        const int q = j0 + 96;                       // >= 0
        const uint32_t* w = freebits + (q >> 5);     // freebits[3] holds blocks 0..31
        const int sh = q & 31;
        const uint32_t lo = __funnelshift_r(w[0], w[1], sh), hi = __funnelshift_r(w[1], w[2], sh);
        return ((unsigned long long)hi << 32) | lo;
    };
    auto find_best = [&](int i, const uint4* rv) {
        // branch-free arg-max over this thread's 64 candidates: key = overlap << 8 | (63 - e), so
        // that equal overlaps resolve to the lowest block
        uint32_t bk = 0;
        const int j0 = i - W + half * (W + 1);       // upper half skips i itself
        if (i < NB && partner[i] < 0) {
            const unsigned long long m = window(j0);
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const uint32_t wv[4] = {rv[u].x, rv[u].y, rv[u].z, rv[u].w};
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int c = u * 8 + e;
                    const uint32_t v = (wv[e >> 1] >> ((e & 1) * 16)) & 0xffffu;
                    const uint32_t key = ((v + 1u) << 8) | (uint32_t)(63 - c);
                    bk = max(bk, ((m >> c) & 1ull) ? key : 0u);
                }
            }
        }
        int bo = (int)(bk >> 8) - 1;                                  // -1: no free candidate
        int bj = bk ? j0 + 63 - (int)(bk & 0xffu) : -1;
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
            if (j > i && best[j] == i) {
                partner[i] = (int16_t)j;
                partner[j] = (int16_t)i;
                atomicAnd(&freebits[3 + (i >> 5)], ~(1u << (i & 31)));
                atomicAnd(&freebits[3 + (j >> 5)], ~(1u << (j & 31)));
            }
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

// One warp per pair: bitmaps of the two selection rows in shared memory, then an ordered
// compaction of their union into the pair's list.
constexpr int LIST_WARPS = 8;

__global__ void __launch_bounds__(LIST_WARPS * 32)
pair_list_kernel(const AttnArgs a, const int2* __restrict__ pairs, int* __restrict__ lists) {
    extern __shared__ uint32_t bm[];   // [LIST_WARPS][2][nwords]
    const int NB = a.NB;
    const int NP = (NB + 1) >> 1;
    const int nwords = (NB + 31) >> 5;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bh = blockIdx.y;
    const int b = bh / a.H, h = bh % a.H;
    const int kh = a.k_per_head[h];
    const int pair = blockIdx.x * LIST_WARPS + warp;
    if (pair >= NP) return;
    const int2 pq = pairs[(int64_t)bh * NP + pair];
    uint32_t* bitsA = bm + (warp * 2) * nwords;
    uint32_t* bitsB = bitsA + nwords;
    for (int w = lane; w < nwords; w += 32) { bitsA[w] = 0u; bitsB[w] = 0u; }
    __syncwarp();
    const int32_t* selA = a.sel + ((int64_t)bh * NB + pq.x) * a.kmax;
    for (int t = lane; t < kh; t += 32) {
        const int J = selA[t];
        if (J >= 0 && J < NB) atomicOr(&bitsA[J >> 5], 1u << (J & 31));
    }
    if (pq.y >= 0) {
        const int32_t* selB = a.sel + ((int64_t)bh * NB + pq.y) * a.kmax;
        for (int t = lane; t < kh; t += 32) {
            const int J = selB[t];
            if (J >= 0 && J < NB) atomicOr(&bitsB[J >> 5], 1u << (J & 31));
        }
    }
    __syncwarp();
    int* out = lists + b * a.list_batch + a.list_off[h] + pair * list_stride(kh, NB);
    int running = 0;
    for (int w0 = 0; w0 < nwords; w0 += 32) {
        const int w = w0 + lane;
        const uint32_t ba = w < nwords ? bitsA[w] : 0u;
        const uint32_t bb = w < nwords ? bitsB[w] : 0u;
        uint32_t u = ba | bb;
        const int incl = warp_incl_scan(__popc(u));
        int off = running + incl - __popc(u);
        while (u) {
            const int bit = __ffs(u) - 1;
            u &= u - 1;
            out[1 + off++] = ((w * 32 + bit) << 2) | ((ba >> bit) & 1u) | (((bb >> bit) & 1u) << 1);
        }
        running += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) out[0] = running;
}

}  // namespace plan

static size_t pairs_bytes(int B, int H, int NB) {
    return align_up((size_t)B * H * ((size_t)(NB + 1) / 2) * sizeof(int2), 256);
}
static size_t overlap_bytes(int B, int H, int NB) {
    return align_up((size_t)B * H * NB * 2 * PLAN_WINDOW * sizeof(uint16_t), 256);
}
static int64_t lists_ints_per_batch(int H, int NB, const int32_t* k_per_head) {
    int64_t n = 0;
    for (int h = 0; h < H; ++h) n += ((int64_t)(NB + 1) / 2) * list_stride(k_per_head[h], NB);
    return n;
}

size_t pair_plan_bytes(int B, int H, int NB, const int32_t* k_per_head) {
    return pairs_bytes(B, H, NB) + overlap_bytes(B, H, NB) +
           align_up((size_t)B * lists_ints_per_batch(H, NB, k_per_head) * sizeof(int), 256);
}

// Layout of mem: pairs | overlaps | lists.
int launch_pair_plan(AttnArgs& a, void* mem, cudaStream_t st) {
    const int NP = (a.NB + 1) / 2;
    int2* pairs = static_cast<int2*>(mem);
    uint16_t* ov = reinterpret_cast<uint16_t*>(static_cast<char*>(mem) + pairs_bytes(a.B, a.H, a.NB));
    int* lists = reinterpret_cast<int*>(reinterpret_cast<char*>(ov) + overlap_bytes(a.B, a.H, a.NB));
    a.pairs = pairs;
    a.lists = lists;
    int64_t off = 0;
    for (int h = 0; h < a.H; ++h) {
        a.list_off[h] = off;
        off += (int64_t)NP * list_stride(a.k_per_head[h], a.NB);
    }
    a.list_batch = off;
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
    dim3 lgrid((NP + plan::LIST_WARPS - 1) / plan::LIST_WARPS, a.B * a.H);
    plan::pair_list_kernel<<<lgrid, plan::LIST_WARPS * 32, (size_t)plan::LIST_WARPS * 2 * nwords * sizeof(uint32_t), st>>>(
        a, pairs, lists);
    USV_CHECK_LAUNCH("pair_list_kernel");
    return USV_OK;
}

}  // namespace usv
