// Pairing plan of the block-sparse attention kernel.
//
// The tcgen05 kernel computes two query blocks per work item over the UNION of their key-block
// lists, so it pays for every key block only one of the two selected.  Which blocks are paired is
// free: this file chooses, per (batch, head), a pairing with large list overlaps, in one kernel
// (pair_plan_kernel: bitmaps, all-pairs overlaps and a greedy matching inside chunks of
// consecutive query blocks, then the union lists).
//
// The result only affects speed: any pairing gives the same attention output.
#include "usv_attn.cuh"

namespace usv {

namespace plan {

constexpr int ROUNDS = 5;      // upper limit; the matching stops as soon as a round finds nothing new
constexpr int CH = 128;        // query blocks per chunk
constexpr int THREADS = 4 * CH;
// bitmap row pitch in 32-bit words: the smallest 4 x odd number that holds the row
__host__ __device__ inline int plan_pitch(int nwords) { const int q = (nwords + 3) / 4; return 4 * (q | 1); }
constexpr int OVP = CH + 8;     // row pitch of the overlap matrix (uint16): rows start 4 banks apart

// One CTA per chunk of CH consecutive query blocks of one (batch, head).
//   1. bitmaps of the chunk's selection rows (shared memory)
//   2. overlap |sel(I) & sel(J)| of every two blocks of the chunk (AND + popcount)
//   3. rounds of "mutual best free partner" (larger overlap first, then the lower block) until a
//      round matches nobody; what is left is paired in index order, an odd block out stays single
//   4. the pairs ordered by their lower block -> pairs[chunk * CH / 2 ...]
//   5. ascending union of the two rows of every pair, each entry flagged with the side(s) that
//      selected it (one warp per pair)
__global__ void __launch_bounds__(THREADS)
pair_plan_kernel(const AttnArgs a, int2* __restrict__ pairs, int* __restrict__ lists) {
    dep_sync();
    // the words behind the sticky status word (fallback count, work counter, ...) start at zero
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x < (WS_HEADER - 4) / 4) a.status[1 + threadIdx.x] = 0u;
    extern __shared__ __align__(16) uint32_t smem_u[];
    __shared__ int16_t partner[CH];
    __shared__ int16_t best[CH];
    __shared__ int16_t order[CH];           // ranks -> blocks (singles, then lower blocks of the pairs)
    __shared__ uint32_t freebits[CH / 32];  // bit set while the block is unmatched
    __shared__ int s_new[2], s_count;       // s_new: one flag per round parity (reset while the other is read)
    const int NB = a.NB;
    const int NP = (NB + 1) >> 1;
    const int nwords = (NB + 31) >> 5;
    const int pitch = plan_pitch(nwords);               // row pitch in words: 4 x odd, so that 16-byte loads of
                                                        // consecutive rows fall into different bank groups
    uint16_t* ov = reinterpret_cast<uint16_t*>(smem_u);            // [CH][OVP], rows 16-byte aligned
    uint32_t* bm = smem_u + CH * OVP / 2;                          // [CH][pitch]
    const int bh = blockIdx.y;
    const int b = bh / a.H, h = bh % a.H;
    const int kh = a.k_per_head[h];
    const int I0 = blockIdx.x * CH;
    const int nI = min(CH, NB - I0);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int2* out_pairs = pairs + (int64_t)bh * NP + blockIdx.x * (CH / 2);
    const int npairs = (nI + 1) >> 1;
    const int lstride = (int)list_stride(kh, NB);
    int* out_lists = lists + b * a.list_batch + a.list_off[h] + (int64_t)blockIdx.x * (CH / 2) * lstride;

    if (kh >= NB) {
        // every list is the full set: pairing is arbitrary and every key block belongs to both sides
        for (int p = threadIdx.x; p < npairs; p += THREADS)
            out_pairs[p] = make_int2(I0 + 2 * p, 2 * p + 1 < nI ? I0 + 2 * p + 1 : -1);
        for (int p = warp; p < npairs; p += THREADS / 32) {
            int* out = out_lists + (int64_t)p * lstride;
            const int flags = 2 * p + 1 < nI ? 3 : 1;
            for (int j = lane; j < NB; j += 32) out[1 + j] = (j << 2) | flags;
            if (lane == 0) out[0] = NB;
        }
        return;
    }

    // 1. bitmaps
    for (int i = threadIdx.x; i < CH * pitch; i += THREADS) bm[i] = 0u;
    __syncthreads();
    const int32_t* sel = a.sel + ((int64_t)bh * NB + I0) * a.kmax;
    const int total = nI * kh;
    for (int i0 = threadIdx.x; i0 < total; i0 += 16 * THREADS) {
        int J[16], R[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) {         // sixteen independent loads in flight
            const int i = i0 + u * THREADS;
            R[u] = i < total ? i / kh : -1;
            J[u] = i < total ? sel[(int64_t)R[u] * a.kmax + (i - R[u] * kh)] : -1;
        }
#pragma unroll
        for (int u = 0; u < 16; ++u)
            if (J[u] >= 0 && J[u] < NB) atomicOr(&bm[R[u] * pitch + (J[u] >> 5)], 1u << (J[u] & 31));
    }
    if (threadIdx.x < CH) partner[threadIdx.x] = -1;
    if (threadIdx.x < CH / 32) {
        const int first = threadIdx.x * 32;
        freebits[threadIdx.x] = first >= nI ? 0u : (nI - first >= 32 ? 0xffffffffu : (1u << (nI - first)) - 1u);
    }
    for (int i = threadIdx.x; i < CH * OVP / 2; i += THREADS) smem_u[i] = 0u;   // overlaps of blocks past the end: 0
    __syncthreads();

    // 2. overlaps of every two blocks of the chunk.  A thread takes four rows i (one row block)
    // against one row j, 128 bits of each at a time: the four i rows are the same for most of a
    // warp (broadcast), consecutive lanes take consecutive j.  The matrix is symmetric, so only
    // j >= (first row of the block) is computed and written to both places.  In a full chunk the
    // row blocks are folded in pairs (block f with block 31 - f: together always CH + 4 values of
    // j), which gives every thread the same number of items.
    {
        const int nq = pitch / 4;
        const int nIb = (nI + 3) / 4;
        const bool folded = nI == CH;
        const int per = CH + 4;
        const int items = folded ? (CH / 8) * per : nIb * nI;
        for (int p = threadIdx.x; p < items; p += THREADS) {
            int ib, j;
            if (folded) {
                const int f = p / per, t = p - f * per;
                const int len = CH - 4 * f;            // values of j of block f
                ib = t < len ? f : CH / 4 - 1 - f;
                j = t < len ? 4 * f + t : 4 * ib + (t - len);
            } else {
                ib = p / nI;
                j = p - ib * nI;
                if (j < 4 * ib) continue;
            }
            const uint4* y = reinterpret_cast<const uint4*>(bm + j * pitch);
            const uint4* x = reinterpret_cast<const uint4*>(bm + ib * 4 * pitch);   // rows past nI are zero
            int cnt[4] = {0, 0, 0, 0};
#pragma unroll 2
            for (int w = 0; w < nq; ++w) {
                const uint4 yv = y[w];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint4 xv = x[q * nq + w];
                    cnt[q] += __popc(xv.x & yv.x) + __popc(xv.y & yv.y) + __popc(xv.z & yv.z) + __popc(xv.w & yv.w);
                }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int i = ib * 4 + q;
                if (i < nI && i != j) {
                    const uint16_t c = (uint16_t)min(cnt[q], 65535);
                    ov[i * OVP + j] = c;
                    if (j >= 4 * ib + 4) ov[j * OVP + i] = c;
                }
            }
        }
    }
    __syncthreads();

    // 3. matching: four threads per block, each scans a quarter of the chunk (four 16-byte loads);
    // key = overlap << 8 | (CH - 1 - j): the largest key is the largest overlap, then the lowest block
    {
        const int i = threadIdx.x >> 2, quarter = threadIdx.x & 3;
        const int j0 = quarter * (CH / 4);
        const uint4* row = reinterpret_cast<const uint4*>(ov + i * OVP + j0);
        for (int r = 0; r < ROUNDS; ++r) {
            if (threadIdx.x == 0) s_new[r & 1] = 0;
            uint32_t bk = 0;
            if (i < nI && ((freebits[i >> 5] >> (i & 31)) & 1u)) {
                uint32_t mask = freebits[j0 >> 5];
                if (i >= j0 && i < j0 + CH / 4) mask &= ~(1u << (i - j0));
#pragma unroll
                for (int u = 0; u < CH / 32; ++u) {
                    const uint4 v = row[u];
                    const uint32_t wv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const int c = u * 8 + e;
                        const uint32_t o = (wv[e >> 1] >> ((e & 1) * 16)) & 0xffffu;
                        const uint32_t key = ((o + 1u) << 8) | (uint32_t)(CH - 1 - (j0 + c));
                        bk = max(bk, ((mask >> c) & 1u) ? key : 0u);
                    }
                }
            }
            bk = max(bk, __shfl_xor_sync(0xffffffffu, bk, 1));
            bk = max(bk, __shfl_xor_sync(0xffffffffu, bk, 2));
            if (quarter == 0) best[i] = bk ? (int16_t)(CH - 1 - (int)(bk & 0xffu)) : (int16_t)-1;
            __syncthreads();
            if (threadIdx.x < nI) {
                const int me = threadIdx.x, j = best[me];
                if (j > me && best[j] == me) {
                    partner[me] = (int16_t)j;
                    partner[j] = (int16_t)me;
                    atomicAnd(&freebits[me >> 5], ~(1u << (me & 31)));
                    atomicAnd(&freebits[j >> 5], ~(1u << (j & 31)));
                    s_new[r & 1] = 1;
                }
            }
            __syncthreads();
            if (!s_new[r & 1]) break;
        }
    }
    // blocks still single are paired in index order; 4. then the pairs are ordered by their lower
    // block (warp 0: two ordered compactions over the chunk)
    if (warp == 0) {
        int run = 0;
#pragma unroll
        for (int c = 0; c < CH / 32; ++c) {
            const int i = c * 32 + lane;
            const bool single = i < nI && partner[i] < 0;
            const unsigned m = __ballot_sync(0xffffffffu, single);
            if (single) order[run + __popc(m & ((1u << lane) - 1u))] = (int16_t)i;
            run += __popc(m);
        }
        __syncwarp();
        for (int q = lane; 2 * q + 1 < run; q += 32) {
            const int x = order[2 * q], y = order[2 * q + 1];
            partner[x] = (int16_t)y;
            partner[y] = (int16_t)x;
        }
        __syncwarp();
        run = 0;
#pragma unroll
        for (int c = 0; c < CH / 32; ++c) {
            const int i = c * 32 + lane;
            const bool low = i < nI && (partner[i] < 0 || partner[i] > i);
            const unsigned m = __ballot_sync(0xffffffffu, low);
            if (low) order[run + __popc(m & ((1u << lane) - 1u))] = (int16_t)i;
            run += __popc(m);
        }
        if (lane == 0) s_count = run;
    }
    __syncthreads();
    for (int p = threadIdx.x; p < s_count; p += THREADS) {
        const int i = order[p];
        out_pairs[p] = make_int2(I0 + i, partner[i] >= 0 ? I0 + partner[i] : -1);
    }
    // 5. union lists
    for (int p = warp; p < s_count; p += THREADS / 32) {
        const int i = order[p], j = partner[i];
        const uint32_t* bitsA = bm + i * pitch;
        const uint32_t* bitsB = bm + (j >= 0 ? j : i) * pitch;
        int* out = out_lists + (int64_t)p * lstride;
        int running = 0;
        for (int w0 = 0; w0 < nwords; w0 += 32) {
            const int w = w0 + lane;
            const uint32_t ba = w < nwords ? bitsA[w] : 0u;
            const uint32_t bb = (w < nwords && j >= 0) ? bitsB[w] : 0u;
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
}

static size_t plan_smem(int NB) {
    const int nwords = (NB + 31) >> 5;
    return (size_t)CH * OVP * sizeof(uint16_t) + (size_t)CH * plan_pitch(nwords) * sizeof(uint32_t);
}

}  // namespace plan

static size_t pairs_bytes(int B, int H, int NB) {
    return align_up((size_t)B * H * ((size_t)(NB + 1) / 2) * sizeof(int2), 256);
}
static int64_t lists_ints_per_batch(int H, int NB, const int32_t* k_per_head) {
    int64_t n = 0;
    for (int h = 0; h < H; ++h) n += ((int64_t)(NB + 1) / 2) * list_stride(k_per_head[h], NB);
    return n;
}

size_t pair_plan_bytes(int B, int H, int NB, const int32_t* k_per_head) {
    return pairs_bytes(B, H, NB) + align_up((size_t)B * lists_ints_per_batch(H, NB, k_per_head) * sizeof(int), 256);
}

// Layout of mem: pairs | lists.
int launch_pair_plan(AttnArgs& a, void* mem, cudaStream_t st) {
    const int NP = (a.NB + 1) / 2;
    int2* pairs = static_cast<int2*>(mem);
    int* lists = reinterpret_cast<int*>(static_cast<char*>(mem) + pairs_bytes(a.B, a.H, a.NB));
    a.pairs = pairs;
    a.lists = lists;
    int64_t off = 0;
    for (int h = 0; h < a.H; ++h) {
        a.list_off[h] = off;
        off += (int64_t)NP * list_stride(a.k_per_head[h], a.NB);
    }
    a.list_batch = off;
    const size_t smem = plan::plan_smem(a.NB);
    cudaError_t e = cudaFuncSetAttribute(plan::pair_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return fail(USV_ERR_CUDA, "sparse_attn: plan smem attribute: %s", cudaGetErrorString(e));
    dim3 grid((a.NB + plan::CH - 1) / plan::CH, a.B * a.H);
    launch_dep(plan::pair_plan_kernel, dim3(grid), dim3(plan::THREADS), smem, st, a, pairs, lists);
    USV_CHECK_LAUNCH("pair_plan_kernel");
    return USV_OK;
}

}  // namespace usv
