// Top-k key-block selection.
//
// Rows of up to 2048 scores: one WARP per row, select_warp_kernel (with more of a row per lane
// the register file holds too few warps: measured slower than the CTA kernel below).  The
// row sits in registers as order-preserving keys, striped over the lanes; the key T of the k-th
// largest element is found bit by bit (at most 32 warp-wide counts, fewer when a candidate cuts
// the row at exactly k), then every element above T and the first (k - above) elements equal to
// T are emitted in ascending index (two ballots per 32 elements give the positions).
//
// Longer rows: one CTA per row, select_kernel.
//
// The row is mapped to order-preserving 32-bit keys in shared memory.  Four 8-bit radix passes
// (most significant digit first) find the key T of the k-th largest element and the number of
// elements strictly above it.  The output pass gives every thread a contiguous stretch of the
// row: it counts what it keeps (every key above T, and the first (k - above) keys equal to T,
// which is exactly "k largest, ties to the lowest index"), one block-wide scan places it, and it
// writes its indices in ascending order.  Rows that keep everything skip the search.
#include "usv_common.cuh"

namespace usv {

constexpr int SEL_THREADS = 256;
constexpr int SEL_MAX_NB = 8192;

struct SelHeads {
    int k[USV_MAX_HEADS];
};

// Block-wide exclusive scan of one int per thread (SEL_THREADS threads); returns the exclusive
// prefix and writes the block total to *total.  `scratch` holds >= 9 ints.
__device__ __forceinline__ int block_excl_scan(int v, int* scratch, int* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int incl = warp_incl_scan(v);
    if (lane == 31) scratch[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = lane < SEL_THREADS / 32 ? scratch[lane] : 0;
        int wi = warp_incl_scan(w);
        if (lane < SEL_THREADS / 32) scratch[lane] = wi - w;
        if (lane == SEL_THREADS / 32 - 1) scratch[8] = wi;
    }
    __syncthreads();
    const int res = scratch[warp] + incl - v;
    *total = scratch[8];
    __syncthreads();
    return res;
}

__global__ void __launch_bounds__(SEL_THREADS) select_kernel(const float* __restrict__ scores,
                                                             int32_t* __restrict__ sel, int H,
                                                             int NBq, int NBk, int kmax,
                                                             const SelHeads heads) {
    dep_sync();
    extern __shared__ uint32_t keys[];   // NBk order-preserving keys
    __shared__ int hist[256];
    __shared__ int scratch[9];
    __shared__ uint32_t s_prefix;
    __shared__ int s_remaining, s_eq_total;

    const int row = blockIdx.x;  // (b*H + h)*NBq + I
    const int h = (row / NBq) % H;
    const int k = heads.k[h];
    const float* src = scores + (int64_t)row * NBk;
    int32_t* out = sel + (int64_t)row * kmax;

    if (k >= NBk) {   // keep everything: no search
        for (int j = threadIdx.x; j < NBk; j += SEL_THREADS) out[j] = j;
        for (int t = NBk + threadIdx.x; t < kmax; t += SEL_THREADS) out[t] = -1;
        return;
    }
    for (int j = threadIdx.x; j < NBk; j += SEL_THREADS) keys[j] = float_key(src[j]);
    if (threadIdx.x == 0) {
        s_prefix = 0;
        s_remaining = k;
    }
    __syncthreads();

    // Radix select: after the pass for digit `shift`, s_prefix holds the top bits of T and
    // s_remaining the rank of T among the elements that share those bits.
    for (int shift = 24; shift >= 0; shift -= 8) {
        hist[threadIdx.x] = 0;
        __syncthreads();
        const uint32_t prefix = s_prefix;
        const uint32_t mask = shift == 24 ? 0u : (0xffffffffu << (shift + 8));
        for (int j = threadIdx.x; j < NBk; j += SEL_THREADS) {
            const uint32_t key = keys[j];
            if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255], 1);
        }
        __syncthreads();
        if (threadIdx.x < 32) {
            // 256 bins, scanned from the top; each lane owns 8 consecutive bins.
            const int lane = threadIdx.x;
            const int remaining = s_remaining;  // read by every lane before the scan's shuffles
            int local[8], sum = 0;
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                local[t] = hist[255 - (lane * 8 + t)];
                sum += local[t];
            }
            const int incl = warp_incl_scan(sum);
            int before = incl - sum;  // elements in bins above this lane's bins
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                if (before < remaining && remaining <= before + local[t]) {
                    s_prefix = prefix | ((uint32_t)(255 - (lane * 8 + t)) << shift);
                    s_remaining = remaining - before;
                    s_eq_total = local[t];   // after the last pass: how many keys equal T
                }
                before += local[t];
            }
        }
        __syncthreads();
    }
    const uint32_t T = s_prefix;
    const int need_eq = s_remaining;  // how many elements equal to T are kept (lowest indices)
    const bool all_eq = need_eq == s_eq_total;   // no tie straddles the cut (the usual case)

    // Ordered output.  Thread t owns the contiguous indices [t L, t L + L): it counts what it keeps,
    // one block-wide scan gives its first output slot, and it writes its indices in order.
    const int L = (NBk + SEL_THREADS - 1) / SEL_THREADS;
    const int j0 = threadIdx.x * L, j1 = min(j0 + L, NBk);
    int eq_base = 0;
    if (!all_eq) {   // ties across the cut: the lowest indices among the equal keys win
        int ne = 0;
        for (int j = j0; j < j1; ++j) ne += keys[j] == T ? 1 : 0;
        int tot;
        eq_base = block_excl_scan(ne, scratch, &tot);
    }
    int cnt = 0;
    {
        int eq_seen = eq_base;
        for (int j = j0; j < j1; ++j) {
            const uint32_t key = keys[j];
            if (key > T) ++cnt;
            else if (key == T) { if (all_eq || eq_seen < need_eq) ++cnt; ++eq_seen; }
        }
    }
    int tot_out;
    int p = block_excl_scan(cnt, scratch, &tot_out);
    {
        int eq_seen = eq_base;
        for (int j = j0; j < j1; ++j) {
            const uint32_t key = keys[j];
            bool take = key > T;
            if (key == T) { take = all_eq || eq_seen < need_eq; ++eq_seen; }
            if (take) out[p++] = j;
        }
    }
    for (int t = k + threadIdx.x; t < kmax; t += SEL_THREADS) out[t] = -1;
}

// One warp per row; lane l holds the scores of indices i * 32 + l, i < KPL (every load of the
// row is one contiguous 128-byte line per warp).
template <int KPL>
__global__ void __launch_bounds__(256, 2) select_warp_kernel(const float* __restrict__ scores,
                                                          int32_t* __restrict__ sel, int H, int NBq,
                                                          int NBk, int kmax, const SelHeads heads,
                                                          int64_t rows) {
    dep_sync();
    const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int lane = threadIdx.x & 31;
    const uint32_t lt = (1u << lane) - 1u;
    const int h = (int)((row / NBq) % H);
    const int k = heads.k[h];
    const float* src = scores + row * NBk;
    int32_t* out = sel + row * kmax;
    if (k >= NBk) {   // keep everything: no search (uniform over the warp)
        for (int j = lane; j < NBk; j += 32) out[j] = j;
        for (int t = NBk + lane; t < kmax; t += 32) out[t] = -1;
        return;
    }
    uint32_t key[KPL];
#pragma unroll
    for (int i = 0; i < KPL; ++i) key[i] = (i * 32 + lane < NBk) ? float_key(__ldg(src + i * 32 + lane)) : 0u;   // 0 < any real key
    // Largest T with count(key >= T) >= k, one bit at a time.  As soon as a candidate leaves
    // exactly k keys at or above it, those k are the answer and no tie can straddle the cut.
    // The bits above the highest one in which two real keys differ are common to all of them and
    // to T: the search starts below them.
    uint32_t kor = 0u, kand = 0xffffffffu;
#pragma unroll
    for (int i = 0; i < KPL; ++i)
        if (i * 32 + lane < NBk) { kor |= key[i]; kand &= key[i]; }
    kor = __reduce_or_sync(0xffffffffu, kor);
    kand = __reduce_and_sync(0xffffffffu, kand);
    const uint32_t diff = kor ^ kand;
    const int top = diff ? 31 - __clz(diff) : -1;               // highest differing bit (-1: all keys equal)
    uint32_t T = top >= 31 ? 0u : (kand & ~((2u << (top < 0 ? 0 : top)) - 1u));
    if (top < 0) T = kand;
    bool exact = false;
#pragma unroll 1
    for (int bit = top; bit >= 0; --bit) {
        const uint32_t cand = T | (1u << bit);
        int c = 0;
#pragma unroll
        for (int i = 0; i < KPL; ++i) c += key[i] >= cand ? 1 : 0;
        const int tot = __reduce_add_sync(0xffffffffu, c);
        if (tot >= k) T = cand;
        if (tot == k) { exact = true; break; }
    }
    // keys above the cut are kept; of the keys equal to T (the k-th largest key, when the search
    // ran to the last bit) the lowest indices fill what is left
    const uint32_t cut = exact ? T - 1u : T;   // kept outright: key > cut
    int need_eq = 0;
    if (!exact) {
        int ngt = 0;
#pragma unroll
        for (int i = 0; i < KPL; ++i) ngt += key[i] > T ? 1 : 0;
        need_eq = k - __reduce_add_sync(0xffffffffu, ngt);
    }
    int base = 0, eq_seen = 0;
#pragma unroll
    for (int i = 0; i < KPL; ++i) {
        if (i * 32 < NBk) {   // uniform over the warp
            const bool gt = key[i] > cut;
            const bool eq = !exact && key[i] == T && i * 32 + lane < NBk;
            const uint32_t eqb = __ballot_sync(0xffffffffu, eq);
            const bool take = gt || (eq && eq_seen + __popc(eqb & lt) < need_eq);
            const uint32_t tkb = __ballot_sync(0xffffffffu, take);
            if (take) out[base + __popc(tkb & lt)] = i * 32 + lane;
            base += __popc(tkb);
            eq_seen += __popc(eqb);
        }
    }
    for (int t = k + lane; t < kmax; t += 32) out[t] = -1;
}

}  // namespace usv

extern "C" int usv_select_blocks(int B, int H, int NBq, int NBk, const float* scores,
                                 const int32_t* k_per_head, int kmax, int32_t* sel, void* stream) {
    using namespace usv;
    if (B <= 0 || H <= 0 || NBq <= 0 || NBk <= 0)
        return fail(USV_ERR_INVALID_ARG, "select_blocks: B,H,NBq,NBk must be positive");
    if (H > USV_MAX_HEADS) return fail(USV_ERR_UNSUPPORTED, "select_blocks: H > %d", USV_MAX_HEADS);
    if (NBk > SEL_MAX_NB) return fail(USV_ERR_UNSUPPORTED, "select_blocks: NBk > %d", SEL_MAX_NB);
    if (scores == nullptr || sel == nullptr || k_per_head == nullptr)
        return fail(USV_ERR_INVALID_ARG, "select_blocks: null pointer");
    SelHeads heads;
    int kmx = 0;
    for (int h = 0; h < H; ++h) {
        if (k_per_head[h] < 1 || k_per_head[h] > NBk)
            return fail(USV_ERR_INVALID_ARG, "select_blocks: k_per_head[%d]=%d outside [1,%d]", h,
                        k_per_head[h], NBk);
        heads.k[h] = k_per_head[h];
        kmx = k_per_head[h] > kmx ? k_per_head[h] : kmx;
    }
    if (kmax < kmx) return fail(USV_ERR_INVALID_ARG, "select_blocks: kmax=%d < max k=%d", kmax, kmx);
    const int64_t rows = (int64_t)B * H * NBq;
    if (rows > 2147483647LL) return fail(USV_ERR_UNSUPPORTED, "select_blocks: too many rows");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const unsigned wg = (unsigned)((rows + 7) / 8);
#define USV_SEL_WARP(KPL) launch_dep(select_warp_kernel<KPL>, dim3(wg), dim3(256), 0, st, scores, sel, H, NBq, NBk, kmax, heads, rows)
    if (NBk <= 256) USV_SEL_WARP(8);
    else if (NBk <= 512) USV_SEL_WARP(16);
    else if (NBk <= 1024) USV_SEL_WARP(32);
    else if (NBk <= 1536) USV_SEL_WARP(48);
    else if (NBk <= 2048) USV_SEL_WARP(64);
    else launch_dep(select_kernel, dim3((unsigned)rows), dim3(SEL_THREADS), (size_t)NBk * sizeof(uint32_t), st, scores, sel, H, NBq, NBk, kmax, heads);
#undef USV_SEL_WARP
    USV_CHECK_LAUNCH("select_kernel");
    return USV_OK;
}
