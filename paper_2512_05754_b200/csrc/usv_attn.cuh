// Argument block shared by the block-sparse attention kernels.
#pragma once
#include "usv_common.cuh"

namespace usv {

struct AttnArgs {
    const __nv_bfloat16 *q, *k, *v;
    __nv_bfloat16* o;
    usv_strides sq, sk, sv, so;
    const int32_t* sel;  // [B,H,NB,kmax]
    float* o_f32;        // optional [B,H,N,D]
    float* lse;          // optional [B,H,N]
    unsigned int* status;  // optional device status word (bounded waits report here)
    // Query blocks whose fixed-reference softmax left the safe range: the tcgen05 kernel appends
    // their work ids here; the exact kernel, launched in list mode, recomputes them.
    int* fallback_list;
    int* fallback_count;
    int* work_counter;      // zeroed before the launch: the persistent CTAs of the tcgen05 kernel draw their items from it
    const int2* pairs;      // [B,H,ceil(NB/2)] query-block pairs of the tcgen05 kernel (head-major, not head-ordered)
    // Union key-block lists of the pairs: for (b, h, pair) at lists + b * list_batch + list_off[h] +
    // pair * list_stride(h): [0] = number of entries, then (key block << 2) | in-A | in-B << 1, ascending.
    const int* lists;
    int64_t list_batch;
    int64_t list_off[USV_MAX_HEADS];
    // Fused unmerge (NULL / 0 when off): the tcgen05 kernel stores every output row to all the
    // original tokens that read it back, y[b, n, h*d ...] for n in unmerge_idx[b, off[row] .. off[row+1]),
    // instead of to o.  y: bf16 [B, N_full, H*d] contiguous.
    const int32_t* unmerge_off;   // [B, N+1]
    const int32_t* unmerge_idx;   // [B, N_full]
    __nv_bfloat16* y;
    int N_full;
    const int* work_list;   // list mode of the exact kernel (NULL = one CTA per query block)
    const int* work_count;
    int B, H, N, NB, kmax;
    float scale_log2;    // softmax scale * log2(e)
    int k_per_head[USV_MAX_HEADS];
    int head_order[USV_MAX_HEADS];  // heads sorted by descending k: heavy work is issued first
};

int launch_attn_mma(const AttnArgs& a, int d, cudaStream_t st);
bool attn_pair_supported(const AttnArgs& a, int d);
int launch_attn_pair(const AttnArgs& a, int d, cudaStream_t st);
// fused unmerge: copies the query blocks the exact kernel recomputed (into o) to their original tokens in y
int launch_scatter_fallbacks(const AttnArgs& a, int d, cudaStream_t st);
// ints one pair's list occupies for a head that keeps k of NB key blocks (header + entries)
__host__ __device__ inline int64_t list_stride(int k, int NB) { return 1 + (int64_t)(2 * (int64_t)k < NB ? 2 * k : NB); }
size_t pair_plan_bytes(int B, int H, int NB, const int32_t* k_per_head);
// Fills a.pairs / a.lists / a.list_* (pointing into mem) and enqueues the plan kernels.
int launch_pair_plan(AttnArgs& a, void* mem, cudaStream_t st);

}  // namespace usv
