// Shared declarations of the token-merge kernels: bipartite partition and the tensor-core matcher.
#pragma once
#include "usv_common.cuh"

namespace usv {

struct Part {
    int T, Hh, W, st, sh, sw;
    int nHy, nWx, nB;  // destinations per axis (y, x) and in total
    __host__ __device__ bool is_dst(int n) const {
        const int x = n % W, y = (n / W) % Hh, t = n / (W * Hh);
        return (t % st == 0) && (y % sh == 0) && (x % sw == 0);
    }
    // ordinal (ascending token order) of a destination token
    __host__ __device__ int ord(int n) const {
        const int x = n % W, y = (n / W) % Hh, t = n / (W * Hh);
        return ((t / st) * nHy + y / sh) * nWx + x / sw;
    }
    __host__ __device__ int dst_token(int o) const {
        const int dx = o % nWx, dy = (o / nWx) % nHy, dt = o / (nWx * nHy);
        return ((dt * st) * Hh + dy * sh) * W + dx * sw;
    }
};

struct MatchTcArgs {
    Part p;
    int B, N, nA, nA_pad, nB_pad;
    const int32_t* src_idx;          // [nA] source tokens, ascending
    uint16_t* a_h;                   // fp16 bits [B][nA_pad][128]
    uint16_t* b_h;                   // fp16 bits [B][nB_pad][128]
    float* cand_v;                   // [B][nA][2][4] largest approximate cosines per source and tile parity, descending
    int* cand_i;                     // [B][nA][2][4] their destination ordinals
    int* exact_list;                 // sources (b * nA + rank) that need the fp32 scan of all destinations
    int* exact_count;
    int zero_words;              // 32-bit words from exact_count on that half_kernel sets to zero
    unsigned long long* exact_best;  // one slot per list entry: (key of the best cosine << 32) | ~destination
    float* floor_v;                  // [B][nA_pad] lower bound on each source's approximate row maximum
    int32_t* jstar_s;                // [B][nA] best destination TOKEN per source rank
    float* u_s;                      // [B][nA] its cosine
    unsigned int* status;            // device status word for bounded waits (may be NULL)
};

// bytes of the matcher's scratch for a sequence of N tokens (any partition: sources + destinations = N)
size_t match_tc_bytes(int B, int N);
// mhat: fp32 unit descriptors [B,N,128]; mem: match_tc_bytes(B, N) bytes, 256-byte aligned.
int launch_match_tc(const float* mhat, const Part& p, int B, int N, int nA, const int32_t* src_idx,
                    int32_t* jstar_s, float* u_s, void* mem, unsigned int* status, cudaStream_t st);

}  // namespace usv
