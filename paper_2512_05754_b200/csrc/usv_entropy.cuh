// Arguments of the key-marginal kernels (Sec. 3.4, Eq. 16) and the launcher of the tcgen05 one.
#pragma once
#include "usv_common.cuh"

namespace usv {

struct MargArgs {
    const __nv_bfloat16 *q, *k;
    usv_strides sq, sk;
    const int32_t* sel;
    const float* lse;     // [B,H,N] natural log of the softmax denominator (incl. the max)
    float* marg;          // [B,N], zeroed before the launch
    unsigned int* status; // device status word the bounded waits report to (may be NULL)
    int B, H, N, NB, kmax;
    float scale_log2;     // softmax scale * log2(e)
    float inv_hn;         // 1 / (H N)
    int k_per_head[USV_MAX_HEADS];
};

// d = 128 on the tensor cores (usv_entropy_tc.cu); marg must be zero.
int launch_marginal_tc(const MargArgs& a, cudaStream_t st);

}  // namespace usv
