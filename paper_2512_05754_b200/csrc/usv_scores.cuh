// Tensor-core block scores (usv_scores_tc.cu), d = 128.
#pragma once
#include "usv_common.cuh"

namespace usv {

// scratch the tensor-core scores kernel needs besides the pooled means
size_t scores_tc_bytes(int BH, int NBq, int NBk);
// qbar/kbar: fp32 pooled means [BH][NB][128]; scores: fp32 [BH][NBq][NBk]; mem: scores_tc_bytes(...);
// status: device status word the bounded waits report to
int launch_scores_tc(const float* qbar, const float* kbar, float* scores, int BH, int NBq, int NBk, float scale,
                     void* mem, unsigned int* status, cudaStream_t st);

}  // namespace usv
