// Tensor-core block scores (usv_scores_tc.cu), d = 128.
#pragma once
#include "usv_common.cuh"

namespace usv {

// scratch the tensor-core scores kernel needs besides the pooled means
size_t scores_tc_bytes(int BH, int NBq, int NBk);
// Where the bf16 operand planes [3][BH][NB_pad][128] of q and k live inside mem, and the padded
// row counts (multiples of 128).  The pooling kernel writes them; rows NB .. NB_pad - 1 are zero.
void scores_tc_planes(void* mem, int BH, int NBq, int NBk, __nv_bfloat16** a_pl, __nv_bfloat16** b_pl,
                      int* NBq_pad, int* NBk_pad);
// scores: fp32 [BH][NBq][NBk] from the planes in mem (scores_tc_bytes(...));
// status: device status word the bounded waits report to
int launch_scores_tc(float* scores, int BH, int NBq, int NBk, float scale, void* mem, unsigned int* status,
                     cudaStream_t st);

}  // namespace usv
