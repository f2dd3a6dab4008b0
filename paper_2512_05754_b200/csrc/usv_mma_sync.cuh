// mma.sync (m16n8k16, bf16) building blocks shared by the legacy attention kernel and the
// key-marginal kernel: padded shared-memory tiles filled with cp.async, fragment MMA, ldmatrix.
#pragma once
#include "usv_attn.cuh"

namespace usv {

template <int D>
struct MmaSmem {
    static constexpr int LD = D + 8;  // padded row (elements): conflict-free fragment loads
    static constexpr int TILE = USV_BLOCK * LD;
    static constexpr size_t BYTES = (size_t)TILE * 5 * sizeof(__nv_bfloat16);  // Q + 2K + 2V
};

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem, int src_bytes) {
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(s), "l"(gmem), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;\n" ::); }

__device__ __forceinline__ void mma_bf16_16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t* r, const void* smem_row) {
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem_row);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(s));
}

// Copies rows [row0, row0+64) of one [N, D] matrix (token stride sn) into a padded smem tile;
// rows at or beyond N are zero-filled without touching memory.
template <int D>
__device__ __forceinline__ void load_tile(__nv_bfloat16* dst, const __nv_bfloat16* src, int64_t sn,
                                          int row0, int N) {
    constexpr int LD = MmaSmem<D>::LD;
    constexpr int VPR = D / 8;  // 16-byte vectors per row
    for (int idx = threadIdx.x; idx < USV_BLOCK * VPR; idx += 128) {
        const int r = idx / VPR, c = idx % VPR;
        const int row = row0 + r;
        const int ok = row < N;
        const __nv_bfloat16* g = src + (int64_t)(ok ? row : N - 1) * sn + c * 8;
        cp_async16(dst + r * LD + c * 8, g, ok ? 16 : 0);
    }
}

}  // namespace usv
