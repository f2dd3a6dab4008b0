// Shared host/device helpers of the USV CUDA library (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "usv.h"

namespace usv {

// Records a formatted reason for the calling thread's last failure and returns `code`.
int fail(int code, const char* fmt, ...);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Every workspace starts with a header of this many bytes.  Word 0 is the device status word:
// kernels with bounded waits OR a code into it and nothing but usv_workspace_status /
// usv_workspace_init ever clears it.  Word 1 counts the query blocks the attention kernel handed
// to its exact fallback (reset by every attention call).
constexpr size_t WS_HEADER = 256;

// Validates a [B,H,N,d] view: pointer and strides 16-byte aligned, non-overlapping rows.
int check_view(const char* name, const void* p, const usv_strides* s, int d);

// Counts a kernel launch of this library (read back by usv_kernel_launches).
void note_launch();

#define USV_CHECK_LAUNCH(what)                                                              \
    do {                                                                                    \
        usv::note_launch();                                                                 \
        cudaError_t e__ = cudaGetLastError();                                               \
        if (e__ != cudaSuccess)                                                             \
            return usv::fail(USV_ERR_CUDA, "%s: %s", (what), cudaGetErrorString(e__));      \
    } while (0)

// ---- launches ----------------------------------------------------------------------------
// The kernels of the library are launched with programmatic stream serialization: the CTAs of
// a kernel may be scheduled while the kernel before it in the stream is still running (that
// kernel says so in its first instruction), and they wait for that kernel's completion, and
// the visibility of its writes, in dep_sync(), the first statement of every kernel.  What is
// saved is the launch latency between dependent kernels, 2-3 us each: a tenth of a merge +
// attention step with its 19 small kernels.  Nothing is read or written before dep_sync().
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dep(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
__device__ __forceinline__ void dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void dep_sync() {
    dep_launch();
    dep_wait();
}

// ---- device helpers -------------------------------------------------------------------

__device__ __forceinline__ void bf16x8_to_float(const uint4& v, float* f) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&t);
}

__device__ __forceinline__ uint4 float8_to_bf16x8(const float* f) {
    uint4 v;
    v.x = pack_bf16x2(f[0], f[1]);
    v.y = pack_bf16x2(f[2], f[3]);
    v.z = pack_bf16x2(f[4], f[5]);
    v.w = pack_bf16x2(f[6], f[7]);
    return v;
}

// Order-preserving map float -> uint32: larger float <=> larger key, equal floats <=> equal keys
// (-0 is folded onto +0 first).
__device__ __forceinline__ uint32_t float_key(float f) {
    uint32_t u = __float_as_uint(f + 0.0f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ int warp_incl_scan(int v) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

}  // namespace usv
