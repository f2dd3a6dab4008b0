// Status strings, per-thread error text and argument checks shared by all entry points.
#include <stdarg.h>
#include <string.h>

#include "usv_common.cuh"
#include "usv_tcgen05.cuh"

namespace usv {

static thread_local char g_err[512] = "";
static unsigned long long g_launches = 0;

void note_launch() { __atomic_fetch_add(&g_launches, 1ull, __ATOMIC_RELAXED); }

int fail(int code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

int check_view(const char* name, const void* p, const usv_strides* s, int d) {
    if (p == nullptr || s == nullptr) return fail(USV_ERR_INVALID_ARG, "%s: null pointer", name);
    if (!aligned16(p)) return fail(USV_ERR_UNSUPPORTED, "%s: pointer not 16-byte aligned", name);
    if (s->sn < d || s->sb < 0 || s->sh < 0)
        return fail(USV_ERR_INVALID_ARG, "%s: token stride %lld smaller than d=%d", name,
                    (long long)s->sn, d);
    if ((s->sb % 8) || (s->sh % 8) || (s->sn % 8))
        return fail(USV_ERR_UNSUPPORTED, "%s: strides must be multiples of 8 elements", name);
    return USV_OK;
}

}  // namespace usv

extern "C" const char* usv_status_string(int status) {
    switch (status) {
        case USV_OK: return "ok";
        case USV_ERR_INVALID_ARG: return "invalid argument";
        case USV_ERR_UNSUPPORTED: return "unsupported configuration";
        case USV_ERR_WORKSPACE: return "workspace too small";
        case USV_ERR_CUDA: return "CUDA error";
        case USV_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}

extern "C" const char* usv_last_error(void) { return usv::g_err; }

extern "C" unsigned long long usv_kernel_launches(void) {
    return __atomic_load_n(&usv::g_launches, __ATOMIC_RELAXED);
}

extern "C" const char* usv_build_info(void) { return "usv-b200 sm_100a " __DATE__; }

extern "C" int usv_workspace_init(void* ws, void* stream) {
    if (ws == nullptr) return usv::fail(USV_ERR_INVALID_ARG, "workspace_init: null workspace");
    cudaError_t e = cudaMemsetAsync(ws, 0, usv::WS_HEADER, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return usv::fail(USV_ERR_CUDA, "workspace_init: %s", cudaGetErrorString(e));
    return USV_OK;
}

extern "C" int usv_workspace_status(void* ws, void* stream) {
    if (ws == nullptr) return usv::fail(USV_ERR_INVALID_ARG, "workspace_status: null workspace");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned int word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, ws, sizeof(word), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e == cudaSuccess && word != 0) {
        e = cudaMemsetAsync(ws, 0, sizeof(word), st);   // reported once: the word starts afresh
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    }
    if (e != cudaSuccess)
        return usv::fail(USV_ERR_CUDA, "workspace_status: %s", cudaGetErrorString(e));
    if (word != 0)
        return usv::fail(USV_ERR_TIMEOUT, "device status word = 0x%x (a bounded wait gave up)", word);
    return USV_OK;
}

namespace usv {
// One warp waits, with the library's own bounded wait, on a barrier that nothing ever arrives at.
__global__ void wait_selftest_kernel(unsigned int* status, unsigned long long limit_ns) {
    dep_sync();
    __shared__ __align__(8) unsigned long long bar_mem;
    __shared__ int abort_flag;
    const uint32_t bar = t5::smem_u32(&bar_mem);
    if (threadIdx.x == 0) {
        abort_flag = 0;
        t5::mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    t5::mbar_wait(bar, 0, &abort_flag, status, 0x80000000u, limit_ns);
}
}  // namespace usv

extern "C" int usv_selftest_wait_timeout(void* ws, unsigned int limit_us, void* stream) {
    if (ws == nullptr) return usv::fail(USV_ERR_INVALID_ARG, "selftest_wait_timeout: null workspace");
    if (limit_us == 0 || limit_us > 100000u)
        return usv::fail(USV_ERR_INVALID_ARG, "selftest_wait_timeout: limit %u us outside [1, 100000]", limit_us);
    usv::wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<unsigned int*>(ws),
                                                                             1000ull * limit_us);
    USV_CHECK_LAUNCH("wait_selftest_kernel");
    return USV_OK;
}

extern "C" int usv_sparse_attn_fallbacks(const void* ws, void* stream, int* count) {
    if (ws == nullptr || count == nullptr) return usv::fail(USV_ERR_INVALID_ARG, "sparse_attn_fallbacks: null pointer");
    cudaError_t e = cudaMemcpyAsync(count, static_cast<const char*>(ws) + 4, sizeof(int), cudaMemcpyDeviceToHost,
                                    static_cast<cudaStream_t>(stream));
    if (e == cudaSuccess) e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return usv::fail(USV_ERR_CUDA, "sparse_attn_fallbacks: %s", cudaGetErrorString(e));
    return USV_OK;
}
