// Status strings, per-thread error text and argument checks shared by all entry points.
#include <stdarg.h>
#include <string.h>

#include "usv_common.cuh"

namespace usv {

static thread_local char g_err[512] = "";

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

extern "C" const char* usv_build_info(void) { return "usv-b200 sm_100a " __DATE__; }

extern "C" int usv_workspace_status(const void* ws, void* stream) {
    if (ws == nullptr) return usv::fail(USV_ERR_INVALID_ARG, "workspace_status: null workspace");
    unsigned int word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, ws, sizeof(word), cudaMemcpyDeviceToHost,
                                    static_cast<cudaStream_t>(stream));
    if (e == cudaSuccess) e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess)
        return usv::fail(USV_ERR_CUDA, "workspace_status: %s", cudaGetErrorString(e));
    if (word != 0)
        return usv::fail(USV_ERR_TIMEOUT, "device status word = 0x%x (a bounded wait gave up)", word);
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
