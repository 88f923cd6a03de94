// Context, error reporting and driver entry-point resolution for libcpattn.
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include "internal.h"

namespace cpattn {

static thread_local char g_last_error[512] = "";

int set_error(int code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_last_error, sizeof g_last_error, fmt, ap);
    va_end(ap);
    return code;
}

int check_cuda(cudaError_t e, const char* what) {
    if (e == cudaSuccess) return CP_OK;
    return set_error(CP_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

}  // namespace cpattn

using namespace cpattn;

extern "C" const char* cp_strerror(int code) {
    switch (code) {
        case CP_OK: return "CP_OK";
        case CP_ERR_INVALID_ARG: return "CP_ERR_INVALID_ARG";
        case CP_ERR_UNSUPPORTED: return "CP_ERR_UNSUPPORTED";
        case CP_ERR_WORKSPACE: return "CP_ERR_WORKSPACE";
        case CP_ERR_CUDA: return "CP_ERR_CUDA";
        case CP_ERR_TIMEOUT: return "CP_ERR_TIMEOUT";
        case CP_ERR_BOUNDS: return "CP_ERR_BOUNDS";
        default: return "CP_ERR_UNKNOWN";
    }
}

extern "C" const char* cp_last_error(void) { return g_last_error; }

extern "C" int cp_ctx_create(cp_ctx** out, int device) {
    if (!out) return set_error(CP_ERR_INVALID_ARG, "cp_ctx_create: ctx is NULL");
    *out = nullptr;
    int n = 0;
    if (int rc = check_cuda(cudaGetDeviceCount(&n), "cudaGetDeviceCount")) return rc;
    if (device < 0 || device >= n) return set_error(CP_ERR_INVALID_ARG, "cp_ctx_create: device %d of %d", device, n);
    if (int rc = check_cuda(cudaSetDevice(device), "cudaSetDevice")) return rc;
    cudaDeviceProp prop;
    if (int rc = check_cuda(cudaGetDeviceProperties(&prop, device), "cudaGetDeviceProperties")) return rc;
    if (prop.major != 10)
        return set_error(CP_ERR_UNSUPPORTED, "cp_ctx_create: device is sm_%d%d, this library is sm_100a only",
                         prop.major, prop.minor);
    cp_ctx* c = new cp_ctx();      // value-initialised: every plain member starts as zero
    c->device = device;
    c->num_sms = prop.multiProcessorCount;
    c->stage_bytes = 2u << 20;
    int rc = check_cuda(cudaMalloc(&c->d_status, kStatusBytes), "cudaMalloc(status)");
    if (!rc) rc = check_cuda(cudaMemset(c->d_status, 0, kStatusBytes), "cudaMemset(status)");
    if (!rc) rc = check_cuda(cudaMallocHost(&c->h_status, kStatusWords * sizeof(int32_t)), "cudaMallocHost(status)");
    for (int i = 0; i < kStageBuffers && !rc; ++i) {
        rc = check_cuda(cudaMallocHost(&c->h_stage[i], c->stage_bytes), "cudaMallocHost(stage)");
        if (!rc) rc = check_cuda(cudaEventCreateWithFlags(&c->stage_event[i], cudaEventDisableTiming), "cudaEventCreate");
    }
    if (!rc) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        rc = check_cuda(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q),
                        "cudaGetDriverEntryPoint(cuTensorMapEncodeTiled)");
        if (!rc && (q != cudaDriverEntryPointSuccess || !fn))
            rc = set_error(CP_ERR_CUDA, "cuTensorMapEncodeTiled is not available in this driver");
        c->encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
    }
    if (rc) {
        cp_ctx_destroy(c);
        return rc;
    }
    *out = c;
    return CP_OK;
}

extern "C" int cp_ctx_destroy(cp_ctx* c) {
    if (!c) return CP_OK;
    cudaSetDevice(c->device);
    cudaDeviceSynchronize();
    if (c->d_status) cudaFree(c->d_status);
    if (c->h_status) cudaFreeHost(c->h_status);
    for (int i = 0; i < kStageBuffers; ++i) {
        if (c->h_stage[i]) cudaFreeHost(c->h_stage[i]);
        if (c->stage_event[i]) cudaEventDestroy(c->stage_event[i]);
    }
    delete c;
    return CP_OK;
}

extern "C" int cp_ctx_cache_schedule(cp_ctx* c, int enable) {
    if (!c) return set_error(CP_ERR_INVALID_ARG, "cp_ctx_cache_schedule: ctx is NULL");
    c->cache_on = enable != 0;
    c->cache_valid = false;
    return CP_OK;
}

extern "C" int cp_ctx_poll_status(cp_ctx* c, int32_t* detail) {
    if (!c) return set_error(CP_ERR_INVALID_ARG, "cp_ctx_poll_status: ctx is NULL");
    if (int rc = check_cuda(cudaMemcpy(c->h_status, c->d_status, kStatusWords * sizeof(int32_t),
                                       cudaMemcpyDeviceToHost), "cudaMemcpy(status)")) return rc;
    if (detail) memcpy(detail, c->h_status, kStatusWords * sizeof(int32_t));
    if (c->h_status[0] != 0) {
        int code = c->h_status[0];
        if (code == CP_ERR_BOUNDS)
            set_error(code, "device status: page-table entry %d holds page id %d, outside the pool (block %d); the "
                      "elements behind it were skipped", c->h_status[1], c->h_status[3], c->h_status[2]);
        else
            set_error(code, "device status: code %d, barrier %d, block %d, iteration %d", c->h_status[0],
                      c->h_status[1], c->h_status[2], c->h_status[3]);
        cudaMemset(c->d_status, 0, kStatusWords * sizeof(int32_t));
        return code;
    }
    return CP_OK;
}
