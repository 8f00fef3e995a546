// cerar_allreduce_sim_static: the whole pipeline without a caller-supplied
// workspace.  The (c+N) x p slots of all N workers live in a fixed array that is
// part of this library's device image, so the call needs no allocation at all.
#include <cuda_runtime.h>

#include <cstdio>
#include <mutex>
#include <string>

#include "../../include/cerar.h"

// Capacity of the built-in workspace.  Every GPU on which this library's device
// code gets loaded reserves this much memory until the process exits.
#define CERAR_STATIC_WS_FLOATS (16u * 1024u * 1024u)          /* 64 MiB */

// Device-side storage.  In host code this name is only a handle for the runtime,
// never an address a kernel could use: the real device address is looked up
// below with cudaGetSymbolAddress, once per device.
static __device__ __align__(256) float g_cerar_static_ws[CERAR_STATIC_WS_FLOATS];

extern "C" void cerar_internal_set_error(const char* msg);    // api.cu: text behind cerar_last_error()
extern "C" int cerar_internal_plan_device(const cerar_plan_t* plan);   // api.cu: -1 without device copies

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_mutex;
float* g_device_ptr[kMaxDevices] = {nullptr};                 // looked-up address, per device ordinal
}  // namespace

extern "C" cerar_status_t cerar_allreduce_sim_static(cerar_plan_t* plan, const float* grads, int64_t grads_stride,
                                                     float* out, int64_t out_stride, int64_t d, float scale,
                                                     cerar_stream_t stream) {
    if (!plan) {
        cerar_internal_set_error("plan is NULL");
        return CERAR_ERR_INVALID_ARG;
    }
    const size_t need = cerar_workspace_bytes(plan, d);        // 0 for a bad d: reported by the call below
    const size_t have = (size_t)CERAR_STATIC_WS_FLOATS * sizeof(float);
    if (need > have) {
        char msg[200];
        std::snprintf(msg, sizeof msg,
                      "cerar_allreduce_sim_static: this N, c, d needs %zu bytes of workspace, the built-in "
                      "workspace holds %zu; use cerar_allreduce_sim with your own buffer", need, have);
        cerar_internal_set_error(msg);
        return CERAR_ERR_TOO_LARGE;
    }
    // The plan must have device copies and its device must be the current one BEFORE the array is looked
    // up: the lookup below is what makes the CUDA runtime load this file's device image (and with it
    // reserve the array) on the current device, and that must not happen on a device the call cannot use.
    const int plan_dev = cerar_internal_plan_device(plan);
    if (plan_dev < 0) {
        cerar_internal_set_error("plan has no device copies (no CUDA device, or host_only)");
        return CERAR_ERR_CUDA;
    }
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cerar_internal_set_error(e != cudaSuccess ? cudaGetErrorString(e) : "device ordinal out of range");
        return CERAR_ERR_CUDA;
    }
    if (dev != plan_dev) {
        cerar_internal_set_error("the device the plan was created on must be current");
        return CERAR_ERR_CUDA;
    }
    float* ws = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (!g_device_ptr[dev]) {
            // one-time set-up for this device (it is the current one).  With lazy module loading this
            // is also the moment the 64 MiB are reserved on the device: it can fail for lack of memory
            void* p = nullptr;
            e = cudaGetSymbolAddress(&p, g_cerar_static_ws);
            if (e != cudaSuccess || !p) {
                cerar_internal_set_error(e != cudaSuccess
                                             ? (std::string("built-in workspace could not be set up on this device: ") +
                                                cudaGetErrorString(e)).c_str()
                                             : "symbol address is NULL");
                cudaGetLastError();
                return e == cudaErrorMemoryAllocation ? CERAR_ERR_NOMEM : CERAR_ERR_CUDA;
            }
            g_device_ptr[dev] = static_cast<float*>(p);
        }
        ws = g_device_ptr[dev];
    }
    // Nothing in the workspace has to start at zero: encode writes every D row and
    // each round writes its landing slot before any later step reads it.
    return cerar_allreduce_sim(plan, grads, grads_stride, out, out_stride, ws, d, scale, stream);
}
