// hann_keyswitch_static: the key switch for callers that cannot hand the library a workspace.
//
// Some hosts of this library may neither call cudaMalloc nor set aside an arena: a request handler that must not
// trigger the device-wide synchronisation cudaMalloc/cudaFree imply, or a process whose whole device-memory budget
// was carved up by its own pool at start-up and has nothing left to lend.  For them the scratch of one key switch
// lives in a fixed array inside the library image.  Every GPU that loads the library keeps the array until the
// process exits, so its size is deliberately modest and large rings are refused.
#include <mutex>

#include "internal.h"

// 4 MiB: enough for N = 2^13 with L = 4 (2.6 MiB) or N = 2^14 with L = 2; not for the N = 2^15 / 2^16 sets
#define HANN_STATIC_SCRATCH_BYTES (4u << 20)

static __device__ __align__(256) unsigned char g_static_scratch[HANN_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {};  // device address of g_static_scratch, per device ordinal

}  // namespace

// In host code `g_static_scratch` is only a handle for the runtime, not an address a kernel could use; the device
// address has to be asked for, once per device, while that device is current.  hann_ctx_create does so (a request-time
// call then only reads the cached address); the entry point itself asks again if that has not happened.
int static_scratch_resolve(hann_ctx* c, void** out) {
    if (c->device < 0 || c->device >= kMaxDevices) {
        c->err = "hann_keyswitch_static: device ordinal out of range";
        return HANN_EINVAL;
    }
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[c->device]) {
        int cur = -1;
        if (cudaGetDevice(&cur) != cudaSuccess || cur != c->device) {
            c->err = "hann_keyswitch_static: the context's device is not current";
            return HANN_ECUDA;
        }
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p) {
            c->err = std::string("cudaGetSymbolAddress(g_static_scratch): ") + cudaGetErrorString(e);
            return HANN_ECUDA;
        }
        g_scratch_addr[c->device] = p;
    }
    *out = g_scratch_addr[c->device];
    return HANN_OK;
}

extern "C" int64_t hann_static_scratch_bytes(void) { return (int64_t)HANN_STATIC_SCRATCH_BYTES; }

extern "C" int hann_keyswitch_static(hann_ctx* c, int rot, const void* poly_dev, void* ks0_dev, void* ks1_dev) {
    if (!c) return HANN_EINVAL;
    if (c->kprof) {
        // the per-launch profile creates CUDA events on demand, which is an allocation
        c->err = "hann_keyswitch_static: switch the per-launch profile off first";
        return HANN_EINVAL;
    }
    // what hann_keyswitch carves from its workspace: permuted input, digits, u, lifted
    const int64_t ks_need = keyswitch_ws_bytes(c);
    if (ks_need > (int64_t)HANN_STATIC_SCRATCH_BYTES) {
        c->err = "hann_keyswitch_static: ring too large for the built-in scratch (" + std::to_string(ks_need) + " bytes needed, " +
                 std::to_string(HANN_STATIC_SCRATCH_BYTES) + " available); use hann_keyswitch with a workspace";
        return HANN_ESHAPE;
    }
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess || cudaSetDevice(c->device) != cudaSuccess) {
        c->err = "hann_keyswitch_static: cannot select the context's device";
        return HANN_ECUDA;
    }
    void* scratch = nullptr;
    int rc = static_scratch_resolve(c, &scratch);
    // Nothing in the scratch has to start at zero: each sub-buffer is fully written by one kernel before the next
    // one reads it, so the previous call's contents are simply overwritten.
    if (rc == HANN_OK) rc = hann_keyswitch(c, rot, poly_dev, ks0_dev, ks1_dev, scratch, (size_t)HANN_STATIC_SCRATCH_BYTES);
    cudaSetDevice(prev);
    return rc;
}
