// sepconv_fwd_static: the forward block call for callers that cannot hand over a workspace.
//
// The scratch that sepconv_fwd takes from its caller lives here in a fixed device array that is
// part of the library image, so this call performs no allocation of any kind.
#include <cuda_runtime.h>
#include <cstdio>

#include "../../include/sepconv.h"
#include "kernels.h"

// One array per GPU that loads the library, held until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[SEPCONV_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
// Device address of g_static_scratch on each device.  In host code the symbol g_static_scratch is
// only a handle for the runtime, never a device address, so the address is looked up once per device.
void* g_scratch_addr[kMaxDevices] = {nullptr};
}  // namespace

extern "C" int sepconv_fwd_static(sc_ctx* ctx, const sc_block_desc* desc, const sc_tensor* x,
                                  const sc_tensor* x_res, const int32_t* lengths_dev,
                                  const sc_block_params* params, sc_tensor* y, int32_t* out_lengths_dev,
                                  sc_block_saved* saved, void* cuda_stream) {
    if (!ctx || !desc) return SC_ERR_NULL;
    size_t need = 0;
    int rc = sepconv_workspace_bytes(desc, &need, nullptr);
    if (rc != SC_OK) return rc;
    if (need > (size_t)SEPCONV_STATIC_SCRATCH_BYTES) {
        fprintf(stderr, "sepconv_fwd_static: this block needs %zu bytes of scratch, the built-in buffer holds %zu; "
                        "use sepconv_fwd with a caller-owned workspace\n",
                need, (size_t)SEPCONV_STATIC_SCRATCH_BYTES);
        return SC_ERR_WORKSPACE;
    }
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SC_ERR_CUDA;
    // the array and its address belong to the current device: it must be the one the context lives on
    if (dev != sc::ctx_device(ctx)) {
        fprintf(stderr, "sepconv_fwd_static: the current device (%d) is not the context's device (%d)\n", dev,
                sc::ctx_device(ctx));
        return SC_ERR_UNSUPPORTED;
    }
    if (!g_scratch_addr[dev]) {     // first call on this device: resolve the array's device address (with lazy
                                    // module loading this is also where the device sets the array aside)
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p) {
            fprintf(stderr, "sepconv_fwd_static: cudaGetSymbolAddress failed: %s\n", cudaGetErrorString(e));
            return SC_ERR_CUDA;
        }
        g_scratch_addr[dev] = p;
    }
    void* ws = g_scratch_addr[dev];
    // The array keeps whatever the previous call left.  Every scratch word the forward kernels read
    // they write first in the same call (lengths, frame count, statistics partials, masked copies), so
    // nothing has to start at zero and nothing is enqueued before sepconv_fwd has validated its arguments.
    return sepconv_fwd(ctx, desc, x, x_res, lengths_dev, params, y, out_lengths_dev, saved, nullptr, nullptr,
                       ws, (size_t)SEPCONV_STATIC_SCRATCH_BYTES, cuda_stream);
}
