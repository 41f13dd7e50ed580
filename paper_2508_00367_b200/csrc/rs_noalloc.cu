// rs_block_fwd_static: the block for callers that must not allocate.
//
// Its scratch is the file-scope device array below instead of a caller
// workspace.  Host code may not use the array's name as a pointer (on the host
// it is only a stand-in symbol); the device address comes from
// cudaGetSymbolAddress, looked up once per device.
#include <mutex>
#include <stdio.h>
#include <string.h>

#include "rs_internal.h"

namespace {

// Scratch shared by every rs_block_fwd_static call on a device.  Each GPU that
// loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char rs_static_scratch[RS_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch[kMaxDevices];       // device address of rs_static_scratch, per device
bool g_ready[kMaxDevices];

void say(char* err, size_t err_len, const char* msg) {
    if (err && err_len) snprintf(err, err_len, "%s", msg);
}

// First call on a device: resolve the array's device address and opt the selection
// kernel in to its shared-memory size.  Neither call allocates.
rs_status setup_device(int dev, void** scratch, char* err, size_t err_len) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_ready[dev]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, rs_static_scratch);
        if (e != cudaSuccess || !p) {
            say(err, err_len, cudaGetErrorString(e));
            return RS_ERR_CUDA;
        }
        e = rs::select_init();
        if (e != cudaSuccess) {
            say(err, err_len, cudaGetErrorString(e));
            return RS_ERR_CUDA;
        }
        g_scratch[dev] = p;
        g_ready[dev] = true;
    }
    *scratch = g_scratch[dev];
    return RS_OK;
}

}  // namespace

extern "C" {

size_t rs_static_scratch_bytes(void) { return RS_STATIC_SCRATCH_BYTES; }

rs_status rs_block_fwd_static(const rs_block_desc* desc, const rs_block_weights* weights, const void* x,
                              void* x_out, float* scores, int32_t* keep_idx, void* x_full, void* stream,
                              char* err, size_t err_len) {
    if (!desc || !weights) {
        say(err, err_len, "rs_block_fwd_static: null descriptor or weights");
        return RS_ERR_INVALID_ARG;
    }
    const size_t need = rs_block_workspace_bytes(desc);
    if (need == 0) {
        say(err, err_len, "rs_block_fwd_static: bad descriptor");
        return RS_ERR_INVALID_ARG;
    }
    if (need > RS_STATIC_SCRATCH_BYTES) {
        if (err && err_len)
            snprintf(err, err_len,
                     "rs_block_fwd_static: this block needs %zu bytes of scratch but the built-in array holds %zu; "
                     "use rs_block_fwd with a caller workspace",
                     need, (size_t)RS_STATIC_SCRATCH_BYTES);
        return RS_ERR_WORKSPACE;
    }
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        say(err, err_len, e != cudaSuccess ? cudaGetErrorString(e) : "device index out of range");
        return RS_ERR_CUDA;
    }
    void* scratch = nullptr;
    rs_status st = setup_device(dev, &scratch, err, err_len);
    if (st != RS_OK) return st;
    // A context on the stack: it owns no device memory and only collects the error text.
    rs_ctx ctx;
    memset(&ctx, 0, sizeof(ctx));
    ctx.device = dev;
    st = rs_block_fwd(&ctx, desc, weights, x, x_out, scores, keep_idx, x_full, scratch, RS_STATIC_SCRATCH_BYTES,
                      stream);
    if (st != RS_OK) say(err, err_len, ctx.err);
    return st;
}

}  // extern "C"
