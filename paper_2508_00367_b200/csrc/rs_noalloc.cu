// rs_block_fwd_static: the block for callers that must not allocate.
//
// Its scratch is the file-scope device array below instead of a caller
// workspace.  Host code may not use the array's name as a pointer (on the host
// it is only a stand-in symbol); the device address comes from
// cudaGetSymbolAddress, looked up once per device.
#include <mutex>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "rs_internal.h"

namespace {

// Scratch shared by every rs_block_fwd_static call on a device.  Each GPU that
// loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char rs_static_scratch[RS_STATIC_SCRATCH_BYTES];
// Status word the tensor-core kernels write if one of their bounded waits expires.
static __device__ __align__(256) int rs_static_status[64];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch[kMaxDevices];       // device address of rs_static_scratch, per device
int* g_status[kMaxDevices];         // device address of rs_static_status, per device
bool g_ready[kMaxDevices];
void* g_encode;                     // cuTensorMapEncodeTiled, looked up once (host side, no allocation)
bool g_encode_done;

void say(char* err, size_t err_len, const char* msg) {
    if (err && err_len) snprintf(err, err_len, "%s", msg);
}

// First call on a device: resolve the array's device address and opt the selection
// kernel in to its shared-memory size.  Neither call allocates.
rs_status setup_device(int dev, void** scratch, int** status, void** encode, char* err, size_t err_len) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_encode_done) {
        g_encode = rs::tc_get_encode_fn();
        g_encode_done = true;
    }
    if (!g_ready[dev]) {
        void* p = nullptr;
        void* ps = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, rs_static_scratch);
        if (e == cudaSuccess) e = cudaGetSymbolAddress(&ps, rs_static_status);
        if (e != cudaSuccess || !p || !ps) {
            say(err, err_len, cudaGetErrorString(e));
            return RS_ERR_CUDA;
        }
        g_status[dev] = (int*)ps;
        e = rs::select_init();
        if (e != cudaSuccess) {
            say(err, err_len, cudaGetErrorString(e));
            return RS_ERR_CUDA;
        }
        g_scratch[dev] = p;
        g_ready[dev] = true;
    }
    *scratch = g_scratch[dev];
    *status = g_status[dev];
    *encode = g_encode;
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
    void* encode = nullptr;
    int* status = nullptr;
    rs_status st = setup_device(dev, &scratch, &status, &encode, err, err_len);
    if (st != RS_OK) return st;
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) {
        say(err, err_len, cudaGetErrorString(e));
        return RS_ERR_CUDA;
    }
    // A context on the stack: it owns no device memory and only collects the error text.
    rs_ctx ctx;
    memset(&ctx, 0, sizeof(ctx));
    ctx.device = dev;
    ctx.sm_count = sms;
    ctx.d_status = status;          // same kernels as rs_block_fwd, tensor cores included
    ctx.encode_tiled = encode;
    const char* no_tc = getenv("RS_DISABLE_TC");
    const char* ak = getenv("RS_ATTN_KERNEL");
    ctx.attn_kernel = ak && (ak[0] == '2' || ak[0] == '3') ? ak[0] - '0' : 0;
    ctx.use_tc = (encode != nullptr) && !(no_tc && no_tc[0] == '1');
    st = rs_block_fwd(&ctx, desc, weights, x, x_out, scores, keep_idx, x_full, scratch, RS_STATIC_SCRATCH_BYTES,
                      stream);
    if (st != RS_OK) say(err, err_len, ctx.err);
    return st;
}

rs_status rs_static_async_status(void* stream, char* err, size_t err_len) {
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) {
        say(err, err_len, cudaGetErrorString(e));
        return RS_ERR_CUDA;
    }
    int dev = -1;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        say(err, err_len, e != cudaSuccess ? cudaGetErrorString(e) : "device index out of range");
        return RS_ERR_CUDA;
    }
    int* status = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_ready[dev]) return RS_OK;          // no static call has run on this device yet
        status = g_status[dev];
    }
    int word = 0;
    e = cudaMemcpy(&word, status, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) {
        say(err, err_len, cudaGetErrorString(e));
        return RS_ERR_CUDA;
    }
    if (word == RS_DEV_OK) return RS_OK;
    cudaMemset(status, 0, sizeof(int));
    if (word == RS_DEV_SMEM_ALIGN) {
        say(err, err_len, "rs_block_fwd_static: a kernel's shared memory window was not 1024-byte aligned");
        return RS_ERR_CUDA;
    }
    say(err, err_len, "rs_block_fwd_static: a bounded device-side wait expired");
    return RS_ERR_TIMEOUT;
}

}  // extern "C"
