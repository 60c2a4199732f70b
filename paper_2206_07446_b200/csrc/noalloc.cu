// nnv_conv_exec_static: the execution of one layer for callers that have no device memory to
// offer as scratch.
//
// nnv_conv_exec needs the caller to pass a scratch buffer for the GEMM-based variants (the im2col
// matrix, or the Winograd V and M arrays).  Some users of this library cannot produce one: a
// plug-in that lives inside a host application which owns all device memory and hands out no
// allocator; a control loop with a hard latency bound, where cudaMalloc's implicit device-wide
// synchronisation is not acceptable; start-up code that runs before the process's memory pool
// exists.  For them the scratch lives in the fixed array below, which is part of the library
// image: every GPU that loads libnnv.so holds NNV_STATIC_SCRATCH_BYTES for it until the process
// exits, whether or not this entry point is ever called.
//
// In host code the array's name is only a handle for the runtime, not a device address, so it is
// never handed to a kernel.  The device address is looked up once per device with
// cudaGetSymbolAddress while that device is current, and that pointer is what the kernels get.
#include <mutex>

#include "nnv_internal.h"

namespace nnv {
nnv_status_t do_exec(const nnv_plan& p, int layer, int v, int math, const void* d_in, const void* d_add,
                     const void* d_wt, const void* d_bias, void* d_out, void* d_ws, uint64_t ws_bytes, cudaStream_t st);
}

namespace {

static __device__ __align__(256) unsigned char g_static_scratch[NNV_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

// Device address of the scratch array on the device that is current in the calling thread.
nnv_status_t static_scratch(void** out) {
    int dev = -1;
    NNV_CUDA(cudaGetDevice(&dev));
    NNV_REQUIRE(dev >= 0 && dev < kMaxDevices, NNV_ERR_UNSUPPORTED, "device ordinal %d is beyond the %d this table holds", dev, kMaxDevices);
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        void* ptr = nullptr;
        NNV_CUDA(cudaGetSymbolAddress(&ptr, g_static_scratch));
        NNV_REQUIRE(ptr != nullptr && nnv::aligned256(ptr), NNV_ERR_CUDA, "the static scratch array has no usable device address");
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return NNV_OK;
}

}  // namespace

using namespace nnv;

extern "C" nnv_status_t nnv_conv_exec_static(const nnv_plan_t* p, int32_t layer, int32_t v, int32_t math,
                                             const void* d_in, const void* d_addend, const void* d_wt,
                                             const void* d_bias, void* d_out, void* stream) {
    NNV_REQUIRE(p && d_in && d_wt && d_out, NNV_ERR_INVALID_ARG, "null argument");
    NNV_TRY(check_choice(*p, layer, v, math));
    NNV_REQUIRE(aligned256(d_in) && aligned256(d_wt) && aligned256(d_out) && (!d_addend || aligned256(d_addend)) &&
                    (!d_bias || aligned256(d_bias)),
                NNV_ERR_INVALID_ARG, "device pointers must be 256-byte aligned");
    NNV_REQUIRE(!p->layers[layer].has_bias || d_bias, NNV_ERR_INVALID_ARG, "layer %d has a bias but d_bias is null", layer);
    const uint64_t need = exec_ws_bytes(*p, layer, v, math);
    NNV_REQUIRE(need <= (uint64_t)NNV_STATIC_SCRATCH_BYTES, NNV_ERR_WORKSPACE_TOO_SMALL,
                "layer %d with this kernel needs %llu scratch bytes; the built-in scratch holds %llu -- use nnv_conv_exec "
                "with a caller-provided buffer", layer, (unsigned long long)need, (unsigned long long)NNV_STATIC_SCRATCH_BYTES);
    void* ws = nullptr;
    if (need) NNV_TRY(static_scratch(&ws));
    return do_exec(*p, layer, v, math, d_in, d_addend, d_wt, d_bias, d_out, ws, need, (cudaStream_t)stream);
}
