// exfold_moe_decode_noalloc: the decode call for callers that cannot allocate device memory.
//
// Some hosts of this library may not call cudaMalloc at all once they are running: an engine that
// hands out a fixed memory pool at start-up and forbids later allocations, a plugin that runs inside
// someone else's process and owns no allocator, or code that is already inside a region where an
// allocation would be refused. Such a caller cannot provide the workspace the ordinary decode call
// needs. For them the scratch memory lives in this file, in one device array of fixed size that is
// part of the library image. Every GPU that loads the library carries those bytes until the process
// exits, which is why the size is kept modest and stated in the header.
#include <mutex>

#include "common.cuh"

namespace {

// The scratch itself. Only device code may use this name as an address; on the host it is a
// stand-in for the symbol, and the real device address has to be asked for (see below).
static __device__ __align__(256) unsigned char g_static_scratch[EXFOLD_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the current device; looked up once per device, with that
// device current. Returns nullptr if the runtime cannot resolve the symbol.
void* scratch_for_current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_scratch_ptr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_scratch) != cudaSuccess) return nullptr;
        g_scratch_ptr[dev] = ptr;
    }
    return g_scratch_ptr[dev];
}

}  // namespace

extern "C" int exfold_moe_decode_noalloc(const exfold_layer* layer, const void* x, const float* logits, int64_t B,
                                         const void* w_gate, const void* w_up, const void* w_down,
                                         const exfold_tables* tables, int32_t pool_m, void* y,
                                         const exfold_decode_meta* meta, void* cuda_stream) {
    if (layer == nullptr || B < 1) return EXFOLD_ERR_INVALID_ARG;
    void* ws = scratch_for_current_device();
    if (ws == nullptr) return EXFOLD_ERR_CUDA;
    // The ordinary call checks that the array is large enough before it launches anything, and clears,
    // on the stream, everything in the scratch that has to start at zero (the status record and the
    // fp32 accumulator); the rest is overwritten before it is read.
    int rc = exfold_moe_decode(layer, x, logits, B, w_gate, w_up, w_down, tables, pool_m, y, meta, ws,
                               (size_t)EXFOLD_STATIC_SCRATCH_BYTES, cuda_stream);
    return rc == EXFOLD_ERR_WORKSPACE_TOO_SMALL ? EXFOLD_ERR_EXCEEDS_STATIC_SCRATCH : rc;
}

// The status record of the calls above lives at the start of the built-in array, where the caller cannot
// point exfold_device_status at it; this is the same check for that record.
extern "C" int exfold_device_status_noalloc(void* cuda_stream) {
    void* ws = scratch_for_current_device();
    if (ws == nullptr) return EXFOLD_ERR_CUDA;
    return exfold::read_status_record(ws, reinterpret_cast<cudaStream_t>(cuda_stream));
}

extern "C" int exfold_static_scratch_address(void** address) {
    if (address == nullptr) return EXFOLD_ERR_INVALID_ARG;
    *address = scratch_for_current_device();
    return *address != nullptr ? EXFOLD_OK : EXFOLD_ERR_CUDA;
}
