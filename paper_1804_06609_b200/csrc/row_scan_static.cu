// dba_row_scan_static: the row scan for callers that may not allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off limits: inside a serving process whose memory
// pool was sized and frozen at start-up, in a plug-in that is handed buffers but owns no allocator, or on a
// latency path where an allocation (which may synchronise the device) is not acceptable.  dba_row_scan
// needs a scratch buffer for the per-segment partial results; this variant keeps that scratch in a
// fixed-size array that is part of the library image, so the caller passes inputs and outputs only.
#include <mutex>

#include "dba_internal.h"

namespace {

constexpr size_t kStaticScratchBytes = 4u << 20;   // 4 MiB, resident on every GPU that loads the library

// In host code this name is only a handle for the runtime, never an address a kernel can use: the device
// address is looked up with cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device; looked up once per device.
cudaError_t scratch_address(int device, void** out) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_ptr[device]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_ptr[device] = p;
    }
    *out = g_scratch_ptr[device];
    return cudaSuccess;
}

}  // namespace

extern "C" dba_status dba_row_scan_static(const void* logits_dev, int32_t logit_dtype, int32_t R, int32_t V,
                                          int64_t row_stride_elems, int32_t n_top, float* row_lse_dev,
                                          float* top_val_dev, int32_t* top_idx_dev, void* cuda_stream) {
    size_t need = 0;
    dba_status st = dba_row_scan_scratch_bytes(R, V, n_top, logit_dtype, &need);
    if (st != DBA_OK) return st;
    if (need > kStaticScratchBytes) return DBA_ERR_UNSUPPORTED;      // problem too large for the fixed scratch
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess) return DBA_ERR_CUDA;
    if (device < 0 || device >= kMaxDevices) return DBA_ERR_UNSUPPORTED;
    void* scratch = nullptr;
    if (scratch_address(device, &scratch) != cudaSuccess) return DBA_ERR_CUDA;
    // dba_row_scan overwrites every partial result it later reads and clears its status word itself, so
    // nothing of the previous call's contents survives into this one.
    return dba_row_scan(logits_dev, logit_dtype, R, V, row_stride_elems, n_top, scratch, kStaticScratchBytes,
                        row_lse_dev, top_val_dev, top_idx_dev, cuda_stream);
}

extern "C" size_t dba_row_scan_static_max_bytes(void) { return kStaticScratchBytes; }
