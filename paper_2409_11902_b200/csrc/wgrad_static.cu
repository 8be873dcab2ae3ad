// ac_conv2d_wgrad_compressed_static: the weight gradient for callers that
// cannot hand the library a workspace because they cannot allocate one.
//
// Who that is: code that runs where cudaMalloc is off limits -- inside a
// framework whose caching allocator already owns the whole device (a raw
// cudaMalloc there fails or forces a device-wide synchronisation), inside a
// latency-critical loop that must not take the allocator's lock, or in a
// plug-in that is only given tensors and no allocator handle.
//
// For them the split-K scratch of the fp32-ALU weight-gradient kernel lives
// in a fixed array in device memory that is part of this library's image.
// Every GPU that loads the library carries the array until the process exits.
#include <mutex>

#include "ac_common.h"

namespace ac {
namespace {

// Fixed split-K scratch. Shared by every call on the device; keeps whatever
// the previous call left in it.
static __device__ __align__(256) unsigned char g_static_scratch[AC_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
constexpr long long kMaxStaticSlice = 16384;   // positions per K-slice (the ordinary plan stops at 2048)
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {};  // per device: device address of g_static_scratch

// In host code `g_static_scratch` names a host-side shadow of the symbol, not
// device memory. The device address has to be asked for, once per device and
// with that device current.
ac_status scratch_for_current_device(void** out) {
    int dev = -1;
    AC_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return AC_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        AC_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
        if (!p) return AC_ERR_CUDA;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return AC_OK;
}

}  // namespace
}  // namespace ac

using namespace ac;

extern "C" ac_status ac_conv2d_wgrad_compressed_static(const ac_conv_desc* desc, const void* z,
                                                       const void* dy, float* dw, void* stream) {
    Dims d;
    ac_status st = make_dims(desc, true, &d);
    if (st != AC_OK) return st;
    if (!z || !dy || !dw) return AC_ERR_INVALID_ARG;
    if (!aligned16(z) || !aligned16(dy) || !aligned16(dw)) return AC_ERR_MISALIGNED;
    // As many K-slices as the fixed array holds, but no slice longer than kMaxStaticSlice positions:
    // a slice is one fp32 running sum per output, and its rounding error grows with its length.
    const WgradPlan p = plan_wgrad_simt(d, (size_t)AC_STATIC_SCRATCH_BYTES - kStatusBlockBytes);
    if (p.bytes > (size_t)AC_STATIC_SCRATCH_BYTES || p.simt_k_per_split > kMaxStaticSlice)
        return AC_ERR_WORKSPACE_TOO_SMALL;
    void* scratch = nullptr;
    st = scratch_for_current_device(&scratch);
    if (st != AC_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // The kernel writes every partial sum before the reduction reads it, so
    // only the status block at the front has to start from zero.
    AC_CUDA_TRY(cudaMemsetAsync(scratch, 0, kStatusBlockBytes, s));
    return launch_wgrad_simt(d, p, z, dy, dw, scratch, s);
}
