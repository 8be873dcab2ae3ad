// Internal definitions shared by the translation units of libac (not installed).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ac.h"

namespace ac {

constexpr int kNumSMs = 148;               // B200: the only target of this library
constexpr size_t kStatusBlockBytes = 256;  // first bytes of every wgrad workspace

// Derived sizes of a validated descriptor.
struct Dims {
    int N, Ci, Co, H, W, R, S, sh, sw, ph, pw, k;
    int kh, kw;   // pooling block; k = kh = kw for the square blocks of the paper. Code that reads
                  // only `k` must not be reached with kh != kw (each path's *_supported says so).
    int Hp, Wp;   // pooled size (ceil)
    int Ho, Wo;   // convolution output size
    int dtype, layout;
    int elt;      // bytes per element of X, Z, dY
    // Tensor-core kernels only: the most MMA instructions that may add into one accumulator before
    // it is written out as a partial sum (0: no limit). The tensor core adds into its fp32
    // accumulator with truncation, a bias that grows with the length of the chain; bf16 results
    // (bound 1e-2) never notice, fp32 results assembled from bf16 terms (bound 1e-5) do.
    int max_chain;
    // SMs a weight-gradient plan may count on (ac_set_sm_budget; kNumSMs unless the caller runs several
    // weight gradients side by side): the tensor-core paths launch about this many CTAs, one per SM.
    int sms;
    long long x_elems() const { return (long long)N * Ci * H * W; }
    long long z_elems() const { return (long long)N * Ci * Hp * Wp; }
    long long dy_elems() const { return (long long)N * Co * Ho * Wo; }
    long long dw_elems() const { return (long long)Co * Ci * R * S; }
    long long K() const { return (long long)N * Ho * Wo; }
};

// Validates and expands a descriptor. `need_conv` = false checks only the
// fields ac_compress uses.
// k_h, k_w > 0: a non-uniform pooling block, desc->k is then ignored.
ac_status make_dims(const ac_conv_desc* d, bool need_conv, Dims* out, int k_h = 0, int k_w = 0);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ---- wgrad planning (pure host arithmetic; decides kernel and split-K) ------
enum WgradPath { PATH_SIMT = 0, PATH_TC = 1, PATH_TC2 = 2, PATH_STAGED = 3, PATH_GATHER = 4 };

struct WgradPlan {
    int path;        // WgradPath
    int splits;      // K-slices whose partial dW tensors are summed in fixed order
    // SIMT path: each slice covers `simt_k_per_split` flattened (n,ho,wo) positions
    long long simt_k_per_split;
    // tensor-core path
    int tc_band;     // output rows per K-tile
    int tc_groups;   // CTAs sharing one K-slice, each owning part of the output
    int tc_ktiles;   // K-tiles in the whole problem
    int tc_stages;   // shared-memory pipeline depth
    // staged path: where the staged operands and (NCHW) the kernel's dW sit in the workspace
    size_t st_off_z, st_off_dy, st_off_dw, st_off_small;
    size_t bytes;    // workspace bytes including the status block
};

WgradPlan plan_wgrad(const Dims& d);
// The fp32-ALU path's plan, whatever plan_wgrad picks. K-slices cover 256..2048 positions each unless
// their partial sums would not fit `max_partial_bytes`; then there are fewer, longer slices (one
// slice, written straight to dW, needs no scratch at all).
WgradPlan plan_wgrad_simt(const Dims& d, size_t max_partial_bytes = (size_t)256 << 20);

// ---- launchers (each enqueues on `stream`, returns AC_OK or AC_ERR_CUDA) -----
ac_status launch_compress(const Dims& d, const void* x, void* z, void* y_out, cudaStream_t stream);
ac_status launch_compress_mask(const Dims& d, const void* a, void* z, void* mask, cudaStream_t stream);
ac_status launch_wgrad_simt(const Dims& d, const WgradPlan& p, const void* z, const void* dy,
                            float* dw, void* workspace, cudaStream_t stream);
bool tc_supported(const Dims& d);
void plan_tc(const Dims& d, WgradPlan* p);
void tc_plan_info(const Dims& d, ac_plan_info* info);
ac_status launch_wgrad_tc(const Dims& d, const WgradPlan& p, const void* z, const void* dy,
                          float* dw, void* workspace, cudaStream_t stream);
// TMA-fed tensor-core kernel (no inflation in shared memory); k_eff = useful / issued K
bool tc2_supported(const Dims& d, double* k_eff);
void plan_tc2(const Dims& d, WgradPlan* p);
void tc2_plan_info(const Dims& d, ac_plan_info* info);
ac_status launch_wgrad_tc2(const Dims& d, const WgradPlan& p, const void* z, const void* dy,
                           float* dw, void* workspace, cudaStream_t stream, bool keep_status = false);
int tc2_chain_length(const Dims& d);
double tc2_cost_cycles(const Dims& d, int* tile_copies);
// fp32 and/or NCHW inputs staged for the TMA-fed kernel (wgrad_staged.cu)
bool staged_supported(const Dims& d);
// bf16 NHWC problems the TMA-fed kernel takes directly but that run faster on an inflated copy of Z
// (small odd maps with padding); true: plan and launch them as staged problems
bool staged_inflate_preferred(const Dims& d);
void plan_staged(const Dims& d, WgradPlan* p);
void staged_plan_info(const Dims& d, ac_plan_info* info);
ac_status launch_wgrad_staged(const Dims& d, const WgradPlan& p, const void* z, const void* dy,
                             float* dw, void* workspace, cudaStream_t stream);
// few input channels: the operand gathered into a [positions][taps x channels] matrix (wgrad_staged.cu)
bool gather_supported(const Dims& d);
void plan_gather(const Dims& d, WgradPlan* p);
void gather_plan_info(const Dims& d, ac_plan_info* info);
ac_status launch_wgrad_gather(const Dims& d, const WgradPlan& p, const void* z, const void* dy,
                              float* dw, void* workspace, cudaStream_t stream);
// the same with the operand matrix built inside the kernel (wgrad_gather_fused.cu): layers whose taps share columns
bool gather_fused_supported(const Dims& d);
size_t gather_fused_workspace_bytes(const Dims& d);
void gather_fused_plan_info(const Dims& d, ac_plan_info* info);
ac_status launch_wgrad_gather_fused(const Dims& d, const void* z, const void* dy, float* dw, void* workspace,
                                    cudaStream_t stream);
size_t tc2_collapsed_workspace_bytes(const Dims& d, int* tiles_collapsed, int* tiles_dense);
ac_status launch_wgrad_tc2_collapsed(const Dims& d, const void* z, const void* dy, float* dw,
                                     void* workspace, cudaStream_t stream);
ac_status launch_bounded_wait_selftest(void* workspace, long long limit_cycles, cudaStream_t stream);
ac_status launch_axpby(const float* g, float beta, float* dw, long long elems, cudaStream_t stream);
ac_status launch_splitk_reduce(const float* partials, int splits, long long elems, float* dw,
                               cudaStream_t stream);

// Programmatic dependent launch. A kernel launched with launch_after() may start while the kernel
// before it in the stream is still running, provided that kernel has called
// pdl_launch_dependents() in every CTA; whatever it does before pdl_wait() (barrier set-up, TMEM
// allocation, clearing shared memory) then overlaps the predecessor's tail. pdl_wait() returns once
// the predecessor has completed and its writes are visible; every thread calls it before its first
// access to global memory. With a predecessor that never signals, the launch behaves like an
// ordinary one and pdl_wait() returns at once.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_after(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                Args... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// Profiling hook (ac_set_kernel_timing_events): which = 0 before, 1 after the main kernel.
void record_timing_hook(int which, cudaStream_t stream);

// Raises a kernel's dynamic shared-memory limit once per device (the attribute is per device).
template <typename Kernel>
inline ac_status ensure_smem_limit(Kernel kernel, int bytes, bool (&done)[64]) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return AC_ERR_CUDA;
    if (!done[dev]) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess)
            return AC_ERR_CUDA;
        done[dev] = true;
    }
    return AC_OK;
}

#define AC_CUDA_TRY(expr)                           \
    do {                                            \
        cudaError_t e__ = (expr);                   \
        if (e__ != cudaSuccess) return AC_ERR_CUDA; \
    } while (0)

}  // namespace ac
