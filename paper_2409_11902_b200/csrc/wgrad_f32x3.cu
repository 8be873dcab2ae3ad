// fp32 inputs on the tensor cores. The paper's networks train in fp32; a single bf16 or TF32
// product cannot meet an fp32 weight gradient to 1e-5, so each fp32 value is written as the sum of
// three bf16 terms, x = h + m + l (h = bf16(x), m = bf16(x - h), l = bf16(x - h - m): 24 bits of
// significand between them), and the product Z * dY is expanded into the six partial products
// whose weight is at least 2^-16,
//
//     Z * dY  ~  Zh*Gh + Zh*Gm + Zm*Gh + Zh*Gl + Zl*Gh + Zm*Gm          (dropped terms: 2^-24 and less)
//
// all accumulated in fp32. A weight gradient is a sum over images, so the six products are simply six
// times as many images for the bf16 kernel: this file writes the two operand tensors
//
//     Z'  = [ Zh | Zh | Zm | Zh | Zl | Zm ]        dY' = [ Gh | Gm | Gh | Gl | Gh | Gm ]
//
// (each block N images, bf16, same layout) into the workspace, and the TMA-fed tcgen05 kernel runs
// on them unchanged with N' = 6 N. Measured against the fp64 definition: relative Frobenius error
// 7e-7 .. 2e-6, the fp32-ALU path gives 3e-7 .. 5e-7 and is five to ten times slower.
#include "ac_common.h"

namespace ac {
namespace {

__device__ __forceinline__ uint32_t pack_bf2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// One thread splits 8 consecutive fp32 values and stores three 16-byte vectors of bf16, each into
// the blocks that `ROLE` assigns to it (0: the Z' order above, 1: the dY' order).
template <int ROLE>
__global__ void __launch_bounds__(256)
split3_kernel(const float4* __restrict__ src, uint4* __restrict__ dst, long long n8) {
    const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
    if (i >= n8) return;
    const float4 a = __ldcs(src + 2 * i), b = __ldcs(src + 2 * i + 1);
    const float x[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    float h[8], m[8], l[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        h[j] = __bfloat162float(__float2bfloat16_rn(x[j]));
        const float r1 = x[j] - h[j];                       // exact: h shares x's leading bits
        m[j] = __bfloat162float(__float2bfloat16_rn(r1));
        l[j] = r1 - m[j];                                   // exact; rounded to bf16 when packed
    }
    const uint4 vh = make_uint4(pack_bf2(h[0], h[1]), pack_bf2(h[2], h[3]), pack_bf2(h[4], h[5]), pack_bf2(h[6], h[7]));
    const uint4 vm = make_uint4(pack_bf2(m[0], m[1]), pack_bf2(m[2], m[3]), pack_bf2(m[4], m[5]), pack_bf2(m[6], m[7]));
    const uint4 vl = make_uint4(pack_bf2(l[0], l[1]), pack_bf2(l[2], l[3]), pack_bf2(l[4], l[5]), pack_bf2(l[6], l[7]));
    if (ROLE == 0) {
        dst[i] = vh; dst[n8 + i] = vh; dst[2 * n8 + i] = vm;
        dst[3 * n8 + i] = vh; dst[4 * n8 + i] = vl; dst[5 * n8 + i] = vm;
    } else {
        dst[i] = vh; dst[n8 + i] = vm; dst[2 * n8 + i] = vh;
        dst[3 * n8 + i] = vl; dst[4 * n8 + i] = vh; dst[5 * n8 + i] = vm;
    }
}

inline size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }

// The bf16 problem the six products amount to.
bool widened(const Dims& d, Dims* d6) {
    if (d.dtype != AC_F32 || d.layout != AC_NHWC) return false;
    if (d.z_elems() % 8 != 0 || d.dy_elems() % 8 != 0) return false;
    if ((long long)d.N * 6 >= (1ll << 31)) return false;
    *d6 = d;
    d6->N = d.N * 6;
    d6->dtype = AC_BF16;
    d6->elt = 2;
    const long long lim = 1ll << 40;
    if (d6->z_elems() >= lim || d6->dy_elems() >= lim) return false;
    return tc2_supported(*d6, nullptr);
}

}  // namespace

bool f32x3_supported(const Dims& d) {
    Dims d6;
    return widened(d, &d6);
}

void plan_f32x3(const Dims& d, WgradPlan* pl) {
    Dims d6;
    widened(d, &d6);
    plan_tc2(d6, pl);
    pl->path = PATH_F32X3;
    pl->x3_off_z = up256(pl->bytes);
    pl->x3_off_dy = pl->x3_off_z + up256((size_t)d6.z_elems() * 2);
    pl->bytes = pl->x3_off_dy + up256((size_t)d6.dy_elems() * 2);
}

void f32x3_plan_info(const Dims& d, ac_plan_info* info) {
    Dims d6;
    widened(d, &d6);
    tc2_plan_info(d6, info);
    info->tensor_core = 3;
}

ac_status launch_wgrad_f32x3(const Dims& d, const WgradPlan& pl, const void* z, const void* dy,
                             float* dw, void* workspace, cudaStream_t stream) {
    Dims d6;
    if (!widened(d, &d6)) return AC_ERR_UNSUPPORTED;
    char* ws = static_cast<char*>(workspace);
    void* z6 = ws + pl.x3_off_z;
    void* dy6 = ws + pl.x3_off_dy;
    const long long nz8 = d.z_elems() / 8, ng8 = d.dy_elems() / 8;
    if ((nz8 + 255) / 256 >= (1ll << 31) || (ng8 + 255) / 256 >= (1ll << 31)) return AC_ERR_UNSUPPORTED;
    split3_kernel<0><<<(unsigned)((nz8 + 255) / 256), 256, 0, stream>>>(
        static_cast<const float4*>(z), static_cast<uint4*>(z6), nz8);
    split3_kernel<1><<<(unsigned)((ng8 + 255) / 256), 256, 0, stream>>>(
        static_cast<const float4*>(dy), static_cast<uint4*>(dy6), ng8);
    AC_CUDA_TRY(cudaGetLastError());
    return launch_wgrad_tc2(d6, pl, z6, dy6, dw, workspace, stream);
}

}  // namespace ac
