// Generic weight-gradient kernel on the fp32 ALUs, and the split-K reduction.
//
// dW[co, j] = sum over positions (n,ho,wo) of dY[n,co,ho,wo] * Xt[n,ci,h,w],
// with j = (ci,r,s) in the order of the dW layout, h = ho*stride_h-pad_h+r,
// w = wo*stride_w-pad_w+s, Xt the inflated Z (Section 4 of the paper: each
// pooled value stands for its whole k x k block) and 0 outside [0,H)x[0,W).
// The inflation is an index map (h/k, w/k) applied while the operand tile is
// gathered into shared memory; Xt never exists in global memory.
//
// This path takes every dtype, layout, filter, stride, padding and k. It is
// the fallback for shapes none of the tensor-core paths covers, for callers
// whose workspace has no room for staged operand copies, and the kernel behind
// the workspace-free entry point. The split-K reductions at the end of this
// file serve the tensor-core kernels too.
#include "ac_common.h"

namespace ac {
namespace {

constexpr int BM = 64;   // output channels per block
constexpr int BN = 64;   // (ci,r,s) columns per block
constexpr int BK = 16;   // positions per shared-memory step

__device__ __forceinline__ float ldf(const float* p, long long i) { return __ldg(p + i); }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p, long long i) {
    return __bfloat162float(__ldg(p + i));
}

struct SimtParams {
    int N, Ci, Co, H, W, R, S, sh, sw, ph, pw, kh, kw, Hp, Wp, Ho, Wo;
    int nhwc;
    int J;                 // Ci*R*S
    long long K;           // N*Ho*Wo
    long long k_per_split;
    long long dw_elems;
    int splits;
};

template <typename T>
__global__ void __launch_bounds__(256)
wgrad_simt_kernel(const T* __restrict__ z, const T* __restrict__ dy, float* __restrict__ out,
                  SimtParams p) {
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    const int j0 = blockIdx.x * BN, co0 = blockIdx.y * BM;
    const long long kbeg = (long long)blockIdx.z * p.k_per_split;
    const long long kend = min(kbeg + p.k_per_split, p.K);

    // column of the gathered operand this thread fills: fixed for the whole loop
    const int jl = tid % BN;
    const int j = j0 + jl;
    int ci = 0, r = 0, s = 0;
    const bool jvalid = j < p.J;
    if (jvalid) {
        if (p.nhwc) { ci = j % p.Ci; int t = j / p.Ci; s = t % p.S; r = t / p.S; }
        else        { s = j % p.S; int t = j / p.S; r = t % p.R; ci = t / p.R; }
    }
    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;

    const long long HoWo = (long long)p.Ho * p.Wo;
    for (long long k0 = kbeg; k0 < kend; k0 += BK) {
        // ---- dY tile: As[kk][co] ------------------------------------------
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int kk, col;
            if (p.nhwc) { col = tid % BM; kk = tid / BM + 4 * i; }
            else        { kk = tid % BK; col = tid / BK + 16 * i; }
            const long long pos = k0 + kk;
            const int co = co0 + col;
            float v = 0.f;
            if (pos < kend && co < p.Co) {
                const long long n = pos / HoWo;
                const long long rem = pos - n * HoWo;
                const long long off = p.nhwc ? pos * p.Co + co : (n * p.Co + co) * HoWo + rem;
                v = ldf(dy, off);
            }
            As[kk][col] = v;
        }
        // ---- inflated, padded, shifted input tile: Bs[kk][j] ----------------
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int kk = tid / BN + 4 * i;
            const long long pos = k0 + kk;
            float v = 0.f;
            if (pos < kend && jvalid) {
                const long long n = pos / HoWo;
                const int rem = (int)(pos - n * HoWo);
                const int ho = rem / p.Wo, wo = rem - ho * p.Wo;
                const int h = ho * p.sh - p.ph + r, w = wo * p.sw - p.pw + s;
                if (h >= 0 && h < p.H && w >= 0 && w < p.W) {
                    const int hp = h / p.kh, wp = w / p.kw;
                    const long long off =
                        p.nhwc ? ((n * p.Hp + hp) * (long long)p.Wp + wp) * p.Ci + ci
                               : ((n * p.Ci + ci) * (long long)p.Hp + hp) * p.Wp + wp;
                    v = ldf(z, off);
                }
            }
            Bs[kk][jl] = v;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) a[u] = As[kk][ty * 4 + u];
#pragma unroll
            for (int u = 0; u < 4; ++u) b[u] = Bs[kk][tx * 4 + u];
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int v = 0; v < 4; ++v) acc[u][v] = fmaf(a[u], b[v], acc[u][v]);
        }
        __syncthreads();
    }
    float* dst = out + (long long)blockIdx.z * p.dw_elems;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int co = co0 + ty * 4 + u;
        if (co >= p.Co) continue;
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const int jj = j0 + tx * 4 + v;
            if (jj < p.J) dst[(long long)co * p.J + jj] = acc[u][v];
        }
    }
}

// dw[i] = sum over slices of partials[slice][i], in a fixed order: four
// interleaved running sums combined as (s0+s1)+(s2+s3).
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const float* __restrict__ partials, int splits, long long elems,
                     float* __restrict__ dw) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= elems) return;
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
    int sp = 0;
    for (; sp + 4 <= splits; sp += 4) {
        s0 += __ldcs(partials + (long long)(sp + 0) * elems + i);
        s1 += __ldcs(partials + (long long)(sp + 1) * elems + i);
        s2 += __ldcs(partials + (long long)(sp + 2) * elems + i);
        s3 += __ldcs(partials + (long long)(sp + 3) * elems + i);
    }
    if (sp + 0 < splits) s0 += __ldcs(partials + (long long)(sp + 0) * elems + i);
    if (sp + 1 < splits) s1 += __ldcs(partials + (long long)(sp + 1) * elems + i);
    if (sp + 2 < splits) s2 += __ldcs(partials + (long long)(sp + 2) * elems + i);
    dw[i] = (s0 + s1) + (s2 + s3);
}

// Four consecutive elements per thread (elems % 4 == 0) and SL threads per element
// group: thread (e, sl) adds slices sl, sl + SL, ... in order, then the SL running sums
// of an element group are added in index order. Every order is fixed, so the result is
// reproducible; SL only trades parallelism against slice-loop length when dW is small
// and the slices are many.
template <int SL>
__global__ void __launch_bounds__(256)
splitk_reduce4_kernel(const float4* __restrict__ partials, int splits, long long elems4,
                      float4* __restrict__ dw) {
    constexpr int EL = 256 / SL;
    __shared__ float4 red[SL > 1 ? SL : 1][EL];
    const int e = threadIdx.x % EL, sl = threadIdx.x / EL;
    const long long i = (long long)blockIdx.x * EL + e;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    pdl_wait();   // launched behind the kernel that writes the partial sums, possibly before it ends
    if (i < elems4) {
        int sp = sl;
        for (; sp + 3 * SL < splits; sp += 4 * SL) {       // four loads in flight
            const float4 v0 = __ldcs(partials + (long long)sp * elems4 + i);
            const float4 v1 = __ldcs(partials + (long long)(sp + SL) * elems4 + i);
            const float4 v2 = __ldcs(partials + (long long)(sp + 2 * SL) * elems4 + i);
            const float4 v3 = __ldcs(partials + (long long)(sp + 3 * SL) * elems4 + i);
            acc.x += v0.x; acc.y += v0.y; acc.z += v0.z; acc.w += v0.w;
            acc.x += v1.x; acc.y += v1.y; acc.z += v1.z; acc.w += v1.w;
            acc.x += v2.x; acc.y += v2.y; acc.z += v2.z; acc.w += v2.w;
            acc.x += v3.x; acc.y += v3.y; acc.z += v3.z; acc.w += v3.w;
        }
        for (; sp < splits; sp += SL) {
            const float4 v = __ldcs(partials + (long long)sp * elems4 + i);
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
    }
    if (SL == 1) {
        if (i < elems4) dw[i] = acc;
        return;
    }
    red[sl][e] = acc;
    __syncthreads();
    if (sl == 0 && i < elems4) {
        float4 o = red[0][e];
#pragma unroll
        for (int j = 1; j < SL; ++j) {
            const float4 v = red[j][e];
            o.x += v.x; o.y += v.y; o.z += v.z; o.w += v.w;
        }
        dw[i] = o;
    }
}

template <int SL>
void launch_reduce4(const float* partials, int splits, long long e4, float* dw, cudaStream_t stream) {
    constexpr int EL = 256 / SL;
    launch_after(splitk_reduce4_kernel<SL>, dim3((unsigned)((e4 + EL - 1) / EL)), dim3(256), 0, stream,
                 reinterpret_cast<const float4*>(partials), splits, e4, reinterpret_cast<float4*>(dw));
}

}  // namespace

namespace {
__global__ void __launch_bounds__(256) axpby_kernel(const float* __restrict__ g, float beta, float* dw, long long n) {
    const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
    if (i < n) dw[i] = __fmaf_rn(beta, dw[i], g[i]);
}
}  // namespace

// dw <- beta * dw + g (one rounding per element)
ac_status launch_axpby(const float* g, float beta, float* dw, long long elems, cudaStream_t stream) {
    axpby_kernel<<<(unsigned)((elems + 255) / 256), 256, 0, stream>>>(g, beta, dw, elems);
    AC_CUDA_TRY(cudaGetLastError());
    return AC_OK;
}

ac_status launch_splitk_reduce(const float* partials, int splits, long long elems, float* dw,
                               cudaStream_t stream) {
    if (elems % 4 == 0) {
        const long long e4 = elems / 4;
        // enough threads to fill the chip (148 SMs x 1024), at most one thread per 2 slices
        int sl = 1;
        while (sl < 32 && e4 * sl < 148 * 1024 && sl * 4 <= splits) sl *= 2;
        switch (sl) {
            case 1: launch_reduce4<1>(partials, splits, e4, dw, stream); break;
            case 2: launch_reduce4<2>(partials, splits, e4, dw, stream); break;
            case 4: launch_reduce4<4>(partials, splits, e4, dw, stream); break;
            case 8: launch_reduce4<8>(partials, splits, e4, dw, stream); break;
            case 16: launch_reduce4<16>(partials, splits, e4, dw, stream); break;
            default: launch_reduce4<32>(partials, splits, e4, dw, stream); break;
        }
        AC_CUDA_TRY(cudaGetLastError());
        return AC_OK;
    }
    const unsigned grid = (unsigned)((elems + 255) / 256);
    splitk_reduce_kernel<<<grid, 256, 0, stream>>>(partials, splits, elems, dw);
    AC_CUDA_TRY(cudaGetLastError());
    return AC_OK;
}

ac_status launch_wgrad_simt(const Dims& d, const WgradPlan& pl, const void* z, const void* dy,
                            float* dw, void* workspace, cudaStream_t stream) {
    SimtParams p;
    p.N = d.N; p.Ci = d.Ci; p.Co = d.Co; p.H = d.H; p.W = d.W; p.R = d.R; p.S = d.S;
    p.sh = d.sh; p.sw = d.sw; p.ph = d.ph; p.pw = d.pw; p.kh = d.kh; p.kw = d.kw; p.Hp = d.Hp; p.Wp = d.Wp;
    p.Ho = d.Ho; p.Wo = d.Wo; p.nhwc = d.layout == AC_NHWC;
    p.J = d.Ci * d.R * d.S;
    p.K = d.K();
    p.k_per_split = pl.simt_k_per_split;
    p.dw_elems = d.dw_elems();
    p.splits = pl.splits;
    float* partials = reinterpret_cast<float*>(static_cast<char*>(workspace) + kStatusBlockBytes);
    float* out = pl.splits > 1 ? partials : dw;
    dim3 grid((p.J + BN - 1) / BN, (d.Co + BM - 1) / BM, pl.splits);
    if (grid.y > 65535u || grid.z > 65535u) return AC_ERR_UNSUPPORTED;
    record_timing_hook(0, stream);
    if (d.dtype == AC_F32)
        wgrad_simt_kernel<float><<<grid, 256, 0, stream>>>((const float*)z, (const float*)dy, out, p);
    else
        wgrad_simt_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(
            (const __nv_bfloat16*)z, (const __nv_bfloat16*)dy, out, p);
    record_timing_hook(1, stream);
    AC_CUDA_TRY(cudaGetLastError());
    if (pl.splits > 1) return launch_splitk_reduce(partials, pl.splits, p.dw_elems, dw, stream);
    return AC_OK;
}

}  // namespace ac
