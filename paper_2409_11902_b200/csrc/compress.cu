// Compression kernels: Z = k x k average pooling of the convolution input X
// (Section 4 of the paper; blocks aligned to X's index 0, partial edge blocks
// averaged over the elements they have), optionally fused with the ReLU that
// produces X. Bandwidth bound: every element of X is read once with 16-byte
// loads, sums are formed in fp32 registers (plus one warp shuffle where a
// block spans two lanes), Z is written once.
#include "ac_common.h"

namespace ac {
namespace {

template <typename T> struct VecTraits;
template <> struct VecTraits<float> { static constexpr int VW = 4; };
template <> struct VecTraits<__nv_bfloat16> { static constexpr int VW = 8; };

// 16-byte global load; streaming hint when the buffer is only read.
template <bool STREAM>
__device__ __forceinline__ uint4 load16(const void* p) {
    if (STREAM) return __ldcs(reinterpret_cast<const uint4*>(p));
    return *reinterpret_cast<const uint4*>(p);
}

template <typename T, bool RELU>
__device__ __forceinline__ void unpack(uint4& raw, float* f);

template <>
__device__ __forceinline__ void unpack<float, false>(uint4& raw, float* f) {
    f[0] = __uint_as_float(raw.x); f[1] = __uint_as_float(raw.y);
    f[2] = __uint_as_float(raw.z); f[3] = __uint_as_float(raw.w);
}
template <>
__device__ __forceinline__ void unpack<float, true>(uint4& raw, float* f) {
    f[0] = fmaxf(__uint_as_float(raw.x), 0.f); f[1] = fmaxf(__uint_as_float(raw.y), 0.f);
    f[2] = fmaxf(__uint_as_float(raw.z), 0.f); f[3] = fmaxf(__uint_as_float(raw.w), 0.f);
    raw = make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]),
                     __float_as_uint(f[3]));
}
__device__ __forceinline__ void bf2_to_f(uint32_t u, float& lo, float& hi) {
    lo = __uint_as_float(u << 16);
    hi = __uint_as_float(u & 0xffff0000u);
}
// max(x,0) on two packed bf16 in one instruction (-0 and NaN become +0, like fmaxf(x, 0)).
__device__ __forceinline__ uint32_t relu_bf2(uint32_t u) {
    __nv_bfloat162 v = *reinterpret_cast<__nv_bfloat162*>(&u);
    v = __hmax2(v, __float2bfloat162_rn(0.f));
    return *reinterpret_cast<uint32_t*>(&v);
}
// 0xffff in each half of the result whose bf16 is greater than zero
__device__ __forceinline__ uint32_t positive_bf2(uint32_t u) {
    return __hgt2_mask(*reinterpret_cast<__nv_bfloat162*>(&u), __float2bfloat162_rn(0.f));
}
template <>
__device__ __forceinline__ void unpack<__nv_bfloat16, false>(uint4& raw, float* f) {
    bf2_to_f(raw.x, f[0], f[1]); bf2_to_f(raw.y, f[2], f[3]);
    bf2_to_f(raw.z, f[4], f[5]); bf2_to_f(raw.w, f[6], f[7]);
}
template <>
__device__ __forceinline__ void unpack<__nv_bfloat16, true>(uint4& raw, float* f) {
    raw.x = relu_bf2(raw.x); raw.y = relu_bf2(raw.y);
    raw.z = relu_bf2(raw.z); raw.w = relu_bf2(raw.w);
    unpack<__nv_bfloat16, false>(raw, f);
}

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) {
    return __float2bfloat16_rn(v);
}

template <typename T>
__device__ __forceinline__ uint4 pack(const float* f);
template <>
__device__ __forceinline__ uint4 pack<float>(const float* f) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]),
                      __float_as_uint(f[3]));
}
__device__ __forceinline__ uint32_t f2_to_bf2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
template <>
__device__ __forceinline__ uint4 pack<__nv_bfloat16>(const float* f) {
    return make_uint4(f2_to_bf2(f[0], f[1]), f2_to_bf2(f[2], f[3]), f2_to_bf2(f[4], f[5]),
                      f2_to_bf2(f[6], f[7]));
}

// Mask mode of the fused form: instead of Y = max(A, 0) the kernel stores one bit per element
// (1 where A > 0), which is all a ReLU backward needs. Bit i of the mask is element i of A in
// memory order, least significant bit first. A 16-byte vector is 8 bf16 = one mask byte, or 4
// fp32 = half a byte: two neighbouring lanes then combine their halves with one shuffle.
template <typename T>
__device__ __forceinline__ unsigned positive_bits(const uint4& raw, const float* f);
template <>
__device__ __forceinline__ unsigned positive_bits<float>(const uint4&, const float* f) {
    unsigned b = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) b |= (f[i] > 0.f ? 1u : 0u) << i;
    return b;
}
template <>
__device__ __forceinline__ unsigned positive_bits<__nv_bfloat16>(const uint4& raw, const float*) {
    // word j holds elements 2j (low half) and 2j+1 (high half): pick bit 2j of the low
    // half's flags and bit 16 + 2j + 1 of the high half's, then fold the two halves
    const unsigned r = (positive_bf2(raw.x) & 0x00020001u) | (positive_bf2(raw.y) & 0x00080004u) |
                       (positive_bf2(raw.z) & 0x00200010u) | (positive_bf2(raw.w) & 0x00800040u);
    return (r | (r >> 16)) & 0xffu;
}
template <int VW>
__device__ __forceinline__ void store_mask(unsigned char* mask, long long elem_off, unsigned bits,
                                           bool valid, unsigned lanes) {
    if (VW == 8) {
        if (valid) mask[elem_off >> 3] = (unsigned char)bits;
    } else {
        const unsigned other = __shfl_xor_sync(lanes, bits, 1);
        if (valid && (threadIdx.x & 1) == 0) mask[elem_off >> 3] = (unsigned char)(bits | (other << 4));
    }
}

// ---- NHWC, C a multiple of the vector width --------------------------------
// One thread per output vector (n, p, q, 16 bytes of channels): k*k independent
// 16-byte loads, element-wise fp32 sums, one 16-byte store. Adjacent threads
// hold adjacent channel vectors, so every warp-wide access is contiguous.
// Grid: x covers the (q, channel vector) pairs of one pooled row, y = p, z = n,
// so that no 64-bit division is needed. K > 0: pooling factor known at compile
// time, all loads of up to four rows issued before the first use; K = 0: any k.
// x is not __restrict__: the fused ReLU may run in place (y == x); a thread reads its own
// elements before it writes them and no other thread touches them.
template <typename T, int K, int MODE>   // MODE 0: pool only, 1: also store max(x,0), 2: also store the sign mask, 3: both
__global__ void __launch_bounds__(256)
compress_nhwc_vec(const T* x, T* __restrict__ z, T* y, unsigned char* mask, int H, int W, int CV,
                  int kh, int kw, int Hp, int Wp) {
    pdl_launch_dependents();   // a weight-gradient kernel queued behind this one may begin its set-up
    constexpr bool RELU = MODE != 0, STORE_Y = MODE == 1 || MODE == 3, MASK = MODE >= 2;
    constexpr int VW = VecTraits<T>::VW;
    const unsigned item = blockIdx.x * 256u + threadIdx.x;
    const bool in_range = item < (unsigned)Wp * (unsigned)CV;
    const unsigned lanes = MASK ? __ballot_sync(0xffffffffu, in_range) : 0u;   // pairs leave together
    if (!in_range) return;
    const int q = (int)(item / (unsigned)CV);
    const int cv = (int)(item - (unsigned)q * (unsigned)CV);
    const int p = blockIdx.y;
    const long long n = blockIdx.z;
    const int kkh = K > 0 ? K : kh, kkw = K > 0 ? K : kw;   // K = 0 also serves blocks with kh != kw
    const int h0 = p * kkh, w0 = q * kkw;
    const int h1 = min(h0 + kkh, H), w1 = min(w0 + kkw, W);
    float acc[VW];
#pragma unroll
    for (int i = 0; i < VW; ++i) acc[i] = 0.f;
    if (K > 0) {
        constexpr int KR = K > 0 ? (K > 4 ? 2 : K) : 1;   // rows in flight at once
#pragma unroll
        for (int hb = 0; hb < (K > 0 ? K : 1); hb += KR) {
            uint4 raw[KR][K > 0 ? K : 1];
#pragma unroll
            for (int dh = 0; dh < KR; ++dh)
#pragma unroll
                for (int dw = 0; dw < K; ++dw) {
                    const int h = h0 + hb + dh, w = w0 + dw;
                    raw[dh][dw] = make_uint4(0, 0, 0, 0);
                    if (h < h1 && w < w1)
                        raw[dh][dw] = load16<!STORE_Y>(x + ((((n * H + h) * (long long)W + w) * CV + cv) * VW));
                }
#pragma unroll
            for (int dh = 0; dh < KR; ++dh) {
                float row[VW];
#pragma unroll
                for (int i = 0; i < VW; ++i) row[i] = 0.f;
#pragma unroll
                for (int dw = 0; dw < K; ++dw) {
                    const int h = h0 + hb + dh, w = w0 + dw;
                    float f[VW];
                    unpack<T, RELU>(raw[dh][dw], f);
                    if (STORE_Y && h < h1 && w < w1)
                        *reinterpret_cast<uint4*>(y + ((((n * H + h) * (long long)W + w) * CV + cv) * VW)) =
                            raw[dh][dw];
                    if (MASK)
                        store_mask<VW>(mask, (((n * H + h) * (long long)W + w) * CV + cv) * VW,
                                       positive_bits<T>(raw[dh][dw], f), h < h1 && w < w1, lanes);
#pragma unroll
                    for (int i = 0; i < VW; ++i) row[i] += f[i];
                }
#pragma unroll
                for (int i = 0; i < VW; ++i) acc[i] += row[i];
            }
        }
    } else {
        for (int h = h0; h < h1; ++h) {
            float row[VW];
#pragma unroll
            for (int i = 0; i < VW; ++i) row[i] = 0.f;
            const long long rbase = ((n * H + h) * (long long)W) * CV + cv;
            for (int w = w0; w < w1; ++w) {
                const long long off = (rbase + (long long)w * CV) * VW;
                uint4 raw = load16<!STORE_Y>(x + off);
                float f[VW];
                unpack<T, RELU>(raw, f);
                if (STORE_Y) *reinterpret_cast<uint4*>(y + off) = raw;
#pragma unroll
                for (int i = 0; i < VW; ++i) row[i] += f[i];
            }
#pragma unroll
            for (int i = 0; i < VW; ++i) acc[i] += row[i];
        }
    }
    const float inv = 1.0f / (float)((h1 - h0) * (w1 - w0));
#pragma unroll
    for (int i = 0; i < VW; ++i) acc[i] *= inv;
    *reinterpret_cast<uint4*>(z + ((((n * Hp + p) * (long long)Wp + q) * CV + cv) * VW)) = pack<T>(acc);
}

template <typename T, int MODE>
ac_status launch_nhwc_vec(const T* x, T* z, T* y, unsigned char* mask, long long N, int H, int W, int CV, int kh,
                          int kw, int Hp, int Wp, cudaStream_t st) {
    const long long row_items = (long long)Wp * CV;
    if (row_items >= (1ll << 31) || Hp > 65535 || N > 65535) return AC_ERR_UNSUPPORTED;
    dim3 grid((unsigned)((row_items + 255) / 256), (unsigned)Hp, (unsigned)N);
    switch (kh == kw ? kh : 0) {
        case 1: compress_nhwc_vec<T, 1, MODE><<<grid, 256, 0, st>>>(x, z, y, mask, H, W, CV, kh, kw, Hp, Wp); break;
        case 2: compress_nhwc_vec<T, 2, MODE><<<grid, 256, 0, st>>>(x, z, y, mask, H, W, CV, kh, kw, Hp, Wp); break;
        case 4: compress_nhwc_vec<T, 4, MODE><<<grid, 256, 0, st>>>(x, z, y, mask, H, W, CV, kh, kw, Hp, Wp); break;
        case 8: compress_nhwc_vec<T, 8, MODE><<<grid, 256, 0, st>>>(x, z, y, mask, H, W, CV, kh, kw, Hp, Wp); break;
        default:
            if (MODE >= 2) return AC_ERR_UNSUPPORTED;   // the mask needs warp-uniform loops
            compress_nhwc_vec<T, 0, MODE><<<grid, 256, 0, st>>>(x, z, y, mask, H, W, CV, kh, kw, Hp, Wp);
            break;
    }
    AC_CUDA_TRY(cudaGetLastError());
    return AC_OK;
}

// ---- NCHW, W a multiple of the vector width and of k, k in {2,4,8} ---------
// One thread per (plane, pooled row, 16-byte column chunk): lanes of a warp
// read consecutive 16-byte chunks of a row. Vertical sums over the k rows are
// element-wise; the horizontal sum is a tree inside the vector, finished with
// one warp shuffle when a block spans two lanes (fp32, k = 8).
template <typename T, int K, int MODE, typename I>
__global__ void __launch_bounds__(256)
compress_nchw_vec(const T* x, T* __restrict__ z, T* y, unsigned char* mask, int H, int W, int Hp,
                  int Wp, long long total) {
    pdl_launch_dependents();   // a weight-gradient kernel queued behind this one may begin its set-up
    constexpr bool RELU = MODE != 0, STORE_Y = MODE == 1 || MODE == 3, MASK = MODE >= 2;
    constexpr int VW = VecTraits<T>::VW;
    const int WV = W / VW;
    I idx = (I)blockIdx.x * 256u + threadIdx.x;     // I = unsigned when the item count fits 32 bits
    const bool active = idx < (I)total;
    if (!active) idx = (I)(total - 1);  // keep whole warps alive for the shuffle
    const I t0 = idx / (I)WV;
    const int wv = (int)(idx - t0 * (I)WV);
    const I nci = t0 / (I)Hp;
    const int p = (int)(t0 - nci * (I)Hp);
    const long long nc = (long long)nci;
    const int h0 = p * K;
    const int h1 = min(h0 + K, H);
    float acc[VW];
#pragma unroll
    for (int i = 0; i < VW; ++i) acc[i] = 0.f;
#pragma unroll
    for (int dh = 0; dh < K; ++dh) {
        const int h = h0 + dh;
        const long long off = ((nc * H + h) * (long long)WV + wv) * VW;
        unsigned bits = 0;
        if (h < h1) {
            uint4 raw = load16<!STORE_Y>(x + off);
            float f[VW];
            unpack<T, RELU>(raw, f);
            if (STORE_Y && active) *reinterpret_cast<uint4*>(y + off) = raw;
            if (MASK) bits = positive_bits<T>(raw, f);
#pragma unroll
            for (int i = 0; i < VW; ++i) acc[i] += f[i];
        }
        if (MASK) store_mask<VW>(mask, off, bits, active && h < h1, 0xffffffffu);
    }
    const float inv = 1.0f / (float)((h1 - h0) * K);
    if (K <= VW) {
        constexpr int NO = (K <= VW) ? VW / K : 1;  // outputs per thread
        float out[NO];
#pragma unroll
        for (int j = 0; j < NO; ++j) {
            // pairwise tree over the K partial sums of output j
            float s[K];
#pragma unroll
            for (int i = 0; i < K; ++i) s[i] = acc[(j * K + i) % VW];
#pragma unroll
            for (int w = K / 2; w >= 1; w /= 2)
#pragma unroll
                for (int i = 0; i < w; ++i) s[i] += s[i + w];
            out[j] = s[0] * inv;
        }
        if (active) {
            T* zp = z + (nc * Hp + p) * (long long)Wp + (long long)wv * NO;
#pragma unroll
            for (int j = 0; j < NO; ++j) zp[j] = from_f<T>(out[j]);
        }
    } else {
        // K == 2 * VW: lanes 2j and 2j+1 hold the two halves of one block
        float s = (acc[0] + acc[1 % VW]) + (acc[2 % VW] + acc[3 % VW]);
        s += __shfl_xor_sync(0xffffffffu, s, 1);
        if (active && (wv & 1) == 0)
            z[(nc * Hp + p) * (long long)Wp + (wv >> 1)] = from_f<T>(s * inv);
    }
}

// ---- any layout, any k, any size: one thread per element of Z ---------------
template <typename T, bool RELU>
__global__ void __launch_bounds__(256)
compress_generic(const T* x, T* __restrict__ z, T* y, int C, int H, int W, int kh, int kw, int Hp, int Wp,
                 int nhwc, long long total) {
    pdl_launch_dependents();   // a weight-gradient kernel queued behind this one may begin its set-up
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    int c, p, q;
    long long n, t = idx;
    if (nhwc) { c = (int)(t % C); t /= C; q = (int)(t % Wp); t /= Wp; p = (int)(t % Hp); n = t / Hp; }
    else      { q = (int)(t % Wp); t /= Wp; p = (int)(t % Hp); t /= Hp; c = (int)(t % C); n = t / C; }
    const int h0 = p * kh, w0 = q * kw;
    const int h1 = min(h0 + kh, H), w1 = min(w0 + kw, W);
    float acc = 0.f;
    for (int h = h0; h < h1; ++h) {
        float row = 0.f;
        for (int w = w0; w < w1; ++w) {
            const long long off = nhwc ? ((n * H + h) * (long long)W + w) * C + c
                                       : ((n * C + c) * (long long)H + h) * W + w;
            float v = to_f(x[off]);
            if (RELU) { v = fmaxf(v, 0.f); y[off] = from_f<T>(v); }
            row += v;
        }
        acc += row;
    }
    z[idx] = from_f<T>(acc * (1.0f / (float)((h1 - h0) * (w1 - w0))));
}

// ---- NHWC, C not a multiple of the vector width but rows of W * C elements that are -----------
// (a network's 3-channel input). The input rows of RB pooled rows go through shared memory: they are
// fetched with 16-byte loads that are contiguous across the block (a row of W * C elements is one
// dense run of bytes, whatever C is), each thread then forms outputs from 2- or 4-byte shared-memory
// reads, and the pooled rows leave as 16-byte stores again when their length allows it.
// Grid: x = group of RB pooled rows, y = image. Dynamic shared memory: kh * RB input rows + RB
// output rows.
// CC, KK: channel count and (square) pooling factor when known at compile time (0: run-time values),
// so that the index arithmetic per output has no division and the sums unroll.
template <typename T, bool RELU, int CC, int KK>
__global__ void __launch_bounds__(256)
compress_nhwc_rows(const T* x, T* __restrict__ z, T* y, int C_, int H, int W, int kh_, int kw_, int Hp, int Wp,
                   int RB, int vec_out) {
    extern __shared__ __align__(16) unsigned char rows_smem[];
    pdl_launch_dependents();
    constexpr int VW = VecTraits<T>::VW;
    const int C = CC > 0 ? CC : C_, kh = KK > 0 ? KK : kh_, kw = KK > 0 ? KK : kw_;
    const int row_el = W * C, out_el = Wp * C;
    const int row_v = row_el / VW;                        // 16-byte vectors per input row
    T* in = reinterpret_cast<T*>(rows_smem);              // [kh * RB][row_el]
    T* out = in + (size_t)kh * RB * row_el;               // [RB][out_el]
    const int p0 = blockIdx.x * RB;
    const long long n = blockIdx.y;
    const int h_begin = p0 * kh;
    const int h_end = min(H, (p0 + RB) * kh);             // input rows [h_begin, h_end) are this block's
    const int nrows = h_end - h_begin;
    const T* src = x + (n * H + h_begin) * (long long)row_el;
    // all of a thread's loads are issued before the first is used
    for (int v = threadIdx.x; v < nrows * row_v; v += 256) {
        uint4 raw = load16<!RELU>(src + (size_t)v * VW);
        if (RELU) {
            float f[VW];
            unpack<T, true>(raw, f);                      // raw becomes max(raw, 0)
            *reinterpret_cast<uint4*>(y + (n * H + h_begin) * (long long)row_el + (size_t)v * VW) = raw;
        }
        reinterpret_cast<uint4*>(in)[v] = raw;
    }
    __syncthreads();
    const int prows = min(RB, Hp - p0);
    for (int r = 0; r < prows; ++r) {
        const int h0 = (p0 + r) * kh, h1 = min(h0 + kh, H);
        const T* band = in + (size_t)(h0 - h_begin) * row_el;
        // consecutive threads, consecutive outputs: their shared-memory reads are about 2 elements apart
        for (int j = threadIdx.x; j < out_el; j += 256) {
            const int q = j / C, c = j - q * C;
            const int w0 = q * kw;
            const T* cell = band + w0 * C + c;
            float acc = 0.f;
            float cnt;
            if (KK > 0 && h1 - h0 == KK && w0 + KK <= W) {
#pragma unroll
                for (int dh = 0; dh < (KK > 0 ? KK : 1); ++dh) {
                    float row = 0.f;
#pragma unroll
                    for (int dw = 0; dw < (KK > 0 ? KK : 1); ++dw) row += to_f(cell[dh * row_el + dw * C]);
                    acc += row;
                }
                cnt = (float)(KK * KK);
            } else {
                const int w1 = min(w0 + kw, W);
                for (int h = h0; h < h1; ++h) {
                    float row = 0.f;
                    for (int w = w0; w < w1; ++w) row += to_f(cell[(h - h0) * row_el + (w - w0) * C]);
                    acc += row;
                }
                cnt = (float)((h1 - h0) * (w1 - w0));
            }
            const T val = from_f<T>(acc * (1.0f / cnt));
            if (vec_out) out[r * out_el + j] = val;
            else z[((n * Hp + p0 + r) * (long long)Wp) * C + j] = val;
        }
    }
    if (!vec_out) return;
    __syncthreads();
    uint4* dst = reinterpret_cast<uint4*>(z + ((n * Hp + p0) * (long long)Wp) * C);
    for (int v = threadIdx.x; v < prows * out_el / VW; v += 256) dst[v] = reinterpret_cast<const uint4*>(out)[v];
}

// Whether the row kernel takes the problem, and with how many pooled rows per block (0: no).
template <typename T>
int rows_per_block(const Dims& d) {
    constexpr int VW = VecTraits<T>::VW;
    const long long row_el = (long long)d.W * d.Ci, out_el = (long long)d.Wp * d.Ci;
    if (d.layout != AC_NHWC || row_el % VW != 0 || d.N > 65535) return 0;
    const long long per_row = (d.kh * row_el + out_el) * (long long)sizeof(T);      // shared memory per pooled row
    if (per_row > 40 * 1024) return 0;
    long long rb = (24 * 1024) / per_row;      // about 24 KB per block (measured best of 4 ... 40 KB on a 3-channel 224 x 224 input)
    if (rb < 1) rb = 1;
    if (rb > d.Hp) rb = d.Hp;
    return (int)rb;
}

inline unsigned blocks_for(long long total) { return (unsigned)((total + 255) / 256); }

template <typename T, int K, int MODE>
void launch_nchw_vec(const Dims& d, const T* x, T* z, T* y, unsigned char* mask, long long total,
                     cudaStream_t st) {
    const unsigned g = blocks_for(total);
    if (total < (1ll << 32))
        compress_nchw_vec<T, K, MODE, unsigned><<<g, 256, 0, st>>>(x, z, y, mask, d.H, d.W, d.Hp, d.Wp, total);
    else
        compress_nchw_vec<T, K, MODE, unsigned long long><<<g, 256, 0, st>>>(x, z, y, mask, d.H, d.W, d.Hp,
                                                                              d.Wp, total);
}

// MODE 2 and 3 (sign mask) run on the vector kernels only: a mask byte covers 8 consecutive elements,
// so C (NHWC) or W (NCHW) must be a multiple of 8 and k one of 1, 2, 4, 8.
template <typename T, int MODE>
ac_status launch_typed(const Dims& d, const T* x, T* z, T* y, unsigned char* mask, cudaStream_t st) {
    constexpr int VW = VecTraits<T>::VW;
    const long long zt = d.z_elems();
    if (zt >= (1ll << 31) * 256) return AC_ERR_UNSUPPORTED;
    const bool square = d.kh == d.kw;
    const bool pow2k = square && (d.k == 2 || d.k == 4 || d.k == 8);
    if (square && d.k == 1 && d.x_elems() % (MODE >= 2 ? 8 : VW) == 0) {
        // a copy (or a plain ReLU): treat the tensor as one row of 16-byte vectors
        const long long nv = d.x_elems() / VW;
        if (nv < (1ll << 31))
            return launch_nhwc_vec<T, MODE>(x, z, y, mask, 1, 1, (int)nv, 1, 1, 1, 1, (int)nv, st);
    }
    if (d.layout == AC_NHWC && d.Ci % (MODE >= 2 ? 8 : VW) == 0) {
        const ac_status st_ =
            launch_nhwc_vec<T, MODE>(x, z, y, mask, d.N, d.H, d.W, d.Ci / VW, d.kh, d.kw, d.Hp, d.Wp, st);
        if (st_ != AC_ERR_UNSUPPORTED) return st_;
    }
    if (d.layout == AC_NCHW && pow2k && d.W % (MODE >= 2 ? 8 : VW) == 0 && d.W % d.k == 0 &&
        (VW % d.k == 0 || d.k == 2 * VW)) {
        const long long total = (long long)d.N * d.Ci * d.Hp * (d.W / VW);
        if (d.k == 2) launch_nchw_vec<T, 2, MODE>(d, x, z, y, mask, total, st);
        else if (d.k == 4) launch_nchw_vec<T, 4, MODE>(d, x, z, y, mask, total, st);
        else launch_nchw_vec<T, 8, MODE>(d, x, z, y, mask, total, st);
    } else {
        if (MODE >= 2) return AC_ERR_UNSUPPORTED;
        if (const int rb = rows_per_block<T>(d)) {
            const long long out_el = (long long)d.Wp * d.Ci;
            const int vec_out = (out_el % VW == 0) ? 1 : 0;     // then every pooled row starts 16-byte aligned
            const size_t smem = (size_t)rb * (d.kh * (size_t)d.W * d.Ci + out_el) * sizeof(T);
            dim3 grid((unsigned)((d.Hp + rb - 1) / rb), (unsigned)d.N);
            const bool k2 = d.kh == 2 && d.kw == 2, c3 = d.Ci == 3;
            if (c3 && k2)
                compress_nhwc_rows<T, MODE != 0, 3, 2><<<grid, 256, smem, st>>>(x, z, y, d.Ci, d.H, d.W, d.kh, d.kw, d.Hp,
                                                                                d.Wp, rb, vec_out);
            else if (c3)
                compress_nhwc_rows<T, MODE != 0, 3, 0><<<grid, 256, smem, st>>>(x, z, y, d.Ci, d.H, d.W, d.kh, d.kw, d.Hp,
                                                                                d.Wp, rb, vec_out);
            else if (k2)
                compress_nhwc_rows<T, MODE != 0, 0, 2><<<grid, 256, smem, st>>>(x, z, y, d.Ci, d.H, d.W, d.kh, d.kw, d.Hp,
                                                                                d.Wp, rb, vec_out);
            else
                compress_nhwc_rows<T, MODE != 0, 0, 0><<<grid, 256, smem, st>>>(x, z, y, d.Ci, d.H, d.W, d.kh, d.kw, d.Hp,
                                                                                d.Wp, rb, vec_out);
            AC_CUDA_TRY(cudaGetLastError());
            return AC_OK;
        }
        compress_generic<T, MODE != 0><<<blocks_for(zt), 256, 0, st>>>(
            x, z, y, d.Ci, d.H, d.W, d.kh, d.kw, d.Hp, d.Wp, d.layout == AC_NHWC, zt);
    }
    AC_CUDA_TRY(cudaGetLastError());
    return AC_OK;
}

}  // namespace

ac_status launch_compress(const Dims& d, const void* x, void* z, void* y_out, cudaStream_t st) {
    if (d.dtype == AC_F32) {
        return y_out ? launch_typed<float, 1>(d, (const float*)x, (float*)z, (float*)y_out, nullptr, st)
                     : launch_typed<float, 0>(d, (const float*)x, (float*)z, nullptr, nullptr, st);
    }
    using B = __nv_bfloat16;
    return y_out ? launch_typed<B, 1>(d, (const B*)x, (B*)z, (B*)y_out, nullptr, st)
                 : launch_typed<B, 0>(d, (const B*)x, (B*)z, nullptr, nullptr, st);
}

ac_status launch_compress_mask(const Dims& d, const void* a, void* z, void* mask, cudaStream_t st) {
    if (d.x_elems() % 8 != 0) return AC_ERR_UNSUPPORTED;
    if (d.dtype == AC_F32)
        return launch_typed<float, 2>(d, (const float*)a, (float*)z, nullptr, (unsigned char*)mask, st);
    using B = __nv_bfloat16;
    return launch_typed<B, 2>(d, (const B*)a, (B*)z, nullptr, (unsigned char*)mask, st);
}

// the same, also storing Y = max(A, 0) (y may be a)
ac_status launch_compress_mask_y(const Dims& d, const void* a, void* y, void* z, void* mask, cudaStream_t st) {
    if (d.x_elems() % 8 != 0) return AC_ERR_UNSUPPORTED;
    if (d.dtype == AC_F32)
        return launch_typed<float, 3>(d, (const float*)a, (float*)z, (float*)y, (unsigned char*)mask, st);
    using B = __nv_bfloat16;
    return launch_typed<B, 3>(d, (const B*)a, (B*)z, (B*)y, (unsigned char*)mask, st);
}

// ReLU backward from the sign mask: dx[i] = bit i of the mask ? dy[i] : 0, eight elements (one mask byte) per thread.
namespace {
template <typename T>
__global__ void __launch_bounds__(256)
relu_mask_backward_kernel(const unsigned char* __restrict__ mask, const T* dy, T* dx, long long groups) {
    constexpr int V = 16 / (int)sizeof(T);      // elements per 16-byte vector
    const long long g = (long long)blockIdx.x * 256 + threadIdx.x;
    if (g >= groups) return;
    const unsigned int m = mask[g];
    const uint4* src = reinterpret_cast<const uint4*>(dy + g * 8);
    uint4* dst = reinterpret_cast<uint4*>(dx + g * 8);
#pragma unroll
    for (int v = 0; v < 8 / V; ++v) {
        uint4 q = src[v];
        uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (sizeof(T) == 4) {
                if (!((m >> (v * 4 + j)) & 1u)) w[j] = 0u;
            } else {
                const unsigned int b = m >> (v * 8 + 2 * j);
                w[j] &= ((b & 1u) ? 0x0000ffffu : 0u) | ((b & 2u) ? 0xffff0000u : 0u);
            }
        }
        dst[v] = make_uint4(w[0], w[1], w[2], w[3]);
    }
}
}  // namespace

ac_status launch_relu_mask_backward(const Dims& d, const void* mask, const void* dy, void* dx, cudaStream_t st) {
    const long long n = d.x_elems();
    if (n % 8 != 0) return AC_ERR_UNSUPPORTED;
    const long long groups = n / 8, blocks = (groups + 255) / 256;
    if (blocks >= (1ll << 31)) return AC_ERR_UNSUPPORTED;
    if (d.dtype == AC_F32)
        relu_mask_backward_kernel<float><<<(unsigned)blocks, 256, 0, st>>>(
            static_cast<const unsigned char*>(mask), static_cast<const float*>(dy), static_cast<float*>(dx), groups);
    else
        relu_mask_backward_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, 0, st>>>(
            static_cast<const unsigned char*>(mask), static_cast<const __nv_bfloat16*>(dy),
            static_cast<__nv_bfloat16*>(dx), groups);
    AC_CUDA_TRY(cudaGetLastError());
    return AC_OK;
}

}  // namespace ac
