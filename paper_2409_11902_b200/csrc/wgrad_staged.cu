// Problems the TMA-fed tcgen05 kernel cannot read directly, brought to it by one pass over each
// operand ("staging") into the workspace:
//
//  * fp32 inputs. The paper's networks train in fp32; a single bf16 or TF32 product cannot meet an
//    fp32 weight gradient to 1e-5, so each fp32 value is written as the sum of three bf16 terms,
//    x = h + m + l (h = bf16(x), m = bf16(x - h), l = bf16(x - h - m): 24 bits of significand between
//    them), and Z * dY is expanded into the six partial products whose weight is at least 2^-16,
//
//        Z * dY  ~  Zh*Gh + Zh*Gm + Zm*Gh + Zh*Gl + Zl*Gh + Zm*Gm       (dropped terms: 2^-24 and less)
//
//    all accumulated in fp32. A weight gradient is a sum over images, so the six products are simply
//    six times as many images for the bf16 kernel:
//
//        Z'  = [ Zh | Zm | Zh | Zl | Zm | Zh ]        dY' = [ Gm | Gh | Gl | Gh | Gm | Gh ]
//
//    (each block N images, bf16; the leading product Zh*Gh last), and the kernel runs unchanged with
//    N' = 6 N. When the accumulation chains of that launch would need to be cut often (see
//    kMaxChainF32), the five small products (5 N images, sums 2^-8 of the result and less, no bound
//    needed) and the leading one (N images) are run as two launches and added. Against the fp64
//    definition the relative Frobenius error is 7e-7 .. 2e-6 (fp32-ALU path: 3e-7 .. 5e-7, at a
//    fifth to a tenth of the speed).
//
//  * NCHW inputs (either dtype). The kernel's tap shift needs channels innermost, so the staging
//    pass also transposes each image from [C][H*W] to [H*W][C]; the kernel then produces dW as
//    [C_out][R][S][C_in] in the workspace and a last small pass permutes it to [C_out][C_in][R][S].
//
//  * Few input channels (the 3-channel stem convolution; bf16 NHWC). The kernel's unit is a 64-channel
//    vector per cell, which three channels cannot fill. Here the staging pass gathers, for every output
//    position, the inflated and zero-padded values all its taps read into one row of a matrix
//    G[position][(tap, channel)], padded to a multiple of 64 columns; the weight gradient is then the
//    1x1 problem dW'[co][column] = sum over positions of dY[position][co] * G[position][column] on the
//    output map, which the kernel takes as it is, and a last small pass copies the columns to dW.
//    When both strides are multiples of k and k divides H and W, output (ho, wo) reads the pooled
//    element Z[ho*s_h/k + u][wo*s_w/k + v] with u = floor((r - p_h)/k), v = floor((s - p_w)/k) for
//    EVERY position, so taps with equal (u, v) have equal columns: G then keeps one column per distinct
//    (u, v, channel) (7x7, stride 2, pad 3, k = 2: 16 shifts instead of 49 taps; 48 columns instead of
//    147, a third of the bytes written and read) and the last pass copies each column to all its taps.
//
//  * Small odd maps with padding (3x3 on 7x7 at k = 2; bf16 NHWC). The kernel reads Z directly here too, but
//    pays for it: every output class multiplies a whole tile of Z cells (its halo included) into every tap,
//    a pooled row or column that covers a partial block has to be kept in up to four differently zeroed
//    copies, and on a 4x4 grid of cells the halo and the rounding of a K-tile to 16 cells outweigh what the
//    compression saves (128 cell products per image and tap where the inflated 7x7 map needs 64). When the
//    kernel's cost model says so, the staging pass writes the inflated map Xt (a few MB for such layers) and
//    the kernel runs on it with k = 1. The same is done for large odd maps with padding whose tile copies do
//    not fit the shared memory at all.
#include "ac_common.h"
#include "tc_units.h"

namespace ac {
namespace {

// Xt[n][h][w][c] = Z[n][h / kh][w / kw][c] for h < H, w < W, bf16 NHWC, eight channels (16 bytes) per thread.
// With (H, W) the pooled size of a smaller block k' and kh = kw = k / k' this is Z re-blocked to k'.
__global__ void __launch_bounds__(256)
inflate_nhwc_kernel(const uint4* __restrict__ z, uint4* __restrict__ xt, int H, int W, int Hp, int Wp, int C8, int kh,
                    int kw, long long total) {
    const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
    if (i >= total) return;
    const int c = (int)(i % C8);
    long long r = i / C8;
    const int w = (int)(r % W);
    r /= W;
    const int h = (int)(r % H);
    const long long n = r / H;
    xt[i] = __ldg(z + ((n * Hp + h / kh) * Wp + w / kw) * C8 + c);
}

__device__ __forceinline__ uint32_t pack_bf2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// x = h + m + l with h, m, l representable in bf16 (l is rounded when it is packed)
__device__ __forceinline__ void split3(float x, float& h, float& m, float& l) {
    h = __bfloat162float(__float2bfloat16_rn(x));
    const float r1 = x - h;                       // exact: h shares x's leading bits
    m = __bfloat162float(__float2bfloat16_rn(r1));
    l = r1 - m;                                   // exact
}

// Which of (h, m, l) goes to block b of the staged tensor: ROLE 0 is Z', ROLE 1 is dY'.
template <int ROLE>
__device__ __forceinline__ int term_of_block(int b) {
    // Z': h m h l m h      dY': m h l h m h
    return ROLE == 0 ? ((0x012010 >> (4 * b)) & 3) : ((0x010201 >> (4 * b)) & 3);
}

// fp32 NHWC -> six bf16 blocks. One thread splits 8 consecutive values and stores three 16-byte
// vectors, each into the blocks that ROLE assigns to it.
template <int ROLE>
__global__ void __launch_bounds__(256)
split3_kernel(const float4* __restrict__ src, uint4* __restrict__ dst, long long n8) {
    const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
    if (i >= n8) return;
    const float4 a = __ldcs(src + 2 * i), b = __ldcs(src + 2 * i + 1);
    const float x[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    float t[3][8];
#pragma unroll
    for (int j = 0; j < 8; ++j) split3(x[j], t[0][j], t[1][j], t[2][j]);
    uint4 v[3];
#pragma unroll
    for (int q = 0; q < 3; ++q)
        v[q] = make_uint4(pack_bf2(t[q][0], t[q][1]), pack_bf2(t[q][2], t[q][3]), pack_bf2(t[q][4], t[q][5]),
                          pack_bf2(t[q][6], t[q][7]));
#pragma unroll
    for (int blk = 0; blk < 6; ++blk) dst[blk * n8 + i] = v[term_of_block<ROLE>(blk)];
}

__device__ __forceinline__ float load_f(const float* p) { return __ldcs(p); }
__device__ __forceinline__ float load_f(const __nv_bfloat16* p) { return __bfloat162float(*p); }

// NCHW -> NHWC (bf16), one 64-channel x 32-position tile per block of (32, 8) threads; with SPLIT the
// source is fp32 and the three terms go to the six blocks as above. grid = (ceil(P/32), C/64, N).
template <typename TIN, bool SPLIT, int ROLE>
__global__ void __launch_bounds__(256)
to_nhwc_kernel(const TIN* __restrict__ src, uint32_t* __restrict__ dst, int C, int P, long long block_words) {
    __shared__ float tile[64][33];
    const int tx = threadIdx.x, ty = threadIdx.y;
    const int p0 = blockIdx.x * 32, c0 = blockIdx.y * 64;
    const long long n = blockIdx.z;
    const TIN* s = src + (n * C + c0) * (long long)P;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int c = ty + 8 * j, p = p0 + tx;
        tile[c][tx] = p < P ? load_f(s + (long long)c * P + p) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int pl = ty + 8 * j, p = p0 + pl;
        if (p >= P) continue;
        const float x0 = tile[2 * tx][pl], x1 = tile[2 * tx + 1][pl];
        const long long w = ((n * P + p) * (long long)C + c0) / 2 + tx;     // 32-bit word = two channels
        if (!SPLIT) {
            dst[w] = pack_bf2(x0, x1);
        } else {
            float t0[3], t1[3];
            split3(x0, t0[0], t0[1], t0[2]);
            split3(x1, t1[0], t1[1], t1[2]);
#pragma unroll
            for (int blk = 0; blk < 6; ++blk) {
                const int q = term_of_block<ROLE>(blk);
                dst[blk * block_words + w] = pack_bf2(t0[q], t1[q]);
            }
        }
    }
}

// The same transposition with 16-byte accesses on both sides, for maps whose H*W is a multiple of the
// load vector (8 bf16 or 4 fp32 positions): a 64-channel x 64-position tile per block of 256 threads;
// loads run along the positions of a channel, stores along 8 channels of a position (the 8 threads of
// a position write 128 contiguous bytes). grid = (ceil(P/64), C/64, N).
template <typename TIN, bool SPLIT, int ROLE>
__global__ void __launch_bounds__(256)
to_nhwc_vec_kernel(const TIN* __restrict__ src, uint4* __restrict__ dst, int C, int P, long long block_vecs) {
    constexpr int VL = 16 / (int)sizeof(TIN);          // positions per 16-byte load
    constexpr int LPR = 64 / VL;                        // loads per tile row
    __shared__ float tile[64][65];
    const int t = threadIdx.x;
    const int p0 = blockIdx.x * 64, c0 = blockIdx.y * 64;
    const long long n = blockIdx.z;
    const TIN* s = src + (n * C + c0) * (long long)P;
#pragma unroll
    for (int pass = 0; pass < 64 * LPR / 256; ++pass) {
        const int idx = pass * 256 + t, c = idx / LPR, pv = (idx - c * LPR) * VL;
        float f[VL];
        if (p0 + pv < P) {
            const uint4 raw = __ldcs(reinterpret_cast<const uint4*>(s + (long long)c * P + p0 + pv));
            if (sizeof(TIN) == 4) {
                f[0] = __uint_as_float(raw.x); f[1] = __uint_as_float(raw.y);
                f[2 % VL] = __uint_as_float(raw.z); f[3 % VL] = __uint_as_float(raw.w);
            } else {
                const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    f[(2 * j) % VL] = __uint_as_float(w[j] << 16);
                    f[(2 * j + 1) % VL] = __uint_as_float(w[j] & 0xffff0000u);
                }
            }
        } else {
#pragma unroll
            for (int j = 0; j < VL; ++j) f[j] = 0.f;
        }
#pragma unroll
        for (int j = 0; j < VL; ++j) tile[c][pv + j] = f[j];
    }
    __syncthreads();
#pragma unroll
    for (int pass = 0; pass < 2; ++pass) {
        const int idx = pass * 256 + t, pl = idx / 8, c8 = idx - pl * 8, p = p0 + pl;
        if (p >= P) continue;
        float x[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) x[j] = tile[c8 * 8 + j][pl];
        const long long v = ((n * P + p) * (long long)C + c0) / 8 + c8;      // 16-byte vector = 8 channels
        if (!SPLIT) {
            dst[v] = make_uint4(pack_bf2(x[0], x[1]), pack_bf2(x[2], x[3]), pack_bf2(x[4], x[5]), pack_bf2(x[6], x[7]));
        } else {
            float tm[3][8];
#pragma unroll
            for (int j = 0; j < 8; ++j) split3(x[j], tm[0][j], tm[1][j], tm[2][j]);
            uint4 o[3];
#pragma unroll
            for (int q = 0; q < 3; ++q)
                o[q] = make_uint4(pack_bf2(tm[q][0], tm[q][1]), pack_bf2(tm[q][2], tm[q][3]),
                                  pack_bf2(tm[q][4], tm[q][5]), pack_bf2(tm[q][6], tm[q][7]));
#pragma unroll
            for (int blk = 0; blk < 6; ++blk) dst[blk * block_vecs + v] = o[term_of_block<ROLE>(blk)];
        }
    }
}

// dW [Co][RS][Ci] -> [Co][Ci][RS]
__global__ void __launch_bounds__(256)
permute_dw_kernel(const float* __restrict__ src, float* __restrict__ dst, int Ci, int RS, long long total) {
    const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
    if (i >= total) return;
    const int t = (int)(i % RS);
    const long long r = i / RS;
    const int ci = (int)(r % Ci);
    const long long co = r / Ci;
    dst[i] = src[(co * RS + t) * Ci + ci];
}

// ---- few input channels: gathered operand ------------------------------------------------------
struct GatherParams {
    int Ci, H, W, Hp, Wp, Ho, Wo, k;
    int kshift;         // log2 k if k is a power of two, else -1
    int sh, sw, ph, pw;
    int collapsed;      // 1: one column per distinct Z shift (u, v); 0: one per tap (r, s)
    int mh, mw;         // collapsed: Z rows / columns per output row / column (s_h / k, s_w / k)
    int u0, v0;         // collapsed: first shift
    int na, nb;         // rows and columns of shifts (collapsed: nU, nV) or taps (R, S)
    int cols, Mp;       // valid columns (shifts or taps, times C_in), row length of G (multiple of 64)
    int rows;           // N * H_o output rows
    int rows_per_block;
};

// G[position][column], eight columns (one 16-byte vector) per thread, a block per `rows_per_block`
// output rows. Z is read element by element (it is k^2 times smaller than what is written and stays
// in L2); consecutive threads write consecutive vectors. Positions all of whose taps fall inside
// the map (most of them) skip the bounds checks.
__global__ void __launch_bounds__(256)
gather_kernel(const unsigned short* __restrict__ z, uint4* __restrict__ g, const GatherParams p) {
    __shared__ int tab_ab[256];     // column -> a | b << 8, or -1 behind the last column
    __shared__ int tab_off[256];    // column -> offset in Z elements from the position's first element
    for (int j = threadIdx.x; j < p.Mp; j += 256) {
        int e = -1, off = 0;
        if (j < p.cols) {
            const int t = j / p.Ci, ci = j - t * p.Ci, a = t / p.nb, b = t - a * p.nb;
            e = a | (b << 8);
            off = p.collapsed ? (a * p.Wp + b) * p.Ci + ci : ci;
        }
        tab_ab[j] = e;
        tab_off[j] = off;
    }
    __syncthreads();
    const int G = p.Mp / 8, per_row = p.Wo * G;
    const int row0 = blockIdx.x * p.rows_per_block;
    const int nrows = min(p.rows_per_block, p.rows - row0);
    for (int v = threadIdx.x; v < nrows * per_row; v += 256) {
        const int r = v / per_row, rem = v - r * per_row, wo = rem / G, j0 = (rem - wo * G) * 8;
        const int row = row0 + r, n = row / p.Ho, ho = row - n * p.Ho;
        const unsigned short* zn = z + (long long)n * p.Hp * p.Wp * p.Ci;
        const int rb = p.collapsed ? ho * p.mh + p.u0 : ho * p.sh - p.ph;
        const int cb = p.collapsed ? wo * p.mw + p.v0 : wo * p.sw - p.pw;
        unsigned short val[8];
        if (p.collapsed) {
            const unsigned short* zb = zn + ((long long)rb * p.Wp + cb) * p.Ci;
            if (rb >= 0 && rb + p.na <= p.Hp && cb >= 0 && cb + p.nb <= p.Wp) {
#pragma unroll
                for (int q = 0; q < 8; ++q) val[q] = tab_ab[j0 + q] >= 0 ? __ldg(zb + tab_off[j0 + q]) : 0;
            } else {
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const int e = tab_ab[j0 + q];
                    const bool in = e >= 0 && (unsigned)(rb + (e & 255)) < (unsigned)p.Hp &&
                                    (unsigned)(cb + (e >> 8)) < (unsigned)p.Wp;
                    val[q] = in ? __ldg(zb + tab_off[j0 + q]) : 0;
                }
            }
        } else {
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const int e = tab_ab[j0 + q];
                int x = rb + (e & 255), y = cb + (e >> 8);      // coordinates of the inflated map
                const bool in = e >= 0 && (unsigned)x < (unsigned)p.H && (unsigned)y < (unsigned)p.W;
                if (p.kshift >= 0) { x >>= p.kshift; y >>= p.kshift; } else { x /= p.k; y /= p.k; }
                val[q] = in ? __ldg(zn + ((long long)x * p.Wp + y) * p.Ci + tab_off[j0 + q]) : 0;
            }
        }
        g[((long long)row * p.Wo + wo) * G + (j0 >> 3)] =
            make_uint4(val[0] | (uint32_t)val[1] << 16, val[2] | (uint32_t)val[3] << 16,
                       val[4] | (uint32_t)val[5] << 16, val[6] | (uint32_t)val[7] << 16);
    }
}

// The same matrix for the collapsed form, built from shared memory: the `na` rows of Z that one output
// row reads are copied in once (coalesced, zeros where the row or column lies outside Z), and every
// 16-byte vector of G is assembled from them, so that global memory sees Z once per output row and
// the eight element reads per vector are shared-memory reads.
constexpr int kGatherRowsSmemMax = 40 * 1024;
constexpr int kGatherRowGroup = 4;      // output rows built per round from one set of Z rows

__global__ void __launch_bounds__(256)
gather_rows_kernel(const unsigned short* __restrict__ z, uint4* __restrict__ g, const GatherParams p) {
    extern __shared__ unsigned short zs[];      // [(kGatherRowGroup - 1) * mh + na][span]
    const int span = ((p.Wo - 1) * p.mw + p.nb) * p.Ci, row_elems = p.Wp * p.Ci;
    // The block has a multiple of G = Mp / 8 threads, so a thread builds the same eight columns for
    // every position it visits: their offsets in zs (from the position's first element) stay in registers.
    const int G = p.Mp / 8, T = blockDim.x, wo_step = T / G;
    const int wo_first = threadIdx.x / G, j0 = (threadIdx.x - wo_first * G) * 8;
    int off[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const int j = j0 + q;
        off[q] = -1;
        if (j < p.cols) {
            const int t = j / p.Ci, ci = j - t * p.Ci, a = t / p.nb, b = t - a * p.nb;
            off[q] = a * span + b * p.Ci + ci;
        }
    }
    const int row0 = blockIdx.x * p.rows_per_block;
    const int row1 = min(row0 + p.rows_per_block, p.rows);
    for (int row = row0; row < row1;) {
        // up to kGatherRowGroup output rows of one image per round: they share most of their Z rows
        const int n = row / p.Ho, ho = row - n * p.Ho, rb = ho * p.mh + p.u0;
        const int ng = min(min(kGatherRowGroup, row1 - row), p.Ho - ho);
        const int nz = (ng - 1) * p.mh + p.na;
        if (row > row0) __syncthreads();      // the rows before these have been read
        for (int a = 0; a < nz; ++a) {
            const int zr = rb + a;
            const bool row_in = zr >= 0 && zr < p.Hp;
            const unsigned short* src = z + ((long long)n * p.Hp + zr) * row_elems;
            for (int x = threadIdx.x; x < span; x += T) {
                const int sx = x + p.v0 * p.Ci;      // element of the Z row
                zs[a * span + x] = row_in && sx >= 0 && sx < row_elems ? __ldg(src + sx) : (unsigned short)0;
            }
        }
        __syncthreads();
        for (int r = 0; r < ng; ++r) {
            uint4* grow = g + (long long)(row + r) * p.Wo * G + (j0 >> 3);
            const unsigned short* zrow = zs + r * p.mh * span;
            for (int wo = wo_first; wo < p.Wo; wo += wo_step) {
                const unsigned short* zb = zrow + wo * p.mw * p.Ci;
                unsigned short val[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) val[q] = off[q] >= 0 ? zb[off[q]] : (unsigned short)0;
                grow[wo * G] = make_uint4(val[0] | (uint32_t)val[1] << 16, val[2] | (uint32_t)val[3] << 16,
                                          val[4] | (uint32_t)val[5] << 16, val[6] | (uint32_t)val[7] << 16);
            }
        }
        row += ng;
    }
}

// dW[co][r][s][ci] = dW'[co][column of (r, s, ci)]
__global__ void __launch_bounds__(256)
scatter_columns_kernel(const float* __restrict__ src, float* __restrict__ dw, const GatherParams p, int R, int S,
                       long long total) {
    const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
    if (i >= total) return;
    const int row = R * S * p.Ci;
    const long long co = i / row;
    int col = (int)(i - co * row);
    if (p.collapsed) {
        const int t = col / p.Ci, ci = col - t * p.Ci, r = t / S, s = t - r * S;
        const int iu = floor_div_i(r - p.ph, p.k) - p.u0, iv = floor_div_i(s - p.pw, p.k) - p.v0;
        col = (iu * p.nb + iv) * p.Ci + ci;
    }
    dw[i] = src[co * p.Mp + col];
}

struct GatherGeom {
    bool ok;
    GatherParams p;
    Dims in;       // the 1x1 problem on the output map
};

GatherGeom gather_geom(const Dims& d) {
    GatherGeom g{};
    if (d.dtype != AC_BF16 || d.layout != AC_NHWC) return g;
    if (d.Ci >= 64 || d.Co % 64 != 0) return g;
    if (d.R > 255 || d.S > 255) return g;
    if (d.kh != d.kw) return g;      // the gather's index map knows square pooling blocks only
    GatherParams& p = g.p;
    p.Ci = d.Ci; p.H = d.H; p.W = d.W; p.Hp = d.Hp; p.Wp = d.Wp; p.Ho = d.Ho; p.Wo = d.Wo; p.k = d.k;
    p.sh = d.sh; p.sw = d.sw; p.ph = d.ph; p.pw = d.pw;
    p.collapsed = d.k > 1 && d.sh % d.k == 0 && d.sw % d.k == 0 && d.H % d.k == 0 && d.W % d.k == 0;
    p.kshift = -1;
    for (int b = 0; b < 30; ++b) if (d.k == (1 << b)) p.kshift = b;
    p.na = d.R;
    p.nb = d.S;
    if (p.collapsed) {
        p.mh = d.sh / d.k; p.mw = d.sw / d.k;
        p.u0 = floor_div_i(-d.ph, d.k); p.v0 = floor_div_i(-d.pw, d.k);
        p.na = floor_div_i(d.R - 1 - d.ph, d.k) - p.u0 + 1;
        p.nb = floor_div_i(d.S - 1 - d.pw, d.k) - p.v0 + 1;
    }
    const long long cols = (long long)p.na * p.nb * d.Ci;
    if (cols > 256) return g;
    p.cols = (int)cols;
    p.Mp = (p.cols + 63) / 64 * 64;
    if (d.K() * p.Mp >= (1ll << 40) || (long long)d.N * d.Ho >= (1ll << 31)) return g;
    if ((long long)d.Hp * d.Wp * d.Ci >= (1ll << 31)) return g;      // offsets within one image are 32-bit
    p.rows = d.N * d.Ho;
    // about 1024 vectors (four per thread) per block, whole output rows
    const long long per_row = (long long)d.Wo * (p.Mp / 8);
    if (per_row >= (1ll << 24)) return g;
    p.rows_per_block = (int)(per_row >= 1024 ? 1 : (1024 + per_row - 1) / per_row);
    Dims in = d;
    in.Ci = p.Mp;
    in.H = in.Hp = d.Ho;
    in.W = in.Wp = d.Wo;
    in.R = in.S = 1;
    in.sh = in.sw = 1;
    in.ph = in.pw = 0;
    in.k = in.kh = in.kw = 1;
    g.in = in;
    g.ok = tc2_supported(in, nullptr);
    return g;
}

inline size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }

// fp32 results: at most this many MMA instructions add into an accumulator before the kernel
// writes it out (adding, in round-to-nearest fp32, to what it wrote before) and starts it afresh.
// The tensor core adds into its fp32 accumulator with truncation; on pooled ReLU(N(0,1)) x
// N(0, 1e-4) data the bias is about 1.8e-8 of the final sum per instruction of the chain. Measured
// relative Frobenius error / time, batch 64, 128 channels, 28 x 28 (batch 32, 64 x 64):
//     no bound  6.6e-6 / 127 us  (1.8e-5 / 245 us: over the fp32 bound)
//     256       3.3e-6 / 133 us  (3.2e-6 / 292 us)
//     192       2.1e-6 / 143 us  (2.4e-6 / 306 us)
//     128       1.6e-6 / 151 us  (1.3e-6 / 332 us)
constexpr int kMaxChainF32 = 128;

// The bf16 NHWC problem(s) the staged operands amount to: `a` is the first launch; `b.N > 0` means
// a second launch on the last block alone (the leading product), whose result is added to the first's.
struct Inner {
    Dims a, b;
};

// The dense problem on the inflated map, when the cost model expects it to beat the kernel's own reading of Z
// by a margin (the inflation pass is charged at the copy bandwidth plus a launch), or when the kernel cannot
// read Z itself (large odd maps with padding, whose four tile copies do not fit the shared memory).
bool inflate_problem(const Dims& d, Dims* out) {
    if (d.dtype != AC_BF16 || d.layout != AC_NHWC || (d.kh == 1 && d.kw == 1) || d.max_chain != 0) return false;
    int copies = 0;
    const double direct = tc2_cost_cycles(d, &copies);      // negative: the kernel cannot read this Z at all
    // Candidates: the fully inflated map (k' = 1) where the tile needs several copies or cannot be read at all, and,
    // for square blocks of 4 and more, Z re-blocked to a smaller block k' = k/2, k/4, ... >= 2 (the same inflated
    // map, see reblocked_dims): sixteen or sixty-four output classes cost more per K-tile than four, and 64-channel
    // layers pair their taps only when every class agrees on the shifts.
    double best = -1.0;
    Dims best_in{};
    for (int k2 = d.kh == d.kw ? d.k / 2 : 1; k2 >= 1; k2 /= 2) {
        if (k2 > 1 && (d.k % k2 != 0 || d.k < 4)) continue;
        if (k2 == 1 && direct >= 0.0 && copies < 2) break;
        Dims in = d;
        in.k = in.kh = in.kw = k2;
        in.Hp = (d.H + k2 - 1) / k2;
        in.Wp = (d.W + k2 - 1) / k2;
        if (in.z_elems() >= (1ll << 40) || (in.z_elems() / 8 + 255) / 256 >= (1ll << 31)) continue;
        int c2 = 0;
        const double inner = tc2_cost_cycles(in, &c2);
        if (inner < 0.0) continue;
        // the pass: a launch, and its bytes at ~3.4 KB per cycle
        const double cost = inner + 6000.0 + 2.0 * (double)(d.z_elems() + in.z_elems()) * 2.9e-4;
        if (best < 0.0 || cost < best) { best = cost; best_in = in; }
        if (k2 == 1) break;
    }
    if (best < 0.0) return false;
    if (direct >= 0.0 && best >= 0.85 * direct) return false;
    *out = best_in;
    return true;
}

bool inner_problem(const Dims& d, Inner* out) {
    const bool split = d.dtype == AC_F32, transpose = d.layout == AC_NCHW;
    if (!split && !transpose) {
        // the kernel reads these itself, and does unless the inflated map is the faster way
        if (!inflate_problem(d, &out->a)) return false;
        out->b = out->a;
        out->b.N = 0;
        return true;
    }
    if (transpose) {
        if (d.Ci % 64 != 0 || d.Co % 64 != 0 || d.N > 65535) return false;
        if ((long long)d.Hp * d.Wp >= (1ll << 31) || (long long)d.Ho * d.Wo >= (1ll << 31)) return false;
    } else if (d.z_elems() % 8 != 0 || d.dy_elems() % 8 != 0) {
        return false;
    }
    const long long n_in = (long long)d.N * (split ? 6 : 1);
    if (n_in >= (1ll << 31)) return false;
    Dims in = d;
    in.N = (int)n_in;
    in.dtype = AC_BF16;
    in.layout = AC_NHWC;
    in.elt = 2;
    const long long lim = 1ll << 40;
    if (in.z_elems() >= lim || in.dy_elems() >= lim) return false;
    out->a = in;
    out->b = in;
    out->b.N = 0;
    if (!split) return tc2_supported(in, nullptr);
    // one launch with bounded chains, or two: each cut of the chains costs a read-add-store of the
    // accumulators (about 6 us), a second launch about 20 us of fixed work
    Dims one = in, small = in, lead = in;
    one.max_chain = kMaxChainF32;
    small.N = d.N * 5;
    lead.N = d.N;
    lead.max_chain = kMaxChainF32;
    if (!tc2_supported(one, nullptr)) return false;
    out->a = one;
    if (tc2_supported(small, nullptr) && tc2_supported(lead, nullptr)) {
        const int cuts_one = (tc2_chain_length(one) + kMaxChainF32 - 1) / kMaxChainF32 - 1;
        const int cuts_lead = (tc2_chain_length(lead) + kMaxChainF32 - 1) / kMaxChainF32 - 1;
        if (6 * cuts_one > 20 + 6 * cuts_lead) {
            out->a = small;
            out->b = lead;
        }
    }
    return true;
}

template <typename TIN, bool SPLIT>
ac_status stage_nchw(const TIN* z, const TIN* dy, void* z_st, void* dy_st, const Dims& d, cudaStream_t stream) {
    const int Pz = d.Hp * d.Wp, Pg = d.Ho * d.Wo;
    constexpr int VL = 16 / (int)sizeof(TIN);
    const dim3 blk(32, 8);
    if (Pz % VL == 0)
        to_nhwc_vec_kernel<TIN, SPLIT, 0><<<dim3((Pz + 63) / 64, d.Ci / 64, d.N), 256, 0, stream>>>(
            z, static_cast<uint4*>(z_st), d.Ci, Pz, d.z_elems() / 8);
    else
        to_nhwc_kernel<TIN, SPLIT, 0><<<dim3((Pz + 31) / 32, d.Ci / 64, d.N), blk, 0, stream>>>(
            z, static_cast<uint32_t*>(z_st), d.Ci, Pz, d.z_elems() / 2);
    if (Pg % VL == 0)
        to_nhwc_vec_kernel<TIN, SPLIT, 1><<<dim3((Pg + 63) / 64, d.Co / 64, d.N), 256, 0, stream>>>(
            dy, static_cast<uint4*>(dy_st), d.Co, Pg, d.dy_elems() / 8);
    else
        to_nhwc_kernel<TIN, SPLIT, 1><<<dim3((Pg + 31) / 32, d.Co / 64, d.N), blk, 0, stream>>>(
            dy, static_cast<uint32_t*>(dy_st), d.Co, Pg, d.dy_elems() / 2);
    AC_CUDA_TRY(cudaGetLastError());
    return AC_OK;
}

}  // namespace

bool staged_supported(const Dims& d) {
    Inner in;
    return inner_problem(d, &in);
}

bool staged_inflate_preferred(const Dims& d) {
    Dims in;
    return inflate_problem(d, &in);
}

void plan_staged(const Dims& d, WgradPlan* pl) {
    Inner in;
    inner_problem(d, &in);
    plan_tc2(in.a, pl);
    if (in.b.N > 0) {
        WgradPlan pb{};
        plan_tc2(in.b, &pb);
        if (pb.bytes > pl->bytes) pl->bytes = pb.bytes;     // the launches use the partial sums' room in turn
    }
    const long long blocks = d.dtype == AC_F32 ? 6 : 1;
    const bool inflate = d.dtype == AC_BF16 && d.layout == AC_NHWC;      // Xt in place of Z, dY as it is
    pl->path = PATH_STAGED;
    pl->st_off_z = up256(pl->bytes);
    pl->st_off_dy = pl->st_off_z + up256((size_t)((inflate ? in.a.z_elems() : d.z_elems()) * blocks) * 2);
    pl->st_off_dw = pl->st_off_dy + (inflate ? 0 : up256((size_t)(d.dy_elems() * blocks) * 2));
    pl->st_off_small = pl->st_off_dw + (d.layout == AC_NCHW ? up256((size_t)d.dw_elems() * 4) : 0);
    pl->bytes = pl->st_off_small + (in.b.N > 0 ? up256((size_t)d.dw_elems() * 4) : 0);
}

void staged_plan_info(const Dims& d, ac_plan_info* info) {
    Inner in;
    inner_problem(d, &in);
    tc2_plan_info(in.a, info);
    info->tensor_core = d.dtype == AC_BF16 && d.layout == AC_NHWC ? 7 : (in.b.N > 0 ? 4 : 3);
}

ac_status launch_wgrad_staged(const Dims& d, const WgradPlan& pl, const void* z, const void* dy,
                              float* dw, void* workspace, cudaStream_t stream) {
    Inner in;
    if (!inner_problem(d, &in)) return AC_ERR_UNSUPPORTED;
    char* ws = static_cast<char*>(workspace);
    char* z_st = ws + pl.st_off_z;
    char* dy_st = ws + pl.st_off_dy;
    ac_status st = AC_OK;
    if (d.dtype == AC_BF16 && d.layout == AC_NHWC) {
        const long long total = in.a.z_elems() / 8;
        // the inner problem's Z: the inflated map itself (k' = 1) or Z re-blocked to k'
        inflate_nhwc_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(
            static_cast<const uint4*>(z), reinterpret_cast<uint4*>(z_st), in.a.Hp, in.a.Wp, d.Hp, d.Wp, d.Ci / 8,
            d.kh / in.a.kh, d.kw / in.a.kw, total);
        AC_CUDA_TRY(cudaGetLastError());
        return launch_wgrad_tc2(in.a, pl, z_st, dy, dw, workspace, stream);
    }
    if (d.layout == AC_NCHW) {
        if (d.dtype == AC_F32)
            st = stage_nchw<float, true>((const float*)z, (const float*)dy, z_st, dy_st, d, stream);
        else
            st = stage_nchw<__nv_bfloat16, false>((const __nv_bfloat16*)z, (const __nv_bfloat16*)dy, z_st, dy_st,
                                                  d, stream);
        if (st != AC_OK) return st;
    } else {
        const long long nz8 = d.z_elems() / 8, ng8 = d.dy_elems() / 8;
        if ((nz8 + 255) / 256 >= (1ll << 31) || (ng8 + 255) / 256 >= (1ll << 31)) return AC_ERR_UNSUPPORTED;
        split3_kernel<0><<<(unsigned)((nz8 + 255) / 256), 256, 0, stream>>>(
            reinterpret_cast<const float4*>(z), reinterpret_cast<uint4*>(z_st), nz8);
        split3_kernel<1><<<(unsigned)((ng8 + 255) / 256), 256, 0, stream>>>(
            reinterpret_cast<const float4*>(dy), reinterpret_cast<uint4*>(dy_st), ng8);
        AC_CUDA_TRY(cudaGetLastError());
    }
    // where the kernel's [C_out][R][S][C_in] result goes: the caller's dW, or the workspace if it
    // still has to be permuted
    float* out_nhwc = d.layout == AC_NHWC ? dw : reinterpret_cast<float*>(ws + pl.st_off_dw);
    if (in.b.N == 0) {
        st = launch_wgrad_tc2(in.a, pl, z_st, dy_st, out_nhwc, workspace, stream);
        if (st != AC_OK) return st;
    } else {
        float* small = reinterpret_cast<float*>(ws + pl.st_off_small);
        st = launch_wgrad_tc2(in.a, pl, z_st, dy_st, small, workspace, stream);
        if (st != AC_OK) return st;
        st = launch_wgrad_tc2(in.b, pl, z_st + (size_t)d.z_elems() * 5 * 2, dy_st + (size_t)d.dy_elems() * 5 * 2,
                              out_nhwc, workspace, stream, /*keep_status=*/true);
        if (st != AC_OK) return st;
        st = launch_axpby(small, 1.0f, out_nhwc, d.dw_elems(), stream);     // leading product + the rest
        if (st != AC_OK) return st;
    }
    if (d.layout == AC_NHWC) return AC_OK;
    const long long total = d.dw_elems();
    permute_dw_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(out_nhwc, dw, d.Ci, d.R * d.S, total);
    AC_CUDA_TRY(cudaGetLastError());
    return AC_OK;
}

// Few input channels with a pooling block that is a multiple of the stride (k = 4 or 8 at stride 2): the in-kernel
// form wants the stride to be a multiple of k. Z re-blocked to k' = stride, Z'[p][q] = Z[p*k'/k][q*k'/k] (the same
// inflated map: X~[h] = Z[h/k] = Z'[h/k'] when k' divides k), is a tensor of |X| / k'^2 elements that it does take.
bool reblocked_dims(const Dims& d, Dims* out) {
    if (gather_fused_supported(d)) return false;
    if (d.dtype != AC_BF16 || d.layout != AC_NHWC || d.kh != d.kw || d.sh != d.sw) return false;
    const int k2 = d.sh;
    if (k2 < 2 || k2 >= d.k || d.k % k2 != 0) return false;
    Dims r = d;
    r.k = r.kh = r.kw = k2;
    r.Hp = (d.H + k2 - 1) / k2;
    r.Wp = (d.W + k2 - 1) / k2;
    if (r.z_elems() >= (1ll << 40) || (r.z_elems() + 255) / 256 >= (1ll << 31)) return false;
    if (!gather_fused_supported(r) || ((long long)r.Wp * r.Ci) % 8 != 0) return false;
    *out = r;
    return true;
}

// eight consecutive elements of a row of Z' (a row is Wp2 * C elements, a multiple of eight: the in-kernel form asks
// for rows of whole 16-byte units) per thread: eight 2-byte reads of Z, one 16-byte store
__global__ void __launch_bounds__(256)
reblock_nhwc_kernel(const unsigned short* __restrict__ z, uint4* __restrict__ z2, int C, int Hp, int Wp,
                    int Hp2, int Wp2, int f, long long total8) {
    const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
    if (i >= total8) return;
    const int row8 = Wp2 * C / 8;
    const int e0 = (int)(i % row8) * 8;
    long long r = i / row8;
    const int p = (int)(r % Hp2);
    const long long n = r / Hp2;
    const unsigned short* src = z + ((n * Hp + p / f) * (long long)Wp) * C;
    unsigned short v[8];
    int q = e0 / C, c = e0 - q * C;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        v[j] = __ldg(src + (q / f) * C + c);
        if (++c == C) { c = 0; ++q; }
    }
    z2[i] = make_uint4(v[0] | (uint32_t)v[1] << 16, v[2] | (uint32_t)v[3] << 16, v[4] | (uint32_t)v[5] << 16,
                       v[6] | (uint32_t)v[7] << 16);
}

bool gather_supported(const Dims& d) {
    Dims r;
    return gather_fused_supported(d) || reblocked_dims(d, &r) || gather_geom(d).ok;
}

void plan_gather(const Dims& d, WgradPlan* pl) {
    if (gather_fused_supported(d)) {      // the matrix is built inside the kernel: no staged copy
        *pl = WgradPlan{};
        pl->path = PATH_GATHER;
        pl->bytes = gather_fused_workspace_bytes(d);
        return;
    }
    Dims r;
    if (reblocked_dims(d, &r)) {          // the re-blocked Z behind the in-kernel form's own workspace
        *pl = WgradPlan{};
        pl->path = PATH_GATHER;
        pl->st_off_z = up256(gather_fused_workspace_bytes(r));
        pl->bytes = pl->st_off_z + up256((size_t)r.z_elems() * 2);
        return;
    }
    const GatherGeom g = gather_geom(d);
    plan_tc2(g.in, pl);
    pl->path = PATH_GATHER;
    pl->st_off_z = up256(pl->bytes);
    pl->st_off_dy = pl->st_off_z;
    pl->st_off_dw = pl->st_off_z + up256((size_t)g.in.z_elems() * 2);
    pl->st_off_small = pl->st_off_dw;
    pl->bytes = pl->st_off_dw + up256((size_t)g.in.dw_elems() * 4);
}

void gather_plan_info(const Dims& d, ac_plan_info* info) {
    if (gather_fused_supported(d)) {
        gather_fused_plan_info(d, info);
        return;
    }
    Dims r;
    if (reblocked_dims(d, &r)) {
        gather_fused_plan_info(r, info);
        return;
    }
    const GatherGeom g = gather_geom(d);
    tc2_plan_info(g.in, info);
    info->tensor_core = 5;
}

ac_status launch_wgrad_gather(const Dims& d, const WgradPlan& pl, const void* z, const void* dy, float* dw,
                              void* workspace, cudaStream_t stream) {
    if (gather_fused_supported(d)) return launch_wgrad_gather_fused(d, z, dy, dw, workspace, stream);
    Dims r;
    if (reblocked_dims(d, &r)) {
        uint4* z2 = reinterpret_cast<uint4*>(static_cast<char*>(workspace) + pl.st_off_z);
        const long long total8 = r.z_elems() / 8;
        reblock_nhwc_kernel<<<(unsigned)((total8 + 255) / 256), 256, 0, stream>>>(
            static_cast<const unsigned short*>(z), z2, d.Ci, d.Hp, d.Wp, r.Hp, r.Wp, d.k / r.k, total8);
        AC_CUDA_TRY(cudaGetLastError());
        return launch_wgrad_gather_fused(r, z2, dy, dw, workspace, stream);
    }
    const GatherGeom g = gather_geom(d);
    if (!g.ok) return AC_ERR_UNSUPPORTED;
    char* ws = static_cast<char*>(workspace);
    uint4* gm = reinterpret_cast<uint4*>(ws + pl.st_off_z);
    float* dw_cols = reinterpret_cast<float*>(ws + pl.st_off_dw);
    GatherParams gp = g.p;
    const long long rows_smem =
        2ll * ((kGatherRowGroup - 1) * gp.mh + gp.na) * (((long long)gp.Wo - 1) * gp.mw + gp.nb) * gp.Ci;
    if (gp.collapsed && rows_smem <= kGatherRowsSmemMax) {
        // a thread works out its eight column offsets once per block: give a block about 64 vectors per
        // thread, as long as that leaves four blocks for every SM
        const long long per_row = (long long)gp.Wo * (gp.Mp / 8);
        long long rpb = (16384 + per_row - 1) / per_row;
        if (rpb > gp.rows / (4 * kNumSMs)) rpb = gp.rows / (4 * kNumSMs);
        if (rpb > gp.rows_per_block) gp.rows_per_block = (int)rpb;
        const unsigned blocks = (unsigned)((gp.rows + gp.rows_per_block - 1) / gp.rows_per_block);
        gather_rows_kernel<<<blocks, 256 / (gp.Mp / 8) * (gp.Mp / 8), (size_t)rows_smem, stream>>>(
            static_cast<const unsigned short*>(z), gm, gp);
    } else {
        const unsigned blocks = (unsigned)((gp.rows + gp.rows_per_block - 1) / gp.rows_per_block);
        gather_kernel<<<blocks, 256, 0, stream>>>(static_cast<const unsigned short*>(z), gm, gp);
    }
    AC_CUDA_TRY(cudaGetLastError());
    const ac_status st = launch_wgrad_tc2(g.in, pl, gm, dy, dw_cols, workspace, stream);
    if (st != AC_OK) return st;
    const long long total = d.dw_elems();
    scatter_columns_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(dw_cols, dw, gp, d.R, d.S, total);
    AC_CUDA_TRY(cudaGetLastError());
    return AC_OK;
}

}  // namespace ac
