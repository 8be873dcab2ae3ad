// Compressed weight gradient of a layer with few input channels (a network's first convolution),
// with the gathered operand built inside the kernel.
//
// When both strides are multiples of k and k divides H and W, output (ho, wo) reads, through tap
// (r, s), Z[ho*s_h/k + u][wo*s_w/k + v] with u = floor((r - p_h)/k), v = floor((s - p_w)/k): the
// same pooled element for every tap with the same (u, v) (Section 4's inflation makes neighbouring
// taps read one block mean). So the weight gradient is
//     dW'[co][(u, v, ci)] = sum over positions of dY[position][co] * Z[ho*m_h + u][wo*m_w + v][ci],
// one column per distinct shift (4 x 4 x 3 = 48 for a 7x7 stride-2 stem at k = 2), copied to all the
// taps that share it. wgrad_staged.cu computes this by writing the matrix G[position][column] to
// the workspace and running the TMA-fed kernel on it; for the ResNet stem at batch 256 that matrix
// is as large as dY (411 MB) and is written once and read once. Here sixteen warps build each K-tile
// of G directly in shared memory, in the 128-byte-swizzled layout the MMA reads (what TMA would have
// written), from a strip of Z rows that they keep in shared memory; G never exists in global memory.
//
// Roles: warp 0 fetches the dY tiles by TMA; sixteen warps build the G tiles (and drain the
// accumulators at the end); warp 1 issues the MMAs: D[column][co] += G^T dY, fp32 in tensor memory.
// K (the positions) is split over the CTAs; a last small kernel sums the slices in a fixed order
// and copies every column to its taps.
#include <cuda.h>

#include <cstring>

#include "ac_common.h"
#include "tc_ptx.cuh"
#include "tc_units.h"

namespace ac {
namespace {

using namespace tc;

constexpr int kGfBuilders = 512;    // a multiple of the 16-byte chunks per row of G (8 or 16): a thread's chunk never changes
constexpr int kGfStripWarp = 2 + kGfBuilders / 32;     // the last warp
// warp 0: dY tiles by TMA, warp 1: MMA + tensor memory, the builders (build, then drain), last warp: Z strips by
// TMA. Issuing a tensor copy holds a warp for several hundred cycles, so the two streams have a warp each.
constexpr int kGfThreads = 64 + kGfBuilders + 32;
constexpr int kGfSlotsA = 3;
constexpr int kGfMaxSlotsB = 4;
constexpr int kGfSlotsS = 4;        // ring of Z strips
constexpr uint32_t kGfSmemBudget = 200 * 1024;

struct GfParams {
    CUtensorMap tmB;                // dY as (Co, Wo, N*Ho)
    CUtensorMap tmZ;                // Z as (Wp*Ci/2 pairs of bf16, Hp, N), no swizzle
    int x0;                         // first strip element of a Z row (a multiple of 8, may be negative), `lead` before v0*Ci
    int lead;
    float* out;
    uint32_t* status;
    int keep_status;
    int Ci, Hp, Wp, Ho, Wo, R, S, ph, pw, k;
    int mh, mw, u0, v0, na, nb, cols, Mp;
    int RB, npos, KT, ksteps, ktiles, splits, groups, BN, nchunks, slotsB;
    int span, nz;                   // the strip of Z a K-tile reads: nz rows of span elements (span a multiple of 8)
    uint32_t a_chunk_bytes, a_slot_bytes, b_chunk_bytes, b_slot_bytes, b_box_bytes, strip_bytes, strip_box_bytes, tmem_cols;
    long long slice_elems;          // Co * Mp floats per K-slice
    long long dw_elems;
};

extern __shared__ __align__(1024) unsigned char gf_smem[];

__device__ __forceinline__ void gf_timeout(int* abort_s, uint32_t* status, uint32_t code) {
    if (atomicExch(abort_s, 1) == 0) {
        status[1] = code;
        atomicExch(&status[0], 1u);
    }
}

// 3-D tile load; coordinates innermost first. No multicast.
__device__ __forceinline__ void tma_load_3d(uint32_t dst_smem, const void* tmap, uint64_t* bar, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4, %5}], [%2];" ::"r"(dst_smem),
        "l"(reinterpret_cast<uint64_t>(tmap)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

__global__ void __launch_bounds__(kGfThreads, 1) wgrad_gather_fused_kernel(const __grid_constant__ GfParams p) {
    __shared__ uint64_t fullA[kGfSlotsA], emptyA[kGfSlotsA], fullB[kGfMaxSlotsB], emptyB[kGfMaxSlotsB], done_bar;
    __shared__ uint64_t fullS[kGfSlotsS], emptyS[kGfSlotsS];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    volatile int* abort_flag = &abort_s;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int group = blockIdx.x % p.groups, split = blockIdx.x / p.groups;
    const int co0 = group * p.BN;
    const int kt_begin = (int)((long long)p.ktiles * split / p.splits);
    const int kt_end = (int)((long long)p.ktiles * (split + 1) / p.splits);
    const uint32_t smem_base = (smem_u32(gf_smem) + 1023u) & ~1023u;
    unsigned char* smem_gen = gf_smem + (smem_base - smem_u32(gf_smem));
    const uint32_t a_base = smem_base, b_base = a_base + kGfSlotsA * p.a_slot_bytes;
    unsigned char* a_gen = smem_gen;
    unsigned char* b_gen = smem_gen + (size_t)kGfSlotsA * p.a_slot_bytes;
    const uint32_t s_base = b_base + p.slotsB * p.b_slot_bytes;      // kGfSlotsS strips
    const unsigned short* strip = reinterpret_cast<const unsigned short*>(b_gen + (size_t)p.slotsB * p.b_slot_bytes);
    const int strip_el = (int)(p.strip_bytes / 2);

    // ------------------------------------------------------------------ set-up
    if (warp == 0) {
        if (lane == 0) {
            prefetch_tmap(&p.tmB);
            prefetch_tmap(&p.tmZ);
            // a tile is full, and its strip read, once each of the builder warps has said so
            for (int s = 0; s < kGfSlotsA; ++s) { mbar_init(&fullA[s], kGfBuilders / 32); mbar_init(&emptyA[s], 1); }
            for (int s = 0; s < kGfSlotsS; ++s) { mbar_init(&fullS[s], 1); mbar_init(&emptyS[s], kGfBuilders / 32); }
            for (int s = 0; s < p.slotsB; ++s) { mbar_init(&fullB[s], 1); mbar_init(&emptyB[s], 1); }
            mbar_init(&done_bar, 1);
            abort_s = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
    } else if (warp == 1) {
        tmem_alloc(&tmem_base_s, p.tmem_cols);
    } else if (warp < kGfStripWarp) {
        // Everything the MMAs read but nobody writes later must be zero: the input tiles' cells behind
        // the last position and the padding columns of their rows, and the gradient tiles' cells
        // behind the box that TMA fills.
        const int b = tid - 64;
        const uint4 zero4 = make_uint4(0, 0, 0, 0);
        uint4* a4 = reinterpret_cast<uint4*>(a_gen);
        for (int i = b; i < (int)(kGfSlotsA * p.a_slot_bytes / 16); i += kGfBuilders) a4[i] = zero4;
        const int tail0 = p.npos * 8, tail1 = p.KT * 8;      // 16-byte units per 64-channel chunk
        for (int sc = 0; sc < p.slotsB * p.nchunks; ++sc) {
            uint4* chunk = reinterpret_cast<uint4*>(b_gen + (size_t)sc * p.b_chunk_bytes);
            for (int c = tail0 + b; c < tail1; c += kGfBuilders) chunk[c] = zero4;
        }
        fence_proxy_async_smem();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    pdl_wait();      // nothing above touched global memory
    if (blockIdx.x == 0 && tid == 0 && !p.keep_status) { p.status[0] = 0u; p.status[1] = 0u; }

    if (warp == 0) {
        // ------------------------------------------------------------ dY tiles by TMA
        for (int kt = kt_begin, i = 0; kt < kt_end; ++kt, ++i) {
            const int sb = i % p.slotsB;
            if (i >= p.slotsB) {
                const bool got = mbar_wait(&emptyB[sb], ((i / p.slotsB) & 1) ^ 1, abort_flag);
                if (!__all_sync(0xffffffffu, got)) {
                    if (lane == 0) gf_timeout(&abort_s, p.status, 0x480u + sb);
                    break;
                }
            }
            if (lane == 0) mbar_arrive_expect_tx(&fullB[sb], (uint32_t)p.nchunks * p.b_box_bytes);
            __syncwarp();
            if (lane < p.nchunks)
                tma_load_3d(b_base + sb * p.b_slot_bytes + lane * p.b_chunk_bytes, &p.tmB, &fullB[sb], co0 + 64 * lane,
                            0, kt * p.RB);
        }
    } else if (warp == kGfStripWarp) {
        // ------------------------------------------------------------ Z strips by TMA
        for (int kt = kt_begin, i = 0; kt < kt_end; ++kt, ++i) {
            // the strip of Z this K-tile reads: rows rb .. rb + nz - 1 of image n, from element x0 on; rows and
            // elements outside Z arrive as zeros (the convolution's padding)
            const int ss = i % kGfSlotsS;
            if (i >= kGfSlotsS) {
                const bool got = mbar_wait(&emptyS[ss], ((i / kGfSlotsS) & 1) ^ 1, abort_flag);
                if (!__all_sync(0xffffffffu, got)) {
                    if (lane == 0) gf_timeout(&abort_s, p.status, 0x4C0u + ss);
                    break;
                }
            }
            if (lane == 0) {
                const int row0 = kt * p.RB, n = row0 / p.Ho, ho = row0 - n * p.Ho;
                mbar_arrive_expect_tx(&fullS[ss], p.strip_box_bytes);
                tma_load_3d(s_base + ss * p.strip_bytes, &p.tmZ, &fullS[ss], p.x0 / 2, ho * p.mh + p.u0, n);
            }
            __syncwarp();
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        const uint32_t idesc = make_idesc(p.BN);
        const uint32_t hi = desc_hi(1024, 2);      // both operands MN-major, 128-byte swizzle, 8-row atoms
        const bool leader = elect_one();
        bool ok = true;
        for (int kt = kt_begin, i = 0; kt < kt_end && ok; ++kt, ++i) {
            const int sa = i % kGfSlotsA, sb = i % p.slotsB;
            bool got = mbar_wait(&fullA[sa], (i / kGfSlotsA) & 1, abort_flag);
            if (!__all_sync(0xffffffffu, got)) {
                if (leader) gf_timeout(&abort_s, p.status, 0x500u + sa);
                ok = false;
                break;
            }
            got = mbar_wait(&fullB[sb], (i / p.slotsB) & 1, abort_flag);
            if (!__all_sync(0xffffffffu, got)) {
                if (leader) gf_timeout(&abort_s, p.status, 0x580u + sb);
                ok = false;
                break;
            }
            tc_fence_after();
            uint32_t a_lo = desc_lo(a_base + sa * p.a_slot_bytes, p.a_chunk_bytes);
            uint32_t b_lo = desc_lo(b_base + sb * p.b_slot_bytes, p.b_chunk_bytes);
            for (int kk = 0; kk < p.ksteps; ++kk) {
                if (leader) mma_bf16_words(tmem_base, a_lo, hi, b_lo, hi, idesc, (i | kk) == 0 ? 0u : 1u);
                a_lo += 128;      // 16 cells x 128 bytes
                b_lo += 128;
            }
            if (leader) { mma_commit(&emptyA[sa]); mma_commit(&emptyB[sb]); }
            __syncwarp();
        }
        if (ok && leader) mma_commit(&done_bar);
        __syncwarp();
    } else {
        // ------------------------------------------------------------ builders of the G tiles
        const int b = tid - 64;
        // this thread's chunk of every row of G it builds: columns 8c .. 8c+7 = shift row a, element e of the
        // nb*Ci contiguous strip elements that row contributes (-1: padding column)
        const int nvec = p.Mp / 8, nvec_log2 = p.Mp == 64 ? 3 : 4;      // Mp is 64 or 128
        const int c = b & (nvec - 1), pl_first = b >> nvec_log2, pl_step = kGfBuilders >> nvec_log2;
        const int r_first = pl_first / p.Wo, wo_first = pl_first - r_first * p.Wo;
        const size_t chunk_off = (size_t)(c >> 3) * p.a_chunk_bytes;
        int coff[8];
        {
            const int nbci = p.nb * p.Ci;
            int a = (c * 8) / nbci, e = c * 8 - a * nbci;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                coff[q] = a < p.na ? a * p.span + e : -1;
                if (++e == nbci) { e = 0; ++a; }
            }
        }
        // fast path: twelve elements per strip row and a number of strip rows per position that divides the
        // number of builder threads (a thread then stays with one strip row)
        const bool fast12 = p.nb * p.Ci == 12 && kGfBuilders % p.na == 0;
        const int a12 = fast12 ? b % p.na : 0, pl12 = fast12 ? b / p.na : 0, step12 = fast12 ? kGfBuilders / p.na : 1;
        const int r12 = pl12 / p.Wo, wo12 = pl12 - r12 * p.Wo;
        bool ok = true;
        for (int kt = kt_begin, i = 0; kt < kt_end; ++kt, ++i) {
            const int sa = i % kGfSlotsA;
            const int ss = i % kGfSlotsS;
            const unsigned short* cur = strip + (size_t)ss * strip_el + p.lead;
            // one lane per warp polls the barriers (hundreds of threads spinning on shared memory would compete
            // with the MMA's operand reads); the warp-wide vote also orders the other lanes behind the wait
            if (lane == 0) {
                if (!mbar_wait(&fullS[ss], (i / kGfSlotsS) & 1, abort_flag)) { gf_timeout(&abort_s, p.status, 0x440u + ss); ok = false; }
                if (ok && i >= kGfSlotsA && !mbar_wait(&emptyA[sa], ((i / kGfSlotsA) & 1) ^ 1, abort_flag)) {
                    gf_timeout(&abort_s, p.status, 0x400u + sa);
                    ok = false;
                }
            }
            ok = __all_sync(0xffffffffu, ok);
            if (ok && fast12) {
                // Twelve elements per strip row (four shifts of three channels, say): a thread copies the
                // 24 bytes one strip row contributes to one row of G -- seven aligned 32-bit reads, shifted
                // by one element when the run starts on an odd one, three 8-byte stores -- instead of
                // assembling 16-byte chunks from 2-byte reads. Shared-memory bandwidth is what bounds
                // this kernel (the MMA reads its operands from there too).
                unsigned char* slot = a_gen + (size_t)sa * p.a_slot_bytes;
                int r = r12, wo = wo12;
                for (int pl = pl12; pl < p.npos; pl += step12) {
                    const int idx = ss * strip_el + p.lead + (r * p.mh + a12) * p.span + wo * p.mw * p.Ci;
                    const uint32_t* w32 = reinterpret_cast<const uint32_t*>(strip) + (idx >> 1);
                    uint32_t w[7], o[6];
#pragma unroll
                    for (int j = 0; j < 7; ++j) w[j] = w32[j];
                    if (idx & 1) {
#pragma unroll
                        for (int j = 0; j < 6; ++j) o[j] = __funnelshift_r(w[j], w[j + 1], 16);
                    } else {
#pragma unroll
                        for (int j = 0; j < 6; ++j) o[j] = w[j];
                    }
                    unsigned char* cell = slot + (size_t)pl * 128;
#pragma unroll
                    for (int j = 0; j < 3; ++j) {
                        const int off = a12 * 24 + 8 * j, cc = off >> 4;      // byte offset in the row of G, its 16-byte chunk
                        unsigned char* dst = cell + (size_t)(cc >> 3) * p.a_chunk_bytes + (((cc & 7) ^ (pl & 7)) << 4) + (off & 8);
                        *reinterpret_cast<uint2*>(dst) = make_uint2(o[2 * j], o[2 * j + 1]);
                    }
                    wo += step12;
                    while (wo >= p.Wo) { wo -= p.Wo; ++r; }
                }
                fence_proxy_async_smem();
            } else if (ok) {
                unsigned char* slot = a_gen + (size_t)sa * p.a_slot_bytes;
                // one (position, 16-byte chunk) pair per step; the chunk, and with it the eight strip
                // offsets, are this thread's for good, the position advances by a fixed number of cells
                int r = r_first, wo = wo_first;
                for (int pl = pl_first; pl < p.npos; pl += pl_step) {
                    const unsigned short* zb = cur + r * p.mh * p.span + wo * p.mw * p.Ci;
                    unsigned short val[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) val[q] = coff[q] >= 0 ? zb[coff[q]] : (unsigned short)0;
                    // cell pl, 16-byte chunk c of its 64-channel block: the swizzle exchanges chunk c
                    // with c ^ (cell mod 8) (slots are 1024-byte aligned, so cell mod 8 is address bits 7-9)
                    unsigned char* dst = slot + chunk_off + (size_t)pl * 128 + (((c & 7) ^ (pl & 7)) << 4);
                    *reinterpret_cast<uint4*>(dst) =
                        make_uint4(val[0] | (uint32_t)val[1] << 16, val[2] | (uint32_t)val[3] << 16,
                                   val[4] | (uint32_t)val[5] << 16, val[6] | (uint32_t)val[7] << 16);
                    wo += pl_step;
                    while (wo >= p.Wo) { wo -= p.Wo; ++r; }
                }
                fence_proxy_async_smem();      // the MMA reads these cells through the async proxy
            }
            // no barrier across the builder warps: each reports its share of the tile built (and its reads of
            // the strip done) and goes on to the next tile
            if (!__all_sync(0xffffffffu, ok)) break;
            if (lane == 0) { mbar_arrive(&fullA[sa]); mbar_arrive(&emptyS[ss]); }
        }

        // ------------------------------------------------------------ drain
        bool done = mbar_wait(&done_bar, 0, abort_flag);
        if (!done) gf_timeout(&abort_s, p.status, 0x600u);
        done = __all_sync(0xffffffffu, done);
        if (done) {
            tc_fence_after();
            if (warp == 2 && lane == 0) pdl_launch_dependents();
            const int quarter = warp & 3, m = quarter * 32 + lane;      // accumulator row = column of G
            float* dst = p.out + (long long)split * p.slice_elems;
            const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
            // the builder warps that share a quarter of the tensor-memory lanes take the 32-column chunks in turn
            for (int ch = (warp - 2) >> 2; ch < p.BN / 32; ch += kGfBuilders / 128) {
                uint32_t v[32];
                tmem_ld32(lane_base + (uint32_t)(ch * 32), v);
                if (m < p.Mp) {
                    float* q = dst + (long long)(co0 + ch * 32) * p.Mp + m;
#pragma unroll
                    for (int j = 0; j < 32; ++j) q[(long long)j * p.Mp] = __uint_as_float(v[j]);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, p.tmem_cols);
}

// dW[co][r][s][ci] = sum over K-slices of slice[co][column of (r, s, ci)]. One warp per element of dW:
// lane l adds slices l, l + 32, ... in order, then the 32 running sums are combined by a butterfly
// (a fixed tree), so the result does not depend on anything but the slices.
struct GfReduceParams {
    int splits, R, S, Ci, ph, pw, k, u0, v0, nb, Mp;
    long long slice_elems, total;
};

__global__ void __launch_bounds__(256) gf_reduce_scatter_kernel(const float* __restrict__ partials, GfReduceParams q,
                                                                float* __restrict__ dw) {
    pdl_wait();
    const long long i = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (i >= q.total) return;
    const int lane = threadIdx.x & 31;
    const int row = q.R * q.S * q.Ci;
    const long long co = i / row;
    const int rem = (int)(i - co * row);
    const int t = rem / q.Ci, ci = rem - t * q.Ci, r = t / q.S, s = t - r * q.S;
    const int iu = floor_div_i(r - q.ph, q.k) - q.u0, iv = floor_div_i(s - q.pw, q.k) - q.v0;
    const float* src = partials + co * q.Mp + (iu * q.nb + iv) * q.Ci + ci;
    float acc = 0.f;
    for (int sp = lane; sp < q.splits; sp += 32) acc += __ldcs(src + (long long)sp * q.slice_elems);
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, d);
    if (lane == 0) dw[i] = acc;
}

// ------------------------------------------------------------------ host side
struct GfGeom {
    bool ok;
    GfParams p;
    uint32_t smem_bytes;
    size_t bytes;      // workspace: status block + K-slices
};

GfGeom gf_geom(const Dims& d) {
    GfGeom g{};
    GfParams& p = g.p;
    if (d.dtype != AC_BF16 || d.layout != AC_NHWC) return g;
    if (d.Ci >= 64 || d.Co % 64 != 0) return g;
    if (d.kh != d.kw || d.k < 2) return g;
    if (d.sh % d.k != 0 || d.sw % d.k != 0 || d.H % d.k != 0 || d.W % d.k != 0) return g;   // equal columns
    if (d.R > 255 || d.S > 255 || d.Wo > 256) return g;
    p.Ci = d.Ci; p.Hp = d.Hp; p.Wp = d.Wp; p.Ho = d.Ho; p.Wo = d.Wo; p.R = d.R; p.S = d.S;
    p.ph = d.ph; p.pw = d.pw; p.k = d.k;
    p.mh = d.sh / d.k; p.mw = d.sw / d.k;
    p.u0 = floor_div_i(-d.ph, d.k); p.v0 = floor_div_i(-d.pw, d.k);
    p.na = floor_div_i(d.R - 1 - d.ph, d.k) - p.u0 + 1;
    p.nb = floor_div_i(d.S - 1 - d.pw, d.k) - p.v0 + 1;
    const long long cols = (long long)p.na * p.nb * d.Ci;
    if (cols > 128) return g;
    p.cols = (int)cols;
    p.Mp = cols <= 64 ? 64 : 128;
    const int row_el = d.Wp * d.Ci;
    if ((row_el * 2) % 16 != 0) return g;      // the strip is fetched by TMA: rows of Z a whole number of 16-byte units apart
    if ((long long)d.Hp * d.Wp * d.Ci >= (1ll << 31) || (long long)d.N * d.Ho >= (1ll << 31)) return g;
    p.x0 = floor_div_i(p.v0 * d.Ci, 8) * 8;    // ... and its first element rounded down to a 16-byte boundary
    p.lead = p.v0 * d.Ci - p.x0;
    p.span = (p.lead + ((d.Wo - 1) * p.mw + p.nb) * d.Ci + 7) / 8 * 8;
    if (p.span > 512) return g;
    p.BN = d.Co <= 256 ? d.Co : (d.Co % 256 == 0 ? 256 : (d.Co % 128 == 0 ? 128 : 64));
    p.groups = d.Co / p.BN;
    if (p.groups > kNumSMs) return g;
    p.nchunks = p.BN / 64;
    p.tmem_cols = 32;
    while (p.tmem_cols < (uint32_t)p.BN) p.tmem_cols *= 2;
    // K-tile: RB whole output rows of one image (RB divides H_o), at most 256 positions, rounded up to the
    // MMA's K = 16: of the RB that fit the shared memory with at least two gradient slots, the one that wastes
    // the least, the larger one on ties
    double best_eff = 0.0;
    p.RB = 0;
    for (int rb = 1; rb <= d.Ho && rb * d.Wo <= 256; ++rb) {
        if (d.Ho % rb != 0) continue;
        const int kt = (rb * d.Wo + 15) / 16 * 16, nz = (rb - 1) * p.mh + p.na;
        if (nz > 256 || (long long)nz * p.span > 32767) continue;
        const uint32_t chunk = (uint32_t)kt * 128, box = (uint32_t)(nz * p.span * 2);
        const uint32_t fixed = 1024 + kGfSlotsA * (uint32_t)(p.Mp / 64) * chunk + kGfSlotsS * ((box + 16u + 127u) & ~127u);
        if (fixed + 2 * (uint32_t)p.nchunks * chunk > kGfSmemBudget) continue;
        const double eff = (double)rb * d.Wo / kt;
        if (eff >= best_eff) { best_eff = eff; p.RB = rb; }
    }
    if (p.RB == 0) return g;
    p.npos = p.RB * d.Wo;
    p.KT = (p.npos + 15) / 16 * 16;
    p.ksteps = p.KT / 16;
    p.nz = (p.RB - 1) * p.mh + p.na;
    p.a_chunk_bytes = (uint32_t)p.KT * 128;
    // An M = 128 MMA reads two 64-column chunks, a chunk apart. With 64 columns or fewer only the first exists: what
    // the MMA then reads as the second chunk is the next slot (or, behind the last one, the first gradient slot, which
    // is at least as large), and accumulator rows 64-127 hold sums nobody reads.
    p.a_slot_bytes = (uint32_t)(p.Mp / 64) * p.a_chunk_bytes;
    p.b_chunk_bytes = (uint32_t)p.KT * 128;
    p.b_slot_bytes = (uint32_t)p.nchunks * p.b_chunk_bytes;
    p.b_box_bytes = 128u * (uint32_t)p.npos;
    p.strip_box_bytes = (uint32_t)(p.nz * p.span * 2);
    // slot stride: TMA destinations stay 128-byte aligned; 16 bytes to spare, because the builders' 32-bit reads
    // may take in one element behind a run
    p.strip_bytes = (p.strip_box_bytes + 16u + 127u) & ~127u;
    const uint32_t fixed = 1024 + kGfSlotsA * p.a_slot_bytes + kGfSlotsS * p.strip_bytes;
    p.slotsB = (int)((kGfSmemBudget - fixed) / p.b_slot_bytes);
    if (p.slotsB > kGfMaxSlotsB) p.slotsB = kGfMaxSlotsB;
    g.smem_bytes = fixed + p.slotsB * p.b_slot_bytes;
    if (g.smem_bytes < 120 * 1024) g.smem_bytes = 120 * 1024;      // one CTA per SM: tensor memory is not shared
    const long long ktiles = (long long)d.N * d.Ho / p.RB;
    if (ktiles >= (1ll << 30)) return g;
    p.ktiles = (int)ktiles;
    int splits = d.sms / p.groups;
    if (splits < 1) splits = 1;
    if (splits > p.ktiles) splits = p.ktiles;
    const int per_slice = (p.ktiles + splits - 1) / splits;
    p.splits = (p.ktiles + per_slice - 1) / per_slice;
    p.slice_elems = (long long)d.Co * p.Mp;
    p.dw_elems = d.dw_elems();
    g.bytes = kStatusBlockBytes + (size_t)p.splits * p.slice_elems * 4;
    g.ok = true;
    return g;
}

typedef CUresult (*GfEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                               const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                               CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

GfEncodeFn gf_encode_fn() {
    static const GfEncodeFn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            return reinterpret_cast<GfEncodeFn>(f);
        return static_cast<GfEncodeFn>(nullptr);
    }();
    return fn;
}

static_assert(sizeof(GfParams) <= 4000, "kernel parameters must stay below the 4 KB limit");

}  // namespace

bool gather_fused_supported(const Dims& d) { return gf_geom(d).ok; }

size_t gather_fused_workspace_bytes(const Dims& d) { return gf_geom(d).bytes; }

void gather_fused_plan_info(const Dims& d, ac_plan_info* info) {
    const GfGeom g = gf_geom(d);
    info->tensor_core = 6;
    info->splits = g.p.splits;
    info->ctas = g.p.splits * g.p.groups;
    info->groups = g.p.groups;
    info->band_rows = g.p.RB;
    info->k_tile = g.p.KT;
    info->row_pitch = g.p.Wo;
    info->stages = g.p.slotsB;
    info->smem_bytes = (int32_t)g.smem_bytes;
    info->tmem_columns = (int32_t)g.p.tmem_cols;
    info->units_per_cta = 1;
    info->block_n = g.p.BN;
    info->a_cells = g.p.KT;
    info->phases = 1;
}

ac_status launch_wgrad_gather_fused(const Dims& d, const void* z, const void* dy, float* dw, void* workspace,
                                    cudaStream_t stream) {
    GfGeom g = gf_geom(d);
    if (!g.ok) return AC_ERR_UNSUPPORTED;
    GfParams& p = g.p;
    GfEncodeFn enc = gf_encode_fn();
    if (!enc) return AC_ERR_CUDA;
    {
        // dY viewed as (Co, Wo, N*Ho); one copy brings 64 output channels of RB whole output rows
        const cuuint64_t dims[3] = {(cuuint64_t)d.Co, (cuuint64_t)d.Wo, (cuuint64_t)d.N * d.Ho};
        const cuuint64_t strides[2] = {(cuuint64_t)d.Co * 2, (cuuint64_t)d.Wo * d.Co * 2};
        const cuuint32_t box[3] = {64, (cuuint32_t)d.Wo, (cuuint32_t)p.RB};
        const cuuint32_t es[3] = {1, 1, 1};
        if (enc(&p.tmB, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(dy), dims, strides, box, es,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return AC_ERR_CUDA;
    }
    {
        // Z viewed as (pairs of bf16 along a row, Hp, N); one copy brings nz rows of span elements, zeros outside
        const cuuint64_t row_b = (cuuint64_t)d.Wp * d.Ci * 2;
        const cuuint64_t dims[3] = {row_b / 4, (cuuint64_t)d.Hp, (cuuint64_t)d.N};
        const cuuint64_t strides[2] = {row_b, (cuuint64_t)d.Hp * row_b};
        const cuuint32_t box[3] = {(cuuint32_t)p.span / 2, (cuuint32_t)p.nz, 1};
        const cuuint32_t es[3] = {1, 1, 1};
        if (enc(&p.tmZ, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<void*>(z), dims, strides, box, es,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return AC_ERR_CUDA;
    }
    p.status = static_cast<uint32_t*>(workspace);
    p.keep_status = 0;
    float* partials = reinterpret_cast<float*>(static_cast<char*>(workspace) + kStatusBlockBytes);
    p.out = partials;
    static bool attr_done[64] = {};
    {
        const ac_status st_ = ensure_smem_limit(wgrad_gather_fused_kernel, (int)(kGfSmemBudget + 1024), attr_done);
        if (st_ != AC_OK) return st_;
    }
    record_timing_hook(0, stream);
    launch_after(wgrad_gather_fused_kernel, dim3(p.groups * p.splits), dim3(kGfThreads), g.smem_bytes, stream, p);
    record_timing_hook(1, stream);
    AC_CUDA_TRY(cudaGetLastError());
    GfReduceParams q;
    q.splits = p.splits; q.R = d.R; q.S = d.S; q.Ci = d.Ci; q.ph = d.ph; q.pw = d.pw; q.k = d.k;
    q.u0 = p.u0; q.v0 = p.v0; q.nb = p.nb; q.Mp = p.Mp; q.slice_elems = p.slice_elems; q.total = p.dw_elems;
    launch_after(gf_reduce_scatter_kernel, dim3((unsigned)((q.total + 7) / 8)), dim3(256), 0, stream,
                 static_cast<const float*>(partials), q, dw);
    AC_CUDA_TRY(cudaGetLastError());
    return AC_OK;
}

}  // namespace ac
