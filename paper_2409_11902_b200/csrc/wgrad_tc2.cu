// Compressed weight gradient on tcgen05 tensor cores, fed entirely by TMA.
//
// Same contraction as wgrad_tc.cu,
//   dW[co,r,s,ci] = sum_{n,ho,wo} dY[n,ho,wo,co] * Xt[n, ho*sh-ph+r, wo*sw-pw+s, ci],
// Xt = Z inflated by k (Section 4 of the paper), but the inflation is folded
// into the addressing instead of being written out in shared memory.
//
// Take k = 2, stride 1. Xt[h][w] = Z[h/2][w/2], so for the outputs with
// ho = 2i + a, wo = 2j + b (one "class" (a,b) of the four parity classes) tap
// (r,s) reads Z[i + u][j + v] with u = floor((a - ph + r)/2), v = floor((b - pw
// + s)/2): a constant shift of the COMPACT Z tile. In general, when the strides
// divide k, the outputs split into (k/sh)*(k/sw) classes and each (class, tap)
// pair is a shift (u,v) of Z. Zero padding falls out of
// the tile bounds: x < 0 or x >= H  <=>  z < 0 or z >= H/k.
//
// Per K-tile (a band of class rows of one image, or several whole class images of a small map):
//   A operand: the Z halo tile, one TMA copy per 64-channel chunk into the 128-byte-swizzled
//              MN-major layout [cell][64 channels] (128 bytes per cell, as NHWC memory has
//              them); a (class, tap) pair only moves the MMA descriptor's start address by
//              whole cells. With partial pooling blocks (k does not divide H or W) up to four
//              copies of the tile, fetched through tensor maps that end one row / column
//              early, serve the taps that must read zero padding there. With 64 input
//              channels up to three shifted copies let one M = 128 MMA compute two taps.
//   B operand: for each class, the de-interleaved dY tile through a per-class tensor map
//              (strides c_w*Co and c_h*Wo*Co; more than 16 classes: one map over dY walked
//              with element strides), same swizzle, rows past the class's extent
//              zero-filled by TMA.
//   Both use the same flat row pitch Wzq, which is what makes a tap a pure shift.
// Warps 0 and 7 issue the TMA copies (one chunk per lane; each ring slot belongs to one of the two
// warps), warps 1-6 issue tcgen05.mma (each its own accumulator tiles, one elected lane), warps 2-5
// then drain the accumulators from tensor memory. Every CTA keeps all the accumulator tiles that fit
// its 512 TMEM columns; K is split over CTAs and the partial dW tensors are summed in a fixed order
// afterwards.
//
// A stride that is a multiple m of k (k = 1 at stride 2) has one class, and output row i reads Z row
// m*i + u through tap row r (u = floor((r - ph)/k)): row i + floor(u/m) of the phase plane u mod m of Z.
// The planes the taps use are fetched through strided tensor-map views and kept as the tile's copies.
#include <cuda.h>

#include <cstring>
#include <mutex>

#include "ac_common.h"
#include "tc_ptx.cuh"
#include "tc_units.h"

namespace ac {
namespace {

using namespace tc;

constexpr int kThreads2 = 256;        // warps 0 and 7: TMA, warps 1 and 6: MMA (1 owns TMEM), warps 2-5: epilogue (and MMA)
constexpr int kProducers = 2;         // TMA-issuing warps (a third would leave each thread too few registers)
constexpr int kMaxMmaWarps = 6;       // accumulator tiles are dealt out over up to this many issuing warps
constexpr int kMaxUnits2 = 8;
constexpr int kMaxClasses = 64;      // output classes (k/s_h * k/s_w), e.g. k = 8 at stride 1
constexpr int kMaxClassMaps = 16;    // classes that get a tensor map of their own
constexpr int kSlotsA = 2;
constexpr int kMaxSlotsB = 8;
constexpr uint32_t kSmemBudget2 = 220 * 1024;
constexpr bool kEnablePairs = true;   // tap pairing for 64-channel layers (plan_pairs)

struct Tc2Params {
    CUtensorMap tmA[4];               // Z as (Ci, Wp, Hp, N); variants 1-3 leave out the partial last
                                      // row and/or column of Z (see `variants` below)
    CUtensorMap tmB[kMaxClassMaps];   // dY, one strided view per class: (Co, J_b, I_a, N)
    CUtensorMap tmBs;                 // more classes than that: dY itself with element strides (c_w, c_h)
    int strided_map;
    float* out;
    uint32_t* status;
    int keep_status;   // 1: a launch earlier in the same call owns the status block; do not reset it
    int Ci, Co, R, S, sh, sw, ph, pw, kh, kw;   // pooling block kh x kw (square in the paper: kh = kw = k)
    int c_h, c_w, ncls;
    int mh, mw;        // stride / pooling block where the stride is the larger one (phase planes of Z, below), else 1
    int umin, vmin;
    int Wzq, Ic, bands, KT, ksteps, rowsA;
    int NB, rowsB;   // images per K-tile (> 1 only when a tile is a whole class image) and dY rows per image
    int CB, ncgpc, ncib_total, BN, nchunks;
    int taps_per_group, ntapgroups, cibs_per_group, ncibgroups, groups, splits, ktiles;
    int slotsB;
    uint32_t a_slot_bytes, b_slot_bytes, b_chunk_bytes, a_chunk_bytes, a_box_bytes, b_box_bytes, tmem_cols;
    int chunksA;   // 64-channel chunks of the input tile per variant (incl. one never loaded when CB = 64)
    // When k does not divide H (W), the last row (column) of Z is a partial block: it stands for
    // x in [k*(Hp-1), H) but a tap may also reach the padding rows x in [H, k*Hp), which must read
    // 0. A (class, tap) pair whose x falls in that second range at the last Z row is served from a
    // copy of the tile fetched through a tensor map that ends one row (column) earlier.
    // When the stride is a multiple m of the pooling block (k = 1 at stride 2: the uncompressed gradient of a
    // strided layer), output row i reads, through tap row r, Z row m*i + u_r with u_r = floor((r - pad) / k):
    // row i + floor(u_r / m) of the PHASE PLANE u_r mod m of Z (every m-th row from that phase on). The planes a
    // layer's taps use take the place of the variants (phase row * 2 + phase column; no partial blocks then).
    int nvar, var_slot[4], rho_h, rho_w;   // variants in use, variant -> position in the slot, H % k, W % k
    int Hp, Wp, Ho, Wo;                    // pooled and output map sizes (which pairs need a variant)
    long long dw_elems;
    // Paired mode (64 input channels): one accumulator tile holds TWO taps, rows 0-63
    // tap A and rows 64-127 tap B, because the input tile is kept in up to three copies
    // (8 planes each) shifted against each other; see plan_pairs().
    int pair_mode, pu_count, ncopies;
    int copy_du[3], copy_dv[3];                  // shift of copy g in Z rows / columns
    signed char pu_tapA[kMaxUnits2], pu_tapB[kMaxUnits2];
    unsigned int pu_off[kMaxClassMaps][kMaxUnits2];   // A start offset in bytes of (class, unit)
    // Collapsed mode: within one output class, taps that read the same shift (u,v) of Z form
    // the same products, so the class gets one accumulator tile per DISTINCT shift instead of
    // one per tap. Tiles are numbered class by class (cu_total in all); a CTA owns cu_cap
    // consecutive ones and loads only the classes they belong to; the partial tensor is indexed
    // by that number and the reduction adds each tile to every tap that maps to it.
    int collapse, cu_total, cu_cap;
    // K-tiles after which the accumulators are written out (added to what this CTA wrote before) and
    // started afresh; 0: only at the end. Bounds the length of the tensor core's truncating fp32
    // accumulation chains for results that must hold an fp32 bound.
    int chunk_kt;
    long long slice_elems;   // floats of one K-slice of the partial tensor
};

// Whether outputs of class row `a` (ho = a, a + k/s, ...) read, through tap row r, one of the rows
// x in [H, k*Hp) that the convolution pads with zeros but the partial last row of Z covers. Every x
// this pair reads, x = s*ho - pad + r, has the same remainder rem = (s*a - pad + r) mod k, so the one
// candidate is x = k*(Hp-1) + rem with rem >= rho = H mod k; it is read only if the ho it belongs
// to is an output row (a 1x1 layer without padding never reads beyond H, whatever the map size).
// The same function serves columns.
__host__ __device__ inline bool reads_padding_in_partial_block(int s, int a, int pad, int r, int k, int Hp,
                                                               int rho, int Ho) {
    if (rho == 0) return false;
    const int c = s * a - pad + r;
    const int rem = c - floor_div_i(c, k) * k;
    if (rem < rho) return false;
    const int num = k * (Hp - 1) + rem + pad - r;      // s * ho of the candidate
    if (num < 0 || num % s != 0) return false;
    return num / s < Ho;
}

// Shift and phase plane of output class coordinate `a` through tap coordinate r: the Z coordinate read is
// (k/s classes) i + shift, or (stride a multiple m of k, one class) m*i + u = plane (u mod m), coordinate
// i + floor(u / m).
__host__ __device__ inline int tap_shift(int s, int a, int pad, int r, int k, int m, int* phase) {
    const int u = floor_div_i(s * a - pad + r, k);
    if (m <= 1) { *phase = 0; return u; }
    const int q = floor_div_i(u, m);
    *phase = u - q * m;
    return q;
}

// Distinct Z shifts of output class `cls`: rows u0 .. u0+nU-1, columns v0 .. v0+nV-1
// (u = floor((s_h*a - p_h + r) / k) is non-decreasing in r with steps of 0 or 1).
struct ClassShifts { int u0, nU, v0, nV; };
__host__ __device__ inline ClassShifts class_shifts(int cls, int c_w, int sh, int sw, int ph, int pw,
                                                    int kh, int kw, int R, int S) {
    const int a = cls / c_w, b = cls - a * c_w;
    ClassShifts c;
    c.u0 = floor_div_i(sh * a - ph, kh);
    c.nU = floor_div_i(sh * a - ph + R - 1, kh) - c.u0 + 1;
    c.v0 = floor_div_i(sw * b - pw, kw);
    c.nV = floor_div_i(sw * b - pw + S - 1, kw) - c.v0 + 1;
    return c;
}

extern __shared__ __align__(1024) unsigned char tc2_smem[];

// Development aid, compiled in only with -DAC_TC2_TRACE (never in the library as built by
// build.py): per-CTA clock stamps and wait totals, read back with ac_debug_read_trace.
#ifdef AC_TC2_TRACE
constexpr int kTraceWords = 32;
__device__ long long g_trace[kNumSMs * 2 * kTraceWords];
#define TRACE_SET(slot, value) do { if (blockIdx.x < kNumSMs * 2) g_trace[blockIdx.x * kTraceWords + (slot)] = (value); } while (0)
#define TRACE_ADD(slot, value) do { if (blockIdx.x < kNumSMs * 2) g_trace[blockIdx.x * kTraceWords + (slot)] += (value); } while (0)
#define TRACE_CLOCK() clock64()
__device__ __forceinline__ long long trace_gtime() { long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
#else
#define TRACE_SET(slot, value) do { } while (0)
#define TRACE_ADD(slot, value) do { } while (0)
#define TRACE_CLOCK() 0ll
#endif

__device__ __forceinline__ void flag_timeout(int* abort_s, uint32_t* status, uint32_t code) {
    if (atomicExch(abort_s, 1) == 0) {
        status[1] = code;
        atomicExch(&status[0], 1u);
    }
}

// 32 accumulator columns of one row to memory, `stride` floats apart; `add_to`: added to what this
// thread stored there before (all loads first, so that they overlap).
__device__ __forceinline__ void put32(float* q, long long stride, const uint32_t* v, bool add_to) {
    if (!add_to) {
#pragma unroll
        for (int j = 0; j < 32; ++j) q[j * stride] = __uint_as_float(v[j]);
        return;
    }
    float old[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) old[j] = q[j * stride];
#pragma unroll
    for (int j = 0; j < 32; ++j) q[j * stride] = old[j] + __uint_as_float(v[j]);
}

__global__ void __launch_bounds__(kThreads2, 1) wgrad_tc2_kernel(const __grid_constant__ Tc2Params p) {
    __shared__ uint64_t fullA[kSlotsA], emptyA[kSlotsA];
    __shared__ uint64_t fullB[kMaxSlotsB], emptyB[kMaxSlotsB];
    __shared__ uint64_t done_bar, tfree_bar;   // accumulators complete / accumulators read out
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ uint32_t aoff_tab[kMaxClasses][kMaxUnits2];   // A start offset of (class, unit)
    __shared__ int unit_cls[kMaxUnits2];                     // collapsed mode: class (minus cls0) of a tile
    volatile int* abort_flag = &abort_s;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
#ifdef AC_TC2_TRACE
    const long long tr_t0 = clock64();
    if (tid == 0) {
        for (int i = 0; i < kTraceWords; ++i) TRACE_SET(i, 0);
        TRACE_SET(0, trace_gtime());
    }
#endif
    const int group = blockIdx.x % p.groups, split = blockIdx.x / p.groups;
    const int tg = group % p.ntapgroups;
    const int cibg = (group / p.ntapgroups) % p.ncibgroups;
    const int cob = group / (p.ntapgroups * p.ncibgroups);
    const int RS = p.R * p.S;
    const int tap0 = tg * p.taps_per_group;
    const int ntap = min(p.taps_per_group, RS - tap0);
    const int cib0 = cibg * p.cibs_per_group;
    const int ncib = min(p.cibs_per_group, p.ncib_total - cib0);
    // collapsed mode: this CTA's tiles are numbers [cj0, cj0 + nunits) of the class-by-class
    // numbering; they belong to classes [cls0, cls1)
    int cls0 = 0, cls1 = p.ncls, cj0 = 0, cn = 0;
    if (p.collapse) {
        cj0 = tg * p.cu_cap;
        cn = min(p.cu_cap, p.cu_total - cj0);
        int base = 0;
        cls0 = -1;
        for (int c = 0; c < p.ncls; ++c) {
            const ClassShifts cs = class_shifts(c, p.c_w, p.sh, p.sw, p.ph, p.pw, p.kh, p.kw, p.R, p.S);
            const int cnt = cs.nU * cs.nV;
            if (cls0 < 0 && base + cnt > cj0) cls0 = c;
            if (base < cj0 + cn) cls1 = c + 1;
            base += cnt;
        }
    }
    const int ncls_mine = cls1 - cls0;
    const int nunits = p.collapse ? cn : (p.pair_mode ? p.pu_count : ncib * ntap);
    const int co0 = cob * p.BN;
    const int kt_begin = (int)((long long)p.ktiles * split / p.splits);
    const int kt_end = (int)((long long)p.ktiles * (split + 1) / p.splits);
    const int chunk_kt = p.chunk_kt > 0 ? p.chunk_kt : 0x7fffffff;
    // MMA-issuing warps. An issuing warp that turns to another accumulator tile stalls for a few
    // hundred cycles (measured: ~280, whatever the tile's width) while MMAs of other warps go on
    // undisturbed, so every tile gets a warp of its own where possible: warps 1 and 6, then the four
    // epilogue warps, which have nothing else to do until the accumulators are complete. When the
    // accumulators are written out in the middle of the K-slice (chunk_kt), the epilogue warps must
    // stay free for that, and warps 1 and 6 share the tiles.
    const int nmw = p.chunk_kt > 0 ? 2 : min(max(nunits, 1), kMaxMmaWarps);
    const int mw = warp == 1 ? 0 : (warp == 6 ? 1 : warp);      // this warp's place among them (warp 0: none)
    // 1024-byte aligned tile area: A slots first, then B slots
    const uint32_t smem_base = (smem_u32(tc2_smem) + 1023u) & ~1023u;
    unsigned char* smem_gen = tc2_smem + (smem_base - smem_u32(tc2_smem));
    const uint32_t a_base = smem_base, b_base = smem_base + kSlotsA * p.a_slot_bytes;


    // ---------------------------------------------------------------- TMA producers
    // The stream of copies is, for each K-tile, the Z halo tile (one 64-channel chunk per lane, so that
    // the chunks of a tile go out as one warp instruction), then one gradient tile per class (likewise).
    // Issuing one such instruction takes a warp 650-850 cycles (measured with a stand-alone loop: 650
    // for one box, +55 for each further lane), whatever the state of the barriers, while a second
    // warp's copies go out in parallel (two issuing warps: twice the rate). For layers whose tiles
    // carry little arithmetic (1x1 and stride-2 layers: a K-tile of 1000-2000 cycles of MMAs needs two
    // to five copies) one warp cannot keep up, so two warps issue. Each SLOT of the two rings belongs
    // to one producer warp for good: a wait on a slot's barrier tests the parity of its phase, which
    // is only right for a waiter that has seen every earlier phase of that barrier go by (a warp that
    // came to the slot two phases early would find the parity it looks for and overwrite a tile in
    // use). Every warp walks the whole stream in order and issues the copies whose slot is its own;
    // the MMA warps consume in stream order, so the producers need no order among themselves.
    const int pw_idx = warp == 0 ? 0 : warp - 6;      // producer warps 0 and 7 -> 0, 1
    auto produce = [&]() {
        const int nchunk_ld = p.pair_mode ? p.ncopies : ncib * (p.CB / 64);   // 64-channel chunks per variant
        const int nloads = nchunk_ld * p.nvar;
        int tb = 0;
        for (int t = 0, kt = kt_begin; kt < kt_end; ++t, ++kt) {
            const int n = p.NB > 1 ? kt * p.NB : kt / p.bands;
            const int i0 = p.NB > 1 ? 0 : (kt - n * p.bands) * p.Ic;
            const int sa = t % kSlotsA;
            if (sa % kProducers == pw_idx) {
                if (t >= kSlotsA) {
                    [[maybe_unused]] const long long tw = TRACE_CLOCK();
                    const bool got = mbar_wait(&emptyA[sa], ((t / kSlotsA) & 1) ^ 1, abort_flag);
                    if (lane == 0 && warp == 0) TRACE_ADD(8, TRACE_CLOCK() - tw);
                    if (!__all_sync(0xffffffffu, got)) {
                        if (lane == 0) flag_timeout(&abort_s, p.status, 0x100u + sa);
                        return;
                    }
                }
                if (lane == 0) mbar_arrive_expect_tx(&fullA[sa], (uint32_t)nloads * p.a_box_bytes);
                __syncwarp();
                const uint32_t a_slot = a_base + sa * p.a_slot_bytes;
                if (lane < nloads) {
                    const int vs = lane / nchunk_ld, c = lane - vs * nchunk_ld;   // variant position, chunk
                    int var = 0;
                    for (int v = 0; v < 4; ++v) if (p.var_slot[v] == vs) var = v;
                    // paired mode: chunk c is copy c of the same 64 channels, shifted
                    const int ch = p.pair_mode ? 0 : c * 64;
                    const int dv = p.pair_mode ? p.copy_dv[c] : 0, du = p.pair_mode ? p.copy_du[c] : 0;
                    tma_load_4d(a_slot + (vs * p.chunksA + c) * p.a_chunk_bytes, &p.tmA[var], &fullA[sa],
                                cib0 * p.CB + ch, p.vmin + dv, i0 + p.umin + du, n);
                }
            }
            for (int cl = 0; cl < ncls_mine; ++cl, ++tb) {
                const int sb = tb % p.slotsB;
                if ((sb + kSlotsA) % kProducers != pw_idx) continue;      // offset: the warps with an input slot get fewer
                if (tb >= p.slotsB) {
                    [[maybe_unused]] const long long tw = TRACE_CLOCK();
                    const bool got = mbar_wait(&emptyB[sb], ((tb / p.slotsB) & 1) ^ 1, abort_flag);
                    if (lane == 0 && warp == 0) TRACE_ADD(9, TRACE_CLOCK() - tw);
                    if (!__all_sync(0xffffffffu, got)) {
                        if (lane == 0) flag_timeout(&abort_s, p.status, 0x180u + sb);
                        return;
                    }
                }
                if (lane == 0) mbar_arrive_expect_tx(&fullB[sb], (uint32_t)p.nchunks * p.b_box_bytes);
                __syncwarp();
                const uint32_t b_slot = b_base + sb * p.b_slot_bytes;
                if (lane < p.nchunks) {
                    const int cls_id = cls0 + cl;
                    if (p.strided_map) {
                        // one map over dY, traversed with strides (c_w, c_h): the class is the start
                        const int a = cls_id / p.c_w, b = cls_id - a * p.c_w;
                        tma_load_4d(b_slot + lane * p.b_chunk_bytes, &p.tmBs, &fullB[sb], co0 + 64 * lane, b,
                                    p.c_h * i0 + a, n);
                    } else {
                        tma_load_4d(b_slot + lane * p.b_chunk_bytes, &p.tmB[cls_id], &fullB[sb],
                                    co0 + 64 * lane, 0, i0, n);
                    }
                }
            }
        }
    };

    if (warp == 0) {
        // Every tensor map this CTA will use is fetched now, all at once: left to the first copy
        // that names it, each fetch (about half a microsecond) would hold up the issuing warp in turn.
        if (lane < 4) {
            if (p.var_slot[lane] >= 0) prefetch_tmap(&p.tmA[lane]);
        } else if (p.strided_map) {
            if (lane == 4) prefetch_tmap(&p.tmBs);
        } else if (lane - 4 < p.ncls) {
            prefetch_tmap(&p.tmB[lane - 4]);
        }
        if (lane == 0) {
            for (int s = 0; s < kSlotsA; ++s) { mbar_init(&fullA[s], 1); mbar_init(&emptyA[s], nmw); }
            for (int s = 0; s < p.slotsB; ++s) { mbar_init(&fullB[s], 1); mbar_init(&emptyB[s], nmw); }
            mbar_init(&done_bar, nmw);
            mbar_init(&tfree_bar, 4);
            abort_s = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncwarp();
        // The barriers are ready, which is all the other warps need from this one: it reports in
        // at the set-up barrier without waiting there and goes straight on to issuing copies
        // (the first tile lands long before the set-up is over). The other producer warp waits
        // for nothing but this (barrier 3).
        __threadfence_block();
        bar_arrive(3, kProducers * 32);
        bar_arrive(1, kThreads2);
        // Everything up to here touched no global memory and may have run while the kernel before
        // this one in the stream (the compress kernel that writes Z, say) was still finishing.
        pdl_wait();
        // The status block starts clean: CTA 0 resets it here, long before any wait of this launch
        // can run out (a wait gives up only after 2^32 cycles).
        if (blockIdx.x == 0 && lane == 0 && !p.keep_status) { p.status[0] = 0u; p.status[1] = 0u; }
        produce();
        if (lane == 0) TRACE_SET(10, TRACE_CLOCK() - tr_t0);    // producer done
    } else if (warp >= 7) {
        bar_sync(3, kProducers * 32);      // the mbarriers exist
        bar_arrive(1, kThreads2);
        pdl_wait();
        produce();
    }
    // Everything the MMAs may read but no copy ever writes must be finite (it only
    // ever meets zeros of the other operand, or feeds accumulator rows that are
    // discarded): the cells behind the last row of each input plane, the planes of
    // the unused upper 64 rows when CB = 64, and the gradient rows behind the tile.
    if (warp == 1) tmem_alloc(&tmem_base_s, p.tmem_cols);   // about 0.6 us, beside the zero fill
    if (warp >= 2 && warp <= 6) {
        constexpr int kZeroWarps = 5;
        const uint4 zero4 = make_uint4(0, 0, 0, 0);
        const int chunks_real = p.pair_mode ? p.ncopies : ncib * (p.CB / 64);
        const int units16 = (int)(p.a_chunk_bytes / 16), written = p.NB * p.rowsA * p.Wzq * 8;
        const int chunks_slot = p.nvar * p.chunksA;
        for (int sc = warp - 2; sc < kSlotsA * chunks_slot; sc += kZeroWarps) {
            const int s_ = sc / chunks_slot, cs = sc - s_ * chunks_slot, c_ = cs % p.chunksA;
            uint4* chunk = reinterpret_cast<uint4*>(smem_gen + (size_t)s_ * p.a_slot_bytes + (size_t)cs * p.a_chunk_bytes);
            for (int c = (c_ < chunks_real ? written : 0) + lane; c < units16; c += 32) chunk[c] = zero4;
        }
        const int tail0 = p.NB * p.rowsB * p.Wzq * 8, tail1 = p.KT * 8;      // in 16-byte units per chunk
        unsigned char* bgen = smem_gen + (size_t)kSlotsA * p.a_slot_bytes;
        for (int sc = warp - 2; sc < p.slotsB * p.nchunks; sc += kZeroWarps) {
            uint4* chunk = reinterpret_cast<uint4*>(bgen + (size_t)sc * p.b_chunk_bytes);
            for (int c = tail0 + lane; c < tail1; c += 32) chunk[c] = zero4;
        }
        fence_proxy_async_smem();
    }
    if (warp >= 1 && warp <= 6) {
        if (p.collapse && tid == 32) {
            // tile u = number cj0 + u: find its class and its shift inside the class
            int base = 0, u = 0;
            for (int c = 0; c < p.ncls && u < nunits; ++c) {
                const ClassShifts cs = class_shifts(c, p.c_w, p.sh, p.sw, p.ph, p.pw, p.kh, p.kw, p.R, p.S);
                const int cnt = cs.nU * cs.nV;
                while (u < nunits && cj0 + u < base + cnt) {
                    const int j = cj0 + u - base, iu = j / cs.nV, iv = j - iu * cs.nV;
                    unit_cls[u] = c - cls0;
                    aoff_tab[0][u] = (uint32_t)((cs.u0 + iu - p.umin) * p.Wzq + (cs.v0 + iv - p.vmin)) * 128u;
                    ++u;
                }
                base += cnt;
            }
        }
        for (int t2 = tid - 32; !p.collapse && t2 < p.ncls * kMaxUnits2; t2 += 192) {
            const int cls = t2 / kMaxUnits2, u = t2 % kMaxUnits2;
            uint32_t off = 0;
            if (p.pair_mode) {
                off = p.pu_off[cls][u];
            } else if (u < nunits) {
                const int cl = u / ntap, t = u - cl * ntap;
                const int tap = tap0 + t, r = tap / p.S, sx = tap - r * p.S;
                const int a = cls / p.c_w, b = cls - a * p.c_w;
                int fh, fw;
                const int uu = tap_shift(p.sh, a, p.ph, r, p.kh, p.mh, &fh) - p.umin;
                const int vv = tap_shift(p.sw, b, p.pw, sx, p.kw, p.mw, &fw) - p.vmin;
                // which copy of the tile: the phase plane of Z this tap reads (stride a multiple of k), else
                // the one without the partial last row / column of Z if this (class, tap) reaches past H / W there
                const int var = p.mh > 1 || p.mw > 1 ? fh * 2 + fw :
                                (reads_padding_in_partial_block(p.sh, a, p.ph, r, p.kh, p.Hp, p.rho_h, p.Ho) ? 2 : 0) +
                                (reads_padding_in_partial_block(p.sw, b, p.pw, sx, p.kw, p.Wp, p.rho_w, p.Wo) ? 1 : 0);
                off = (uint32_t)(p.var_slot[var] * p.chunksA + cl * (p.CB / 64)) * p.a_chunk_bytes +
                      (uint32_t)(uu * p.Wzq + vv) * 128u;
            }
            aoff_tab[cls][u] = off;
        }
    }
    uint32_t tmem_base = 0;
    if (warp >= 1 && warp <= 6) {
        tc_fence_before();
        bar_sync(1, kThreads2);
        tc_fence_after();
        tmem_base = tmem_base_s;
        if (tid == 32) TRACE_SET(1, TRACE_CLOCK() - tr_t0);      // set-up done
    }

    if (warp >= 1 && mw < nmw) {
        // ---------------------------------------------------------- MMA issuers
        // Warp mw issues the MMAs of tiles mw, mw + nmw, ...
        // The whole warp runs the loop so that the descriptor arithmetic stays in
        // uniform registers; one elected lane issues each MMA and commit.
        const uint32_t idesc = make_idesc(p.BN);
        const uint32_t a_hi0 = desc_hi(1024, 2);             // both operands: 128-byte swizzle, 8-row atoms
        const uint32_t b_hi = desc_hi(1024, 2);              // 128-byte swizzle, 8 rows per atom
        const bool leader = elect_one();
        int tb = 0;
        bool ok = true;
        for (int kt = kt_begin, ta = 0, tac = 0, chunk = 0; kt < kt_end && ok; ++kt, ++ta, ++tac) {
            const int sa = ta % kSlotsA;
            bool got;
            if (tac == chunk_kt) {
                // The accumulation chains have reached their bound: hand the tiles to the epilogue
                // warps and go on from zero once they have read them out.
                if (leader) mma_commit(&done_bar);
                __syncwarp();
                got = mbar_wait(&tfree_bar, chunk & 1, abort_flag);
                if (!__all_sync(0xffffffffu, got)) {
                    if (leader) flag_timeout(&abort_s, p.status, 0x380u);
                    ok = false;
                    break;
                }
                tc_fence_after();
                tac = 0;
                ++chunk;
            }
            [[maybe_unused]] const long long twa = TRACE_CLOCK();
            got = mbar_wait(&fullA[sa], (ta / kSlotsA) & 1, abort_flag);
            if (leader && warp == 1) { TRACE_ADD(2, TRACE_CLOCK() - twa); if (kt == kt_begin) TRACE_SET(3, TRACE_CLOCK() - tr_t0); }
            if (!__all_sync(0xffffffffu, got)) {
                if (leader) flag_timeout(&abort_s, p.status, 0x200u + sa);
                ok = false;
                break;
            }
            const uint32_t a_lo0 = desc_lo(a_base + sa * p.a_slot_bytes, p.a_chunk_bytes);
            for (int cls = 0; cls < ncls_mine; ++cls, ++tb) {
                const int sb = tb % p.slotsB;
                [[maybe_unused]] const long long twb = TRACE_CLOCK();
                got = mbar_wait(&fullB[sb], (tb / p.slotsB) & 1, abort_flag);
                if (leader && warp == 1) TRACE_ADD(4, TRACE_CLOCK() - twb);
                if (!__all_sync(0xffffffffu, got)) {
                    if (leader) flag_timeout(&abort_s, p.status, 0x280u + sb);
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t b_lo0 = desc_lo(b_base + sb * p.b_slot_bytes, p.b_chunk_bytes);
                // a tile starts from zero at its first MMA: the first class of the first K-tile (of
                // this chunk of the K-slice), or, collapsed, the first K-tile (a collapsed tile
                // belongs to one class only)
                const uint32_t first = (p.collapse ? tac : (tac | cls)) == 0 ? 0u : 1u;
                for (int u = mw; u < nunits; u += nmw) {
                    if (p.collapse && unit_cls[u] != cls) continue;
                    // A tap shifts the start by whole 128-byte rows. The swizzle is a function of
                    // the absolute shared-memory address (TMA wrote the tile that way, slots are
                    // 1024-byte aligned), so the descriptor needs no base offset: measured, a
                    // non-zero base offset here gives wrong sums, zero gives the oracle's.
                    uint32_t a_lo = a_lo0 + (aoff_tab[p.collapse ? 0 : cls][u] >> 4);
                    const uint32_t a_hi = a_hi0;
                    uint32_t b_lo = b_lo0;
                    const uint32_t dcol = tmem_base + (uint32_t)u * p.BN;
                    if (leader) mma_bf16_words(dcol, a_lo, a_hi, b_lo, b_hi, idesc, first);
                    for (int kk = 1; kk < p.ksteps; ++kk) {
                        a_lo += 128;   // 16 cells x 128 bytes
                        b_lo += 128;   // 16 rows x 128 bytes
                        if (leader) mma_bf16_words(dcol, a_lo, a_hi, b_lo, b_hi, idesc, 1u);
                    }
                }
                if (leader) mma_commit(&emptyB[sb]);
                __syncwarp();
            }
            if (ok && leader) mma_commit(&emptyA[sa]);
            __syncwarp();
        }
        if (ok && leader) mma_commit(&done_bar);
        if (leader && warp == 1) TRACE_SET(5, TRACE_CLOCK() - tr_t0);   // last MMA issued
    }
    __syncwarp();

    // ---------------------------------------------------------------- epilogue
    const int nchunk_k = p.chunk_kt > 0 ? (kt_end - kt_begin + p.chunk_kt - 1) / p.chunk_kt : 1;
    for (int kchunk = 0; warp >= 2 && warp < 6 && kchunk < nchunk_k; ++kchunk) {
        bool ok = mbar_wait(&done_bar, kchunk & 1, abort_flag);
        if (warp == 2 && lane == 0 && kchunk + 1 == nchunk_k) TRACE_SET(6, TRACE_CLOCK() - tr_t0);   // accumulators complete
        if (!ok) flag_timeout(&abort_s, p.status, 0x300u);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const bool add_to = kchunk > 0;      // later chunks add to what the earlier ones stored
        if (kchunk == 0) pdl_wait();         // first global access of these warps (dW may still be read)
        if (kchunk + 1 == nchunk_k && warp == 2 && lane == 0)
            pdl_launch_dependents();         // the split-K reduction may be brought onto the SMs now
        {
            tc_fence_after();
            const int quarter = warp & 3;            // the TMEM lanes this warp may read
            const int m = quarter * 32 + lane;       // accumulator row
            float* dst = p.out + (long long)split * (p.collapse ? p.slice_elems : p.dw_elems);
            // floats between output channels: dW layout, or collapsed [tile][channel out][channel in]
            const long long cstride = p.collapse ? (long long)p.CB : (long long)RS * p.Ci;
            const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
            const int chunks_per_unit = p.BN / 32, nchunk = nunits * chunks_per_unit;
            // 32 columns at a time, the next chunk's tcgen05.ld in flight while this one is stored
            uint32_t buf[2][32];
            tmem_ld32_issue(lane_base, buf[0]);
            int u = 0, cu = 0;                        // unit and chunk-in-unit of chunk `ch`
#pragma unroll 1
            for (int ch = 0; ch < nchunk; ch += 2) {
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    if (ch + half < nchunk) {
                        tmem_ld_wait();
                        if (ch + half + 1 < nchunk)
                            tmem_ld32_issue(lane_base + (uint32_t)((ch + half + 1) * 32), buf[half ^ 1]);
                        int tap, ci;
                        if (p.collapse) {
                            if (m < p.CB) {
                                float* q = dst + ((((long long)cob * p.ncib_total + cib0) * p.cu_total + cj0 + u) *
                                                      p.BN + cu * 32) * p.CB + m;
                                put32(q, cstride, buf[half], add_to);
                            }
                            tap = -1; ci = 0;
                        } else if (p.pair_mode) {
                            tap = m < 64 ? p.pu_tapA[u] : p.pu_tapB[u];
                            ci = cib0 * p.CB + (m & 63);
                        } else {
                            const int cl = u / ntap;
                            tap = m < p.CB ? tap0 + (u - cl * ntap) : -1;
                            ci = (cib0 + cl) * p.CB + m;
                        }
                        if (tap >= 0) {
                            float* q = dst + ((long long)(co0 + cu * 32) * RS + tap) * p.Ci + ci;
                            put32(q, cstride, buf[half], add_to);
                        }
                        if (++cu == chunks_per_unit) { cu = 0; ++u; }
                    }
                }
            }
        }
        if (kchunk + 1 < nchunk_k) {
            // every tcgen05.ld of this warp has completed: the MMA warps may overwrite the tiles
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tfree_bar);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, p.tmem_cols);
#ifdef AC_TC2_TRACE
    if (tid == 0) { TRACE_SET(7, clock64() - tr_t0); TRACE_SET(11, trace_gtime()); TRACE_SET(12, kt_end - kt_begin); TRACE_SET(13, nunits); }
#endif
}

#ifdef AC_TC2_TRACE
}  // namespace
}  // namespace ac
extern "C" int ac_debug_read_trace(long long* host_out, int words) {
    return (int)cudaMemcpyFromSymbol(host_out, ac::g_trace, sizeof(long long) * words);
}
namespace ac {
namespace {
#endif

// Reduction of the collapsed partial tensor P[slice][co block][ci block][tile][co][ci]:
//   dW[co][r][s][ci] = sum over classes, sum over K-slices of the tile that tap (r,s) maps to in
//   that class. One float4 of ci per thread group; SL threads share the (class, slice) pairs,
// each adding its pairs in order, then the SL running sums are added in index order.
struct CollapseReduceParams {
    int splits, ncls, R, S, Ci, CB, BN, ncib_total, cu_total, c_w, sh, sw, ph, pw, kh, kw;
    long long slice_elems, elems4;
};

template <int SL>
__global__ void __launch_bounds__(256)
collapsed_reduce_kernel(const float4* __restrict__ P, CollapseReduceParams q, float4* __restrict__ dw) {
    constexpr int EL = 256 / SL;
    extern __shared__ unsigned short jmap[];          // [class][tap] -> tile number
    __shared__ float4 red[SL > 1 ? SL : 1][EL];
    const int RS = q.R * q.S;
    {
        // tile numbering: class by class, inside a class row-major over its distinct shifts
        for (int e = threadIdx.x; e < q.ncls * RS; e += 256) {
            const int cls = e / RS, tap = e - cls * RS, r = tap / q.S, sx = tap - r * q.S;
            int base = 0;
            for (int c = 0; c < cls; ++c) {
                const ClassShifts cs = class_shifts(c, q.c_w, q.sh, q.sw, q.ph, q.pw, q.kh, q.kw, q.R, q.S);
                base += cs.nU * cs.nV;
            }
            const ClassShifts cs = class_shifts(cls, q.c_w, q.sh, q.sw, q.ph, q.pw, q.kh, q.kw, q.R, q.S);
            const int a = cls / q.c_w, b = cls - a * q.c_w;
            const int iu = floor_div_i(q.sh * a - q.ph + r, q.kh) - cs.u0;
            const int iv = floor_div_i(q.sw * b - q.pw + sx, q.kw) - cs.v0;
            jmap[e] = (unsigned short)(base + iu * cs.nV + iv);
        }
    }
    __syncthreads();
    const int e = threadIdx.x % EL, sl = threadIdx.x / EL;
    const long long i = (long long)blockIdx.x * EL + e;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i < q.elems4) {
        const int ci4n = q.Ci / 4;
        const int ci = (int)(i % ci4n) * 4;
        const long long t = i / ci4n;
        const int tap = (int)(t % RS), co = (int)(t / RS);
        const int cob = co / q.BN, col = co - cob * q.BN, cib = ci / q.CB, m = ci - cib * q.CB;
        const long long tile0 = ((long long)cob * q.ncib_total + cib) * q.cu_total;
        const int pairs = q.ncls * q.splits;
        for (int pq = sl; pq < pairs; pq += SL) {
            const int cls = pq / q.splits, sp = pq - cls * q.splits;
            const long long off = (long long)sp * q.slice_elems +
                                  ((tile0 + jmap[cls * RS + tap]) * q.BN + col) * q.CB + m;
            const float4 v = __ldcs(P + off / 4);
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
    }
    if (SL == 1) {
        if (i < q.elems4) dw[i] = acc;
        return;
    }
    red[sl][e] = acc;
    __syncthreads();
    if (sl == 0 && i < q.elems4) {
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
void launch_collapsed_reduce(const float* P, const CollapseReduceParams& q, float* dw, cudaStream_t st) {
    constexpr int EL = 256 / SL;
    const size_t smem = (size_t)q.ncls * q.R * q.S * sizeof(unsigned short);
    collapsed_reduce_kernel<SL><<<(unsigned)((q.elems4 + EL - 1) / EL), 256, smem, st>>>(
        reinterpret_cast<const float4*>(P), q, reinterpret_cast<float4*>(dw));
}

// One CTA waits, with the kernels' own bounded wait, on a barrier that nothing will ever
// complete, and reports it through the workspace status block like the real kernels do.
__global__ void bounded_wait_selftest_kernel(uint32_t* status, long long limit_cycles) {
    __shared__ uint64_t never;
    __shared__ int abort_s;
    if (threadIdx.x == 0) {
        mbar_init(&never, 1);
        abort_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (!mbar_wait(&never, 0, &abort_s, limit_cycles)) flag_timeout(&abort_s, status, 0x7E57u);
}

// ------------------------------------------------------------------ host side
struct Tc2Geom {
    Tc2Params p;
    double cta_cycles;   // the cost model's main-loop time of the busiest CTA
    uint32_t smem_bytes;
    int uspan, vspan;
    double k_eff;
    bool ok;
};

// Pairing of taps for a layer with exactly 64 input channels. An MMA has M = 128 rows,
// i.e. 16 planes of 8 channels read from consecutive plane slots; with 64 channels only
// 8 planes are real. If the next 8 plane slots hold the SAME tile shifted by D cells,
// rows 64-127 compute a second tap whose offset is D larger -- provided D is the same
// for every output class. The tile is kept in up to three copies g = 0,1,2 with shifts
// S0 = 0, S1 = D1, S2 = D1 + D2; a pair with difference D1 starts at copy 0, one with
// difference D2 at copy 1, a tap without partner starts at copy 0 and wastes its upper
// rows. Picks D1, D2 that pair the most taps. Returns false if nothing can be paired.
struct PairPlan {
    int count, ncopies;
    int cu[3], cv[3];
    int tapA[kMaxUnits2], tapB[kMaxUnits2], grp[kMaxUnits2];
};

bool plan_pairs(const Dims& d, int c_h, int c_w, int umin, int vmin, int uspan, int vspan, PairPlan* out) {
    const int T = d.R * d.S, C = c_h * c_w;
    if (T > 64) return false;
    static thread_local int ou[kMaxClassMaps][64], ov[kMaxClassMaps][64];
    if (C > kMaxClassMaps) return false;
    for (int c = 0; c < C; ++c)
        for (int t = 0; t < T; ++t) {
            const int a = c / c_w, b = c % c_w, r = t / d.S, sx = t % d.S;
            ou[c][t] = floor_div_i(d.sh * a - d.ph + r, d.kh) - umin;
            ov[c][t] = floor_div_i(d.sw * b - d.pw + sx, d.kw) - vmin;
        }
    auto diff = [&](int t1, int t2, int* du, int* dv) {   // constant over classes?
        *du = ou[0][t2] - ou[0][t1]; *dv = ov[0][t2] - ov[0][t1];
        for (int c = 1; c < C; ++c)
            if (ou[c][t2] - ou[c][t1] != *du || ov[c][t2] - ov[c][t1] != *dv) return false;
        return true;
    };
    auto fits = [&](int t, int su, int sv) {              // tap t may start at a copy shifted by (su, sv)
        for (int c = 0; c < C; ++c)
            if (ou[c][t] - su < 0 || ou[c][t] - su > uspan || ov[c][t] - sv < 0 || ov[c][t] - sv > vspan)
                return false;
        return true;
    };
    int best_units = T;
    PairPlan best{};
    bool found = false;
    for (int p1 = 0; p1 < T * T; ++p1) {
        int d1u, d1v;
        if (p1 / T == p1 % T || !diff(p1 / T, p1 % T, &d1u, &d1v)) continue;
        for (int p2 = -1; p2 < T * T; ++p2) {
            int d2u = 0, d2v = 0;
            if (p2 >= 0 && (p2 / T == p2 % T || !diff(p2 / T, p2 % T, &d2u, &d2v))) continue;
            bool used[64] = {};
            PairPlan pp{};
            for (int t1 = 0; t1 < T; ++t1) {                 // pairs at copy 0
                if (used[t1]) continue;
                for (int t2 = 0; t2 < T; ++t2) {
                    int du, dv;
                    if (t2 == t1 || used[t2] || !diff(t1, t2, &du, &dv) || du != d1u || dv != d1v) continue;
                    if (pp.count >= kMaxUnits2) break;
                    used[t1] = used[t2] = true;
                    pp.tapA[pp.count] = t1; pp.tapB[pp.count] = t2; pp.grp[pp.count] = 0; ++pp.count;
                    break;
                }
            }
            bool any2 = false;
            if (p2 >= 0) {
                for (int t1 = 0; t1 < T; ++t1) {             // pairs at copy 1
                    if (used[t1] || !fits(t1, d1u, d1v)) continue;
                    for (int t2 = 0; t2 < T; ++t2) {
                        int du, dv;
                        if (t2 == t1 || used[t2] || !diff(t1, t2, &du, &dv) || du != d2u || dv != d2v) continue;
                        if (pp.count >= kMaxUnits2) break;
                        used[t1] = used[t2] = true; any2 = true;
                        pp.tapA[pp.count] = t1; pp.tapB[pp.count] = t2; pp.grp[pp.count] = 1; ++pp.count;
                        break;
                    }
                }
            }
            int units = pp.count;
            for (int t = 0; t < T; ++t) units += used[t] ? 0 : 1;
            if (units > kMaxUnits2 || units >= best_units) continue;
            for (int t = 0; t < T; ++t)
                if (!used[t]) { pp.tapA[pp.count] = t; pp.tapB[pp.count] = -1; pp.grp[pp.count] = 0; ++pp.count; }
            pp.ncopies = any2 ? 3 : 2;
            pp.cu[0] = 0; pp.cv[0] = 0; pp.cu[1] = d1u; pp.cv[1] = d1v;
            pp.cu[2] = d1u + d2u; pp.cv[2] = d1v + d2v;
            best = pp; best_units = units; found = true;
        }
    }
    if (found) *out = best;
    return found;
}

// Smallest flat pitch for one axis of the Z tile. The tile holds Z coordinates lo .. lo + P - 1 of
// every line, lines back to back, and an output at class coordinate c in [0, J) reads coordinate
// c + v for every shift v in [lo, hi]. A read that runs past the end of its line lands on the first
// cells of the next one, which is harmless exactly when both the coordinate it wants and the one it
// gets are outside [0, ext): the tensor map fills those with the convolution's zero padding either
// way. For a padded 3x3 layer this lets the right halo of one line double as the left halo of the
// next (P = J + 1 instead of J + 2). With a partial last block the tile is also kept in a copy
// that ends one coordinate earlier (ext - 1, see Tc2Params::nvar); `also_shorter` asks for a pitch
// that is right for both.
int min_flat_pitch(int J, int lo, int hi, int ext, bool also_shorter) {
    for (int P = J; P < J + (hi - lo); ++P) {
        bool ok = true;
        for (int e = ext; e >= ext - (also_shorter ? 1 : 0) && ok; --e)
            for (int c = 0; c < J && ok; ++c)
                for (int v = lo; v <= hi && ok; ++v) {
                    const int t = c + v - lo;
                    if (t < P) continue;
                    const int want = c + v, got = lo + t - P;
                    ok = (want < 0 || want >= e) && (got < 0 || got >= e) && t - P < P;
                }
        if (ok) return P;
    }
    return J + (hi - lo);
}

Tc2Geom build_geom2_with(const Dims& d, bool collapse, bool fill_rectangles, int bn_cap = 256) {
    Tc2Geom g{};
    Tc2Params& p = g.p;
    g.ok = false;
    if (d.dtype != AC_BF16 || d.layout != AC_NHWC) return g;
    // class rows advance Z by exactly one row: s | k (k/s classes), or k | s (one class, s/k phase planes of Z)
    if ((d.kh % d.sh != 0 && d.sh % d.kh != 0) || (d.kw % d.sw != 0 && d.sw % d.kw != 0)) return g;
    p.mh = d.sh % d.kh == 0 ? d.sh / d.kh : 1;
    p.mw = d.sw % d.kw == 0 ? d.sw / d.kw : 1;
    const bool planes = p.mh > 1 || p.mw > 1;
    if (planes && (collapse || p.mh > 2 || p.mw > 2 || d.H % d.kh != 0 || d.W % d.kw != 0)) return g;
    if (d.R * d.S > 64 || d.R > 16 || d.S > 16) return g;
    const UnitPlan up = plan_units(d.Ci, d.Co, d.R * d.S, kMaxUnits2, fill_rectangles, bn_cap);
    if (!up.ok) return g;
    p.c_h = d.kh % d.sh == 0 ? d.kh / d.sh : 1; p.c_w = d.kw % d.sw == 0 ? d.kw / d.sw : 1;
    p.ncls = p.c_h * p.c_w;
    if (p.ncls > kMaxClasses) return g;
    p.strided_map = p.ncls > kMaxClassMaps ? 1 : 0;
    if (d.Ho < p.c_h || d.Wo < p.c_w) return g;            // every class has at least one output
    p.Ci = d.Ci; p.Co = d.Co; p.R = d.R; p.S = d.S; p.sh = d.sh; p.sw = d.sw; p.ph = d.ph; p.pw = d.pw;
    p.kh = d.kh; p.kw = d.kw;
    p.dw_elems = d.dw_elems();
    int umin = 1 << 30, umax = -(1 << 30), vmin = 1 << 30, vmax = -(1 << 30);
    bool phase_h[2] = {false, false}, phase_w[2] = {false, false};
    for (int a = 0; a < p.c_h; ++a)
        for (int r = 0; r < d.R; ++r) {
            int ph_;
            const int u = tap_shift(d.sh, a, d.ph, r, d.kh, p.mh, &ph_);
            phase_h[ph_] = true;
            umin = u < umin ? u : umin; umax = u > umax ? u : umax;
        }
    for (int b = 0; b < p.c_w; ++b)
        for (int s = 0; s < d.S; ++s) {
            int ph_;
            const int v = tap_shift(d.sw, b, d.pw, s, d.kw, p.mw, &ph_);
            phase_w[ph_] = true;
            vmin = v < vmin ? v : vmin; vmax = v > vmax ? v : vmax;
        }
    p.umin = umin; p.vmin = vmin;
    g.uspan = umax - umin; g.vspan = vmax - vmin;
    const int I = (d.Ho + p.c_h - 1) / p.c_h, Jc = (d.Wo + p.c_w - 1) / p.c_w;
    p.Wzq = Jc + g.vspan;
    int rows_whole = I + g.uspan;     // rows per image when a K-tile holds whole images
    if (p.Wzq > 256) return g;
    p.CB = up.CB; p.ncgpc = up.ncgpc; p.ncib_total = up.ncib_total; p.BN = up.BN;
    p.nchunks = up.BN / 64;
    p.taps_per_group = up.taps_per_group; p.ntapgroups = up.ntapgroups;
    p.cibs_per_group = up.cibs_per_group; p.ncibgroups = up.ncibgroups; p.groups = up.groups;
    p.tmem_cols = up.tmem_cols;
    int chunksA = up.CB == 128 ? 2 * up.cibs_per_group : up.cibs_per_group + 1;
    // which copies of the Z tile are needed (see Tc2Params::nvar)
    p.rho_h = d.H % d.kh; p.rho_w = d.W % d.kw;
    p.Hp = d.Hp; p.Wp = d.Wp; p.Ho = d.Ho; p.Wo = d.Wo;
    bool var_used[4] = {false, false, false, false};
    for (int a = 0; a < p.c_h; ++a)
        for (int r = 0; r < d.R; ++r)
            for (int b = 0; b < p.c_w; ++b)
                for (int s_ = 0; s_ < d.S; ++s_) {
                    if (planes) {
                        int fh, fw;
                        tap_shift(d.sh, a, d.ph, r, d.kh, p.mh, &fh);
                        tap_shift(d.sw, b, d.pw, s_, d.kw, p.mw, &fw);
                        var_used[fh * 2 + fw] = true;
                        continue;
                    }
                    var_used[(reads_padding_in_partial_block(d.sh, a, d.ph, r, d.kh, d.Hp, p.rho_h, d.Ho) ? 2 : 0) +
                             (reads_padding_in_partial_block(d.sw, b, d.pw, s_, d.kw, d.Wp, p.rho_w, d.Wo) ? 1 : 0)] = true;
                }
    p.nvar = 0;
    for (int v = 0; v < 4; ++v) p.var_slot[v] = var_used[v] ? p.nvar++ : -1;
    if ((var_used[2] || var_used[3]) && d.Hp < 2) return g;
    if ((var_used[1] || var_used[3]) && d.Wp < 2) return g;
    // extent of the (largest) plane a line of the tile comes from, and whether a plane one shorter is in use too
    const int ext_h = (d.Hp + p.mh - 1) / p.mh, ext_w = (d.Wp + p.mw - 1) / p.mw;
    const bool short_h = planes ? (phase_h[1] && (d.Hp - 1 + p.mh - 1) / p.mh < ext_h) : (var_used[2] || var_used[3]);
    const bool short_w = planes ? (phase_w[1] && (d.Wp - 1 + p.mw - 1) / p.mw < ext_w) : (var_used[1] || var_used[3]);
    PairPlan pairs{};
    p.pair_mode = 0;
    if (kEnablePairs && !collapse && !planes && p.nvar == 1 && d.Ci == 64 && plan_pairs(d, p.c_h, p.c_w, umin, vmin, g.uspan, g.vspan, &pairs) &&
        pairs.count * up.BN <= 512) {
        p.pair_mode = 1;
        p.pu_count = pairs.count;
        p.ncopies = pairs.ncopies;
        for (int i = 0; i < 3; ++i) { p.copy_du[i] = pairs.cu[i]; p.copy_dv[i] = pairs.cv[i]; }
        chunksA = pairs.ncopies;
        p.taps_per_group = d.R * d.S; p.ntapgroups = 1; p.cibs_per_group = 1; p.ncibgroups = 1;
        p.groups = up.ncob;
        p.tmem_cols = 32;
        while (p.tmem_cols < (uint32_t)(pairs.count * up.BN)) p.tmem_cols *= 2;
    }

    // K-tile shape: Ic class rows of one image, or NB whole class images (then the gradient
    // tile keeps the input tile's row count per image so that both stay on one flat pitch;
    // the surplus rows are beyond the class's extent and arrive as zeros). Chosen by a cost
    // model of the busiest CTA's main loop (below).
    const int U = p.collapse ? p.cu_cap : (p.pair_mode ? pairs.count : up.units);
    const double mma_clk = up.BN >= 128 ? up.BN / 2.0 : 48.0;   // N = 64 is shared-memory-read bound
    p.collapse = 0;
    if (collapse) {
        // one accumulator tile per distinct Z shift of each class; needs every class on one copy of
        // the tile (k | H and k | W) and something to collapse
        if (p.nvar != 1) return g;
        int total = 0;
        for (int c = 0; c < p.ncls; ++c) {
            const ClassShifts cs = class_shifts(c, p.c_w, d.sh, d.sw, d.ph, d.pw, d.kh, d.kw, d.R, d.S);
            total += cs.nU * cs.nV;
        }
        if (total >= p.ncls * d.R * d.S || total > 65535 || p.ncls * d.R * d.S > 8192) return g;
        p.collapse = 1;
        p.cu_total = total;
        p.cu_cap = 512 / up.BN < kMaxUnits2 ? 512 / up.BN : kMaxUnits2;
        if (p.cu_cap > total) p.cu_cap = total;
        p.ntapgroups = (total + p.cu_cap - 1) / p.cu_cap;
        p.taps_per_group = d.R * d.S;   // not used for tiles in this mode
        p.cibs_per_group = 1; p.ncibgroups = up.ncib_total;
        p.groups = up.ncob * up.ncib_total * p.ntapgroups;
        chunksA = 2;
        p.tmem_cols = 32;
        while (p.tmem_cols < (uint32_t)(p.cu_cap * up.BN)) p.tmem_cols *= 2;
        p.slice_elems = (long long)up.ncob * up.ncib_total * total * up.BN * up.CB;
    }
    if (!p.pair_mode) {
        p.Wzq = min_flat_pitch(Jc, vmin, vmax, ext_w, short_w);
        rows_whole = min_flat_pitch(I, umin, umax, ext_h, short_h);
    }
    int best_Ic = 0, best_sb = 0, best_NB = 1;
    double best_cost = 1e30, best_eff = 0.0;
    {
        constexpr int want = 2;   // at least two gradient slots
        for (int Ic = 1; Ic <= I; ++Ic) {
            if (Ic + g.uspan > 256) break;
            if (p.strided_map && (p.c_h * (Ic + g.uspan) > 256 || p.c_w * p.Wzq > 256)) break;
            for (int NB = 1; NB <= (Ic == I ? 16 : 1) && NB <= d.N; ++NB) {
                const int rowsA = NB > 1 ? rows_whole : Ic + g.uspan;
                const int KT = ((NB == 1 ? Ic : NB * rowsA) * p.Wzq + 15) / 16 * 16;
                const int NCa = (KT + g.uspan * p.Wzq + g.vspan + 7) / 8 * 8;
                if ((uint32_t)NCa * 128 >= (1u << 18) || (uint32_t)KT * 128 >= (1u << 18)) break;
                const uint32_t a_slot = (uint32_t)p.nvar * chunksA * NCa * 128;
                const uint32_t b_slot = (uint32_t)p.nchunks * KT * 128;
                if (kSlotsA * a_slot + want * b_slot > kSmemBudget2) break;
                int sb = (int)((kSmemBudget2 - kSlotsA * a_slot) / b_slot);
                if (sb > kMaxSlotsB) sb = kMaxSlotsB;
                const int bands = (I + Ic - 1) / Ic;
                const double tiles_per_image = NB == 1 ? (double)bands : 1.0 / NB;
                // Two models of a K-tile's time, both fitted to measurements. Layers with several output
                // classes: a class tile costs max(MMA time, 400 + 80 cycles per MMA), times 1.1 when only
                // two gradient slots fit. Layers with ONE class (stride = k) change their input tile with
                // every gradient tile, and what they pay for is that change: the MMA time plus ~600
                // cycles per K-tile, never less than the ~2050 cycles of a TMA round trip (the input
                // ring is two deep), and no penalty for two gradient slots -- so they want tall tiles
                // (3x3 stride 2 on 56x56 at batch 128: 35.8 us with 4-row tiles, 32.5 us with 6-row ones).
                const double ks = KT / 16, mmas = (double)U * ks;
                double ktile;
                if (p.ncls == 1) {
                    ktile = mmas * mma_clk + 600.0;
                    if (ktile < 2050.0) ktile = 2050.0;
                } else {
                    const double tile = mmas * mma_clk > 400.0 + 80.0 * mmas ? mmas * mma_clk : 400.0 + 80.0 * mmas;
                    ktile = p.ncls * tile * (sb < 3 ? 1.1 : 1.0);
                }
                // what the slowest CTA does: K-tiles are dealt out whole, so the busiest K-slice
                // sets the time (448 tiles over 148 slices means 4 for some and 3 for most)
                const long long kts = NB > 1 ? (d.N + NB - 1) / NB : (long long)d.N * bands;
                long long spl = d.sms / p.groups < 1 ? 1 : d.sms / p.groups;
                if (spl > kts) spl = kts;
                const double cost = (double)((kts + spl - 1) / spl) * ktile;
                if (cost < best_cost * (1.0 - 1e-9)) {
                    best_cost = cost; best_Ic = Ic; best_sb = sb; best_NB = NB;
                    best_eff = (double)d.Ho * d.Wo / (tiles_per_image * p.ncls * KT);
                }
            }
        }
    }
    if (best_Ic == 0) return g;
    p.Ic = best_Ic;
    p.NB = best_NB;
    p.bands = (I + p.Ic - 1) / p.Ic;
    p.rowsA = p.NB > 1 ? rows_whole : p.Ic + g.uspan;
    p.rowsB = p.NB > 1 ? p.rowsA : p.Ic;
    p.KT = ((p.NB == 1 ? p.Ic : p.NB * p.rowsA) * p.Wzq + 15) / 16 * 16;
    p.ksteps = p.KT / 16;
    const int NCa = (p.KT + g.uspan * p.Wzq + g.vspan + 7) / 8 * 8;
    p.a_chunk_bytes = (uint32_t)NCa * 128;
    p.chunksA = chunksA;
    p.a_slot_bytes = (uint32_t)p.nvar * chunksA * p.a_chunk_bytes;
    if (p.pair_mode) {
        for (int u = 0; u < pairs.count; ++u) {
            p.pu_tapA[u] = (signed char)pairs.tapA[u];
            p.pu_tapB[u] = (signed char)pairs.tapB[u];
            const int gq = pairs.grp[u], t = pairs.tapA[u], r = t / d.S, sx = t % d.S;
            for (int c = 0; c < p.ncls; ++c) {
                const int a = c / p.c_w, b = c % p.c_w;
                const int ouA = floor_div_i(d.sh * a - d.ph + r, d.kh) - umin - pairs.cu[gq];
                const int ovA = floor_div_i(d.sw * b - d.pw + sx, d.kw) - vmin - pairs.cv[gq];
                p.pu_off[c][u] = (uint32_t)gq * p.a_chunk_bytes + (uint32_t)(ouA * p.Wzq + ovA) * 128u;
            }
        }
    }
    p.b_chunk_bytes = (uint32_t)p.KT * 128;
    p.b_slot_bytes = (uint32_t)p.nchunks * p.b_chunk_bytes;
    p.a_box_bytes = 128u * p.Wzq * p.rowsA * p.NB;
    p.b_box_bytes = 128u * p.Wzq * p.rowsB * p.NB;
    p.slotsB = best_sb;
    g.k_eff = best_eff;
    const long long ktiles = p.NB > 1 ? (d.N + p.NB - 1) / p.NB : (long long)d.N * p.bands;
    if (ktiles >= (1ll << 30)) return g;
    p.ktiles = (int)ktiles;
    int splits = d.sms / p.groups;
    if (splits < 1) splits = 1;
    if (splits > p.ktiles) splits = p.ktiles;
    {
        // K-tiles are dealt out whole, so the busiest slice has ceil(ktiles / splits) of them: no more
        // slices than that number needs (896 tiles: 128 slices of 7 finish when 148 slices of 6 or 7
        // do, with fewer partial sums to write and reduce, and leave SMs to other streams)
        const int per_slice = (p.ktiles + splits - 1) / splits;
        splits = (p.ktiles + per_slice - 1) / per_slice;
    }
    p.splits = splits;
    p.chunk_kt = 0;
    if (d.max_chain > 0) {
        // MMA instructions that add into one accumulator per K-tile: every class's, or, collapsed,
        // those of the tile's own class
        const int adds_per_ktile = (p.collapse ? 1 : p.ncls) * p.ksteps;
        p.chunk_kt = d.max_chain / adds_per_ktile > 1 ? d.max_chain / adds_per_ktile : 1;
    }
    g.smem_bytes = kSlotsA * p.a_slot_bytes + p.slotsB * p.b_slot_bytes + 1024;
    if (g.smem_bytes < 120 * 1024) g.smem_bytes = 120 * 1024;   // one CTA per SM: TMEM is not shared
    g.cta_cycles = best_cost;
    g.ok = true;
    return g;
}

// Two ways to deal the accumulator tiles to CTAs (see plan_units): taps of one channel block per
// CTA, or taps x channel-blocks rectangles that leave no CTA half empty but need a larger input
// tile in shared memory (hence shorter K-tiles when several copies of it are kept). The cost
// model's time for the busiest CTA decides.
Tc2Geom build_geom2(const Dims& d, bool collapse) {
    const Tc2Geom a = build_geom2_with(d, collapse, false);
    if (collapse) return a;
    const Tc2Geom b = build_geom2_with(d, collapse, true);
    Tc2Geom best = !a.ok ? b : (!b.ok ? a : (b.cta_cycles < a.cta_cycles ? b : a));
    if (best.ok && best.p.nvar > 1 && best.p.BN > 128) {
        // several copies of the input tile (partial pooling blocks): a narrower output-channel block
        // may leave room for longer K-tiles
        for (int fill = 0; fill < 2; ++fill) {
            const Tc2Geom c = build_geom2_with(d, collapse, fill != 0, 128);
            if (c.ok && c.cta_cycles < best.cta_cycles) best = c;
        }
    }
    return best;
}

// The geometry is pure arithmetic on the descriptor but not free (the pairing search):
// the last few descriptors are remembered, so that the planning calls of one
// ac_conv2d_wgrad_compressed (workspace size, support test, launch) and repeated layers pay once.
Tc2Geom make_geom2(const Dims& d, bool collapse = false) {
    constexpr int kEntries = 16;
    static std::mutex mu;
    static Dims keys[2][kEntries];
    static Tc2Geom vals[2][kEntries];
    static int used[2] = {0, 0}, next[2] = {0, 0};
    const int w = collapse ? 1 : 0;
    {
        std::lock_guard<std::mutex> lock(mu);
        for (int i = 0; i < used[w]; ++i)
            if (std::memcmp(&keys[w][i], &d, sizeof(Dims)) == 0) return vals[w][i];
    }
    const Tc2Geom g = build_geom2(d, collapse);
    std::lock_guard<std::mutex> lock(mu);
    keys[w][next[w]] = d; vals[w][next[w]] = g;
    next[w] = (next[w] + 1) % kEntries;
    if (used[w] < kEntries) ++used[w];
    return g;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

// Looked up once; the initialisation of a function-local static is thread-safe.
EncodeTiledFn encode_fn() {
    static const EncodeTiledFn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            return reinterpret_cast<EncodeTiledFn>(f);
        return static_cast<EncodeTiledFn>(nullptr);
    }();
    return fn;
}

static_assert(sizeof(Tc2Params) <= 4000, "kernel parameters must stay below the 4 KB limit");

}  // namespace

ac_status launch_bounded_wait_selftest(void* workspace, long long limit_cycles, cudaStream_t stream) {
    bounded_wait_selftest_kernel<<<1, 64, 0, stream>>>(static_cast<uint32_t*>(workspace), limit_cycles);
    AC_CUDA_TRY(cudaGetLastError());
    return AC_OK;
}

bool tc2_supported(const Dims& d, double* k_eff) {
    const Tc2Geom g = make_geom2(d);
    if (g.ok && k_eff) *k_eff = g.k_eff;
    return g.ok;
}

void plan_tc2(const Dims& d, WgradPlan* pl) {
    const Tc2Geom g = make_geom2(d);
    pl->path = PATH_TC2;
    pl->splits = g.p.splits;
    pl->tc_band = g.p.Ic * g.p.c_h;
    pl->tc_groups = g.p.groups;
    pl->tc_ktiles = g.p.ktiles;
    pl->tc_stages = g.p.slotsB;
    pl->bytes = kStatusBlockBytes + (g.p.splits > 1 ? (size_t)g.p.splits * d.dw_elems() * 4 : 0);
}

void tc2_plan_info(const Dims& d, ac_plan_info* info) {
    const Tc2Geom g = make_geom2(d);
    info->tensor_core = 2;
    info->splits = g.p.splits;
    info->ctas = g.p.splits * g.p.groups;
    info->groups = g.p.groups;
    info->band_rows = g.p.Ic * g.p.c_h;
    info->k_tile = g.p.KT;
    info->row_pitch = g.p.Wzq;
    info->stages = g.p.slotsB;
    info->smem_bytes = (int32_t)g.smem_bytes;
    info->tmem_columns = (int32_t)g.p.tmem_cols;
    info->units_per_cta = g.p.pair_mode ? g.p.pu_count : g.p.cibs_per_group * g.p.taps_per_group;
    info->block_n = g.p.BN;
    info->a_cells = (int32_t)(g.p.a_chunk_bytes / 128);
    info->phases = g.p.ncls;
}

static ac_status launch_tc2_any(const Dims& d, bool collapse, const void* z, const void* dy, float* dw,
                                void* workspace, cudaStream_t stream, bool keep_status = false) {
    Tc2Geom g = make_geom2(d, collapse);
    if (!g.ok) return AC_ERR_UNSUPPORTED;
    Tc2Params& p = g.p;
    p.keep_status = keep_status ? 1 : 0;
    EncodeTiledFn enc = encode_fn();
    if (!enc) return AC_ERR_CUDA;
    for (int var = 0; var < 4; ++var) {
        if (p.var_slot[var] < 0) continue;
        // Z viewed as (Ci, Wp, Hp, N); one copy brings 64 channels of a (rows x Wzq) window.
        // Variants 1-3 end one column and/or one row early: the partial last block reads as zero.
        cuuint64_t dims[4] = {(cuuint64_t)d.Ci, (cuuint64_t)(d.Wp - (var & 1)),
                              (cuuint64_t)(d.Hp - (var >> 1)), (cuuint64_t)d.N};
        cuuint64_t strides[3] = {(cuuint64_t)d.Ci * 2, (cuuint64_t)d.Wp * d.Ci * 2,
                                 (cuuint64_t)d.Hp * d.Wp * d.Ci * 2};
        const char* zbase = static_cast<const char*>(z);
        if (p.mh > 1 || p.mw > 1) {
            // phase plane (fh, fw): rows fh, fh + mh, ... and columns fw, fw + mw, ... of Z
            const int fh = var >> 1, fw = var & 1;
            if (fh >= p.mh || fw >= p.mw || fh >= d.Hp || fw >= d.Wp) return AC_ERR_UNSUPPORTED;
            dims[1] = (cuuint64_t)((d.Wp - fw + p.mw - 1) / p.mw);
            dims[2] = (cuuint64_t)((d.Hp - fh + p.mh - 1) / p.mh);
            strides[0] = (cuuint64_t)p.mw * d.Ci * 2;
            strides[1] = (cuuint64_t)p.mh * d.Wp * d.Ci * 2;
            zbase += ((size_t)fh * d.Wp + fw) * d.Ci * 2;
        }
        const cuuint32_t box[4] = {64, (cuuint32_t)p.Wzq, (cuuint32_t)p.rowsA, (cuuint32_t)p.NB};
        const cuuint32_t es[4] = {1, 1, 1, 1};
        if (enc(&p.tmA[var], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<char*>(zbase), dims, strides, box, es,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return AC_ERR_CUDA;
    }
    if (p.strided_map) {
        const cuuint64_t dims[4] = {(cuuint64_t)d.Co, (cuuint64_t)d.Wo, (cuuint64_t)d.Ho, (cuuint64_t)d.N};
        const cuuint64_t strides[3] = {(cuuint64_t)d.Co * 2, (cuuint64_t)d.Wo * d.Co * 2,
                                       (cuuint64_t)d.Ho * d.Wo * d.Co * 2};
        // the box spans c_w * Wzq columns and c_h * rowsB rows of dY, of which every c_w-th / c_h-th is taken
        const cuuint32_t box[4] = {64, (cuuint32_t)(p.c_w * p.Wzq), (cuuint32_t)(p.c_h * p.rowsB), (cuuint32_t)p.NB};
        const cuuint32_t es[4] = {1, (cuuint32_t)p.c_w, (cuuint32_t)p.c_h, 1};
        if (enc(&p.tmBs, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(dy), dims, strides, box, es,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return AC_ERR_CUDA;
    }
    for (int a = 0; a < p.c_h && !p.strided_map; ++a)
        for (int b = 0; b < p.c_w; ++b) {
            // class (a,b): outputs ho = c_h*i + a, wo = c_w*j + b
            const int Ia = (d.Ho - a + p.c_h - 1) / p.c_h, Jb = (d.Wo - b + p.c_w - 1) / p.c_w;
            const cuuint64_t dims[4] = {(cuuint64_t)d.Co, (cuuint64_t)Jb, (cuuint64_t)Ia, (cuuint64_t)d.N};
            const cuuint64_t strides[3] = {(cuuint64_t)p.c_w * d.Co * 2, (cuuint64_t)p.c_h * d.Wo * d.Co * 2,
                                           (cuuint64_t)d.Ho * d.Wo * d.Co * 2};
            const cuuint32_t box[4] = {64, (cuuint32_t)p.Wzq, (cuuint32_t)p.rowsB, (cuuint32_t)p.NB};
            const cuuint32_t es[4] = {1, 1, 1, 1};
            char* base = static_cast<char*>(const_cast<void*>(dy)) + ((size_t)a * d.Wo + b) * d.Co * 2;
            if (enc(&p.tmB[a * p.c_w + b], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, es,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                return AC_ERR_CUDA;
        }
    p.status = static_cast<uint32_t*>(workspace);
    float* partials = reinterpret_cast<float*>(static_cast<char*>(workspace) + kStatusBlockBytes);
    p.out = (p.splits > 1 || p.collapse) ? partials : dw;
    static bool attr_done[64] = {};
    {
        const ac_status st_ = ensure_smem_limit(wgrad_tc2_kernel, (int)(kSmemBudget2 + 1024), attr_done);
        if (st_ != AC_OK) return st_;
    }
    record_timing_hook(0, stream);
    launch_after(wgrad_tc2_kernel, dim3(p.groups * p.splits), dim3(kThreads2), g.smem_bytes, stream, p);
    record_timing_hook(1, stream);
    AC_CUDA_TRY(cudaGetLastError());
    if (p.collapse) {
        CollapseReduceParams q;
        q.splits = p.splits; q.ncls = p.ncls; q.R = d.R; q.S = d.S; q.Ci = d.Ci; q.CB = p.CB; q.BN = p.BN;
        q.ncib_total = p.ncib_total; q.cu_total = p.cu_total; q.c_w = p.c_w; q.sh = d.sh; q.sw = d.sw;
        q.ph = d.ph; q.pw = d.pw; q.kh = d.kh; q.kw = d.kw; q.slice_elems = p.slice_elems; q.elems4 = p.dw_elems / 4;
        const int pairs = p.ncls * p.splits;
        int sl = 1;
        while (sl < 32 && q.elems4 * sl < 148 * 1024 && sl * 4 <= pairs) sl *= 2;
        switch (sl) {
            case 1: launch_collapsed_reduce<1>(partials, q, dw, stream); break;
            case 2: launch_collapsed_reduce<2>(partials, q, dw, stream); break;
            case 4: launch_collapsed_reduce<4>(partials, q, dw, stream); break;
            case 8: launch_collapsed_reduce<8>(partials, q, dw, stream); break;
            case 16: launch_collapsed_reduce<16>(partials, q, dw, stream); break;
            default: launch_collapsed_reduce<32>(partials, q, dw, stream); break;
        }
        AC_CUDA_TRY(cudaGetLastError());
        return AC_OK;
    }
    if (p.splits > 1) return launch_splitk_reduce(partials, p.splits, p.dw_elems, dw, stream);
    return AC_OK;
}

ac_status launch_wgrad_tc2(const Dims& d, const WgradPlan& pl, const void* z, const void* dy,
                           float* dw, void* workspace, cudaStream_t stream, bool keep_status) {
    (void)pl;
    return launch_tc2_any(d, false, z, dy, dw, workspace, stream, keep_status);
}

// MMA instructions that add into one accumulator over a CTA's whole K-slice
int tc2_chain_length(const Dims& d) {
    const Tc2Geom g = make_geom2(d);
    if (!g.ok) return 0;
    return (g.p.ktiles + g.p.splits - 1) / g.p.splits * g.p.ncls * g.p.ksteps;
}

// The cost model's main-loop time (cycles) of the busiest CTA, and how many copies of the input tile
// the plan keeps (more than one: partial pooling blocks next to the padding). Negative: not supported.
double tc2_cost_cycles(const Dims& d, int* tile_copies) {
    const Tc2Geom g = make_geom2(d);
    if (!g.ok) return -1.0;
    if (tile_copies) *tile_copies = g.p.nvar;
    return g.cta_cycles;
}

// Collapsed form: same dW, fewer MMAs (see Tc2Params::collapse). 0 bytes / AC_ERR_UNSUPPORTED when the
// problem has nothing to collapse or the TMA-fed kernel does not take it.
size_t tc2_collapsed_workspace_bytes(const Dims& d, int* tiles_collapsed, int* tiles_dense) {
    const Tc2Geom g = make_geom2(d, true);
    if (!g.ok) return 0;
    if (tiles_collapsed) *tiles_collapsed = g.p.cu_total;
    if (tiles_dense) *tiles_dense = g.p.ncls * d.R * d.S;
    return kStatusBlockBytes + (size_t)g.p.splits * g.p.slice_elems * 4;
}

ac_status launch_wgrad_tc2_collapsed(const Dims& d, const void* z, const void* dy, float* dw,
                                     void* workspace, cudaStream_t stream) {
    return launch_tc2_any(d, true, z, dy, dw, workspace, stream);
}

}  // namespace ac
