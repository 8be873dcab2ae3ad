// Compressed weight gradient on the 5th-generation tensor cores (tcgen05, TMEM).
//
// dW[co,r,s,ci] = sum_{n,ho,wo} dY[n,ho,wo,co] * Xt[n, ho*sh-ph+r, wo*sw-pw+s, ci]
// with Xt the inflated Z of Section 4 of the paper (each pooled value stands
// for its k x k block) and 0 in the convolution's padding. bf16 inputs, NHWC,
// fp32 accumulation in tensor memory.
//
// Implicit GEMM, D[M = 128 input channels of one filter tap][N = output channels]
// += A[M][K] * B[K][N] with K = output positions:
//   * B (dY) tile: positions of a band of `hb` output rows of one image, laid
//     out flat with row pitch Wq >= Wo; the surplus columns hold zeros.
//   * A (Xt) tile: ONE inflated halo grid per stride phase, same row pitch Wq.
//     Because A and B share the pitch, filter tap (r,s) is the same grid read
//     at a constant cell offset, so the nine taps of a 3x3 filter need no
//     im2col copies: the MMA's shared-memory descriptor just starts
//     `tap_offset * 16` bytes further. This needs a layout whose start address
//     can move in 16-byte steps, which is the un-swizzled MN-major canonical
//     layout: [8-channel group][cell][8 channels], cells 16 bytes apart.
//   * The inflation h/k, w/k and the zero padding are applied by the producer
//     warps while they fill the grid from Z; Xt never exists in global memory.
// One thread issues tcgen05.mma; accumulators for all taps a CTA owns live in
// TMEM (up to 512 columns); four warps drain them with tcgen05.ld at the end.
// K is split over CTAs; partial dW tensors are summed by the split-K reduce.
#include "ac_common.h"
#include "tc_ptx.cuh"

namespace ac {
namespace {

constexpr int kProducerWarps = 8;
constexpr int kProducerThreads = kProducerWarps * 32;
constexpr int kThreads = kProducerThreads + 32;   // + the MMA-issuing warp
constexpr int kMaxStages = 8;
constexpr int kMaxUnits = 8;                       // accumulator tiles per CTA
constexpr uint32_t kSmemBudget = 220 * 1024;

struct TcParams {
    const __nv_bfloat16* z;
    const __nv_bfloat16* dy;
    float* out;            // partial tensors [splits][dW] or dW itself
    uint32_t* status;      // [0] != 0: a wait timed out; [1]: which
    int N, Ci, Co, H, W, R, S, sh, sw, ph, pw, k, Hp, Wp, Ho, Wo;
    int Wq, hb, bands, KT, NC, GH;
    int dr_min, dc_min;
    int nph, phase_slot[4], phase_a[4], phase_b[4];
    int CB, ncgpc, ncib_total, BN;
    int taps_per_group, ntapgroups, cibs_per_group, ncibgroups, ncob;
    int groups, splits, ktiles;
    int stages;
    uint32_t a_stage_bytes, b_stage_bytes, sbo_a, sbo_b, ph_bytes, tmem_cols;
    long long dw_elems;
};

using namespace tc;

__device__ __forceinline__ int floor_div(int a, int b) {
    int q = a / b;
    return (a % b != 0 && ((a < 0) != (b < 0))) ? q - 1 : q;
}

extern __shared__ __align__(1024) unsigned char tc_smem[];

__global__ void __launch_bounds__(kThreads, 1) wgrad_tc_kernel(const __grid_constant__ TcParams p) {
    __shared__ uint64_t full_bar[kMaxStages];
    __shared__ uint64_t empty_bar[kMaxStages];
    __shared__ uint64_t done_bar;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    volatile int* abort_flag = &abort_s;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int group = blockIdx.x % p.groups, split = blockIdx.x / p.groups;
    const int tg = group % p.ntapgroups;
    const int cibg = (group / p.ntapgroups) % p.ncibgroups;
    const int cob = group / (p.ntapgroups * p.ncibgroups);
    const int RS = p.R * p.S;
    const int tap0 = tg * p.taps_per_group;
    const int ntap = min(p.taps_per_group, RS - tap0);
    const int cib0 = cibg * p.cibs_per_group;
    const int ncib = min(p.cibs_per_group, p.ncib_total - cib0);
    const int co0 = cob * p.BN;
    const int kt_begin = (int)((long long)p.ktiles * split / p.splits);
    const int kt_end = (int)((long long)p.ktiles * (split + 1) / p.splits);
    const uint32_t stage_bytes = p.a_stage_bytes + p.b_stage_bytes;
    const uint32_t smem_base = smem_u32(tc_smem);

    if (tid == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(&full_bar[s], kProducerThreads);
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(&done_bar, 1);
        abort_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kProducerWarps) tmem_alloc(&tmem_base_s, p.tmem_cols);
    if (warp < kProducerWarps) {
        // Cells past the last grid row (read by the last K steps of the last taps)
        // and positions past the last tile row are never written again: zero them
        // once so that they are finite (they only ever meet zeros of the other operand).
        const int tailA = p.NC - p.GH * p.Wq, tailB = p.KT - p.hb * p.Wq;
        const int planesA_all = (int)(p.a_stage_bytes / p.sbo_a);
        const uint4 zero4 = make_uint4(0, 0, 0, 0);
        for (int s = 0; s < p.stages; ++s) {
            unsigned char* a_st = tc_smem + (size_t)s * stage_bytes;
            unsigned char* b_st = a_st + p.a_stage_bytes;
            for (int e = tid; e < planesA_all * tailA; e += kProducerThreads) {
                const int pl = e / tailA, c = p.GH * p.Wq + (e - pl * tailA);
                *reinterpret_cast<uint4*>(a_st + (size_t)pl * p.sbo_a + (size_t)c * 16) = zero4;
            }
            for (int e = tid; e < (p.BN / 8) * tailB; e += kProducerThreads) {
                const int pl = e / tailB, q = p.hb * p.Wq + (e - pl * tailB);
                *reinterpret_cast<uint4*>(b_st + (size_t)pl * p.sbo_b + (size_t)q * 16) = zero4;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;

    if (warp < kProducerWarps) {
        // ------------------------------------------------------------ producers
        // A K-tile is filled row by row. A "job" is one row of one plane group
        // (8 planes = 64 channels): first the rows of the inflated input grid(s),
        // then the rows of the output-gradient tile. A warp step covers 4 cells x
        // 8 planes (lane = plane + 8 * cell): 128 contiguous bytes per cell from
        // global memory, and 8 planes x 16 bytes = all 32 banks per quarter warp
        // in shared memory (plane strides are odd multiples of 16 bytes).
        // Steps are dealt round-robin to the warps and handled kBatch at a time:
        // all loads of a batch are issued before its first store.
        constexpr int kBatch = 8;
        const int cgh_n = ncib * p.ncgpc / 8;          // plane groups of the input grid
        const int cogh_n = p.BN / 64;                  // plane groups of the gradient tile
        const int jobsA = p.nph * p.GH * cgh_n;
        const int jobs = jobsA + p.hb * cogh_n;
        const int cpr = (p.Wq + 3) >> 2;               // warp steps per row
        const int steps = jobs * cpr;
        const int cgl = lane & 7, jl = lane >> 3;
        const uint4 zero4 = make_uint4(0, 0, 0, 0);
        const __nv_bfloat16* zsrc = p.z + cib0 * p.CB + cgl * 8;
        const __nv_bfloat16* gsrc = p.dy + co0 + cgl * 8;
        for (int kt = kt_begin, it = 0; kt < kt_end; ++kt, ++it) {
            const int s = it % p.stages;
            const uint32_t ph = (uint32_t)(it / p.stages) & 1u;
            if (it >= p.stages && !mbar_wait(&empty_bar[s], ph ^ 1u, abort_flag)) {
                if (atomicExch((int*)&abort_s, 1) == 0) { p.status[1] = 0x100u + s; atomicExch(&p.status[0], 1u); }
                break;
            }
            const int n = kt / p.bands, band = kt - n * p.bands;
            const int ho0 = band * p.hb;
            unsigned char* a_st = tc_smem + (size_t)s * stage_bytes;
            unsigned char* b_st = a_st + p.a_stage_bytes;
            int job = warp / cpr, chunk = warp - job * cpr;     // step `warp`, then += kProducerWarps
            for (int st0 = warp; st0 < steps; st0 += kProducerWarps * kBatch) {
                uint4 v[kBatch];
                unsigned char* dst[kBatch];
#pragma unroll
                for (int b = 0; b < kBatch; ++b) {
                    dst[b] = nullptr;
                    v[b] = zero4;
                    if (st0 + b * kProducerWarps < steps) {
                        const int gj = chunk * 4 + jl;
                        const __nv_bfloat16* src = nullptr;
                        if (job < jobsA) {
                            const int slot = job / (p.GH * cgh_n);
                            const int rem = job - slot * (p.GH * cgh_n);
                            const int gi = rem / cgh_n, cgh = rem - gi * cgh_n;
                            const int hx = p.sh * (ho0 + p.dr_min + gi) + p.phase_a[slot];
                            const int wx = p.sw * (p.dc_min + gj) + p.phase_b[slot];
                            if (gj < p.Wq) {
                                dst[b] = a_st + (size_t)slot * p.ph_bytes +
                                         (size_t)(cgh * 8 + cgl) * p.sbo_a + (size_t)(gi * p.Wq + gj) * 16;
                                if (hx >= 0 && hx < p.H && wx >= 0 && wx < p.W)
                                    src = zsrc + (((long long)n * p.Hp + hx / p.k) * p.Wp + wx / p.k) * p.Ci +
                                          cgh * 64;
                            }
                        } else {
                            const int jb = job - jobsA;
                            const int i = jb / cogh_n, cogh = jb - i * cogh_n;
                            const int ho = ho0 + i;
                            if (gj < p.Wq) {
                                dst[b] = b_st + (size_t)(cogh * 8 + cgl) * p.sbo_b + (size_t)(i * p.Wq + gj) * 16;
                                if (ho < p.Ho && gj < p.Wo)
                                    src = gsrc + (((long long)n * p.Ho + ho) * p.Wo + gj) * p.Co + cogh * 64;
                            }
                        }
                        if (src) v[b] = __ldg(reinterpret_cast<const uint4*>(src));
                    }
                    chunk += kProducerWarps;
                    while (chunk >= cpr) { chunk -= cpr; ++job; }
                }
#pragma unroll
                for (int b = 0; b < kBatch; ++b)
                    if (dst[b]) *reinterpret_cast<uint4*>(dst[b]) = v[b];
            }
            fence_proxy_async_smem();   // generic-proxy stores -> visible to the tensor core's reads
            mbar_arrive(&full_bar[s]);
        }
    } else if (lane == 0) {
        // ----------------------------------------------------------- MMA issuer
        uint32_t u_aoff[kMaxUnits], u_col[kMaxUnits];
        int nunits = 0;
        for (int cl = 0; cl < ncib; ++cl) {
            for (int t = 0; t < ntap; ++t) {
                const int tap = tap0 + t;
                const int r = tap / p.S, sx = tap - r * p.S;
                const int dr = floor_div(r - p.ph, p.sh), a = (r - p.ph) - dr * p.sh;
                const int dc = floor_div(sx - p.pw, p.sw), b = (sx - p.pw) - dc * p.sw;
                const int slot = p.phase_slot[a * 2 + b];
                const int tapoff = (dr - p.dr_min) * p.Wq + (dc - p.dc_min);
                u_aoff[nunits] = (uint32_t)slot * p.ph_bytes + (uint32_t)(cl * p.ncgpc) * p.sbo_a +
                                 (uint32_t)tapoff * 16u;
                u_col[nunits] = tmem_base + (uint32_t)nunits * p.BN;
                ++nunits;
            }
        }
        const uint32_t idesc = make_idesc(p.BN);
        const int ksteps = p.KT / 16;
        bool ok = true;
        for (int kt = kt_begin, it = 0; kt < kt_end; ++kt, ++it) {
            const int s = it % p.stages;
            const uint32_t ph = (uint32_t)(it / p.stages) & 1u;
            if (!mbar_wait(&full_bar[s], ph, abort_flag)) {
                if (atomicExch((int*)&abort_s, 1) == 0) { p.status[1] = 0x200u + s; atomicExch(&p.status[0], 1u); }
                ok = false;
                break;
            }
            tc_fence_after();
            const uint32_t a_st = smem_base + (uint32_t)s * stage_bytes;
            const uint32_t b_st = a_st + p.a_stage_bytes;
            for (int u = 0; u < nunits; ++u) {
                for (int kk = 0; kk < ksteps; ++kk) {
                    const uint64_t ad = make_desc(a_st + u_aoff[u] + kk * 256, 128, p.sbo_a);
                    const uint64_t bd = make_desc(b_st + kk * 256, 128, p.sbo_b);
                    mma_bf16(u_col[u], ad, bd, idesc, (it > 0 || kk > 0) ? 1u : 0u);
                }
            }
            mma_commit(&empty_bar[s]);   // frees the stage when these MMAs have read it
        }
        if (ok) mma_commit(&done_bar);
    }
    __syncwarp();

    // ---------------------------------------------------------------- epilogue
    if (warp < 4) {
        bool ok = mbar_wait(&done_bar, 0, abort_flag);
        if (!ok && atomicExch((int*)&abort_s, 1) == 0) { p.status[1] = 0x300u; atomicExch(&p.status[0], 1u); }
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
            tc_fence_after();
            const int m = warp * 32 + lane;          // accumulator row = TMEM lane
            float* dst = p.out + (long long)split * p.dw_elems;
            int u = 0;
            for (int cl = 0; cl < ncib; ++cl) {
                const int ci = (cib0 + cl) * p.CB + m;
                for (int t = 0; t < ntap; ++t, ++u) {
                    const int tap = tap0 + t;
                    for (int c0 = 0; c0 < p.BN; c0 += 32) {
                        uint32_t r[32];
                        tmem_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(u * p.BN + c0), r);
                        if (m < p.CB) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                const long long o = ((long long)(co0 + c0 + j) * RS + tap) * p.Ci + ci;
                                dst[o] = __uint_as_float(r[j]);
                            }
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kProducerWarps) tmem_dealloc(tmem_base, p.tmem_cols);
}

// ------------------------------------------------------------------ host side
struct TcGeom {
    TcParams p;
    uint32_t smem_bytes;
    bool ok;
};

int floor_div_h(int a, int b) {
    int q = a / b;
    return (a % b != 0 && ((a < 0) != (b < 0))) ? q - 1 : q;
}

TcGeom make_geom(const Dims& d) {
    TcGeom g{};
    TcParams& p = g.p;
    g.ok = false;
    if (d.dtype != AC_BF16 || d.layout != AC_NHWC) return g;
    if (d.Ci % 64 != 0 || d.Co % 64 != 0) return g;
    if (d.kh != d.kw) return g;      // the producer warps' index map knows square pooling blocks only
    if (d.sh < 1 || d.sh > 2 || d.sw < 1 || d.sw > 2) return g;
    if (d.R * d.S > 64) return g;
    p.N = d.N; p.Ci = d.Ci; p.Co = d.Co; p.H = d.H; p.W = d.W; p.R = d.R; p.S = d.S;
    p.sh = d.sh; p.sw = d.sw; p.ph = d.ph; p.pw = d.pw; p.k = d.k; p.Hp = d.Hp; p.Wp = d.Wp;
    p.Ho = d.Ho; p.Wo = d.Wo;
    p.dw_elems = d.dw_elems();
    // tap (r,s) of output (ho,wo) reads phase grid (a,b) at (ho+dr, wo+dc):
    // r - ph = sh*dr + a, s - pw = sw*dc + b
    const int dr_min = floor_div_h(0 - d.ph, d.sh), dr_max = floor_div_h(d.R - 1 - d.ph, d.sh);
    const int dc_min = floor_div_h(0 - d.pw, d.sw), dc_max = floor_div_h(d.S - 1 - d.pw, d.sw);
    const int drspan = dr_max - dr_min, dcspan = dc_max - dc_min;
    p.dr_min = dr_min; p.dc_min = dc_min;
    for (int i = 0; i < 4; ++i) p.phase_slot[i] = -1;
    p.nph = 0;
    for (int r = 0; r < d.R; ++r)
        for (int s = 0; s < d.S; ++s) {
            const int a = (r - d.ph) - floor_div_h(r - d.ph, d.sh) * d.sh;
            const int b = (s - d.pw) - floor_div_h(s - d.pw, d.sw) * d.sw;
            if (p.phase_slot[a * 2 + b] < 0) {
                p.phase_slot[a * 2 + b] = p.nph;
                p.phase_a[p.nph] = a; p.phase_b[p.nph] = b;
                ++p.nph;
            }
        }
    p.Wq = d.Wo + dcspan;
    p.CB = (d.Ci % 128 == 0) ? 128 : 64;
    p.ncgpc = p.CB / 8;
    p.ncib_total = d.Ci / p.CB;
    p.BN = d.Co <= 256 ? d.Co : (d.Co % 256 == 0 ? 256 : (d.Co % 128 == 0 ? 128 : 64));
    p.ncob = d.Co / p.BN;
    const int U = 512 / p.BN;   // accumulator tiles that fit in tensor memory
    const int ntaps = d.R * d.S;
    if (ntaps <= U) {
        p.ntapgroups = 1;
        p.taps_per_group = ntaps;
        p.cibs_per_group = U / ntaps < p.ncib_total ? U / ntaps : p.ncib_total;
    } else {
        p.ntapgroups = (ntaps + U - 1) / U;
        p.taps_per_group = (ntaps + p.ntapgroups - 1) / p.ntapgroups;
        p.ntapgroups = (ntaps + p.taps_per_group - 1) / p.taps_per_group;
        p.cibs_per_group = 1;
    }
    if (p.cibs_per_group * p.taps_per_group > kMaxUnits) return g;
    p.ncibgroups = (p.ncib_total + p.cibs_per_group - 1) / p.cibs_per_group;
    p.groups = p.ncob * p.ncibgroups * p.ntapgroups;
    uint32_t cols = (uint32_t)(p.cibs_per_group * p.taps_per_group * p.BN);
    p.tmem_cols = 32;
    while (p.tmem_cols < cols) p.tmem_cols *= 2;
    if (p.tmem_cols > 512) return g;

    // band height: best K efficiency among the choices that leave >= 3 stages
    // (>= 2 if nothing does); planes get an odd number of 16-byte cells so that
    // eight planes written at the same cell hit distinct shared-memory banks
    const int planesA = p.cibs_per_group * p.ncgpc + (p.CB == 64 ? 8 : 0);
    int best_hb = 0, best_stages = 0;
    double best_eff = -1.0;
    for (int want = 3; want >= 2 && best_hb == 0; --want) {
        for (int hb = 1; hb <= d.Ho; ++hb) {
            const int KT = (hb * p.Wq + 15) / 16 * 16;
            const int NC = KT + drspan * p.Wq + dcspan;
            const uint32_t sbo_a = (uint32_t)(NC | 1) * 16, sbo_b = (uint32_t)(KT | 1) * 16;
            const uint32_t a_bytes = (uint32_t)p.nph * planesA * sbo_a;
            const uint32_t b_bytes = (uint32_t)(p.BN / 8) * sbo_b;
            const uint32_t st = (a_bytes + b_bytes + 127) / 128 * 128;
            if (sbo_a >= (1u << 18) || sbo_b >= (1u << 18)) break;
            int stages = (int)(kSmemBudget / st);
            if (stages < want) break;
            if (stages > kMaxStages) stages = kMaxStages;
            const int bands = (d.Ho + hb - 1) / hb;
            const double eff = (double)d.Ho * d.Wo / ((double)bands * KT);
            if (eff > best_eff + 1e-9 || (eff > best_eff - 1e-9 && hb > best_hb)) {
                best_eff = eff; best_hb = hb; best_stages = stages;
            }
        }
    }
    if (best_hb == 0) return g;
    p.hb = best_hb;
    p.bands = (d.Ho + p.hb - 1) / p.hb;
    p.KT = (p.hb * p.Wq + 15) / 16 * 16;
    p.NC = p.KT + drspan * p.Wq + dcspan;
    p.GH = p.hb + drspan;
    p.sbo_a = (uint32_t)(p.NC | 1) * 16;
    p.sbo_b = (uint32_t)(p.KT | 1) * 16;
    p.ph_bytes = (uint32_t)planesA * p.sbo_a;
    p.a_stage_bytes = (uint32_t)p.nph * p.ph_bytes;
    p.b_stage_bytes = ((uint32_t)(p.BN / 8) * p.sbo_b + p.a_stage_bytes + 127) / 128 * 128 - p.a_stage_bytes;
    const long long ktiles = (long long)d.N * p.bands;
    if (ktiles >= (1ll << 30)) return g;
    p.ktiles = (int)ktiles;
    p.stages = best_stages;
    if (p.stages > p.ktiles) p.stages = p.ktiles < 2 ? 2 : p.ktiles;
    int splits = d.sms / p.groups;
    if (splits < 1) splits = 1;
    if (splits > p.ktiles) splits = p.ktiles;
    p.splits = splits;
    g.smem_bytes = (uint32_t)p.stages * (p.a_stage_bytes + p.b_stage_bytes);
    if (g.smem_bytes < 120 * 1024) g.smem_bytes = 120 * 1024;   // one CTA per SM: TMEM is not shared
    g.ok = true;
    return g;
}

}  // namespace

bool tc_supported(const Dims& d) { return make_geom(d).ok; }

void plan_tc(const Dims& d, WgradPlan* pl) {
    const TcGeom g = make_geom(d);
    pl->path = PATH_TC;
    pl->splits = g.p.splits;
    pl->tc_band = g.p.hb;
    pl->tc_groups = g.p.groups;
    pl->tc_ktiles = g.p.ktiles;
    pl->tc_stages = g.p.stages;
    pl->bytes = kStatusBlockBytes + (g.p.splits > 1 ? (size_t)g.p.splits * d.dw_elems() * 4 : 0);
}

void tc_plan_info(const Dims& d, ac_plan_info* info) {
    const TcGeom g = make_geom(d);
    info->tensor_core = 1;
    info->splits = g.p.splits;
    info->ctas = g.p.splits * g.p.groups;
    info->groups = g.p.groups;
    info->band_rows = g.p.hb;
    info->k_tile = g.p.KT;
    info->row_pitch = g.p.Wq;
    info->stages = g.p.stages;
    info->smem_bytes = (int32_t)g.smem_bytes;
    info->tmem_columns = (int32_t)g.p.tmem_cols;
    info->units_per_cta = g.p.cibs_per_group * g.p.taps_per_group;
    info->block_n = g.p.BN;
    info->a_cells = g.p.NC;
    info->phases = g.p.nph;
}

ac_status launch_wgrad_tc(const Dims& d, const WgradPlan& pl, const void* z, const void* dy,
                          float* dw, void* workspace, cudaStream_t stream) {
    TcGeom g = make_geom(d);
    if (!g.ok) return AC_ERR_UNSUPPORTED;
    TcParams& p = g.p;
    p.z = static_cast<const __nv_bfloat16*>(z);
    p.dy = static_cast<const __nv_bfloat16*>(dy);
    p.status = static_cast<uint32_t*>(workspace);
    float* partials = reinterpret_cast<float*>(static_cast<char*>(workspace) + kStatusBlockBytes);
    p.out = p.splits > 1 ? partials : dw;
    static bool attr_done[64] = {};
    {
        const ac_status st_ = ensure_smem_limit(wgrad_tc_kernel, (int)kSmemBudget, attr_done);
        if (st_ != AC_OK) return st_;
    }
    record_timing_hook(0, stream);
    wgrad_tc_kernel<<<p.groups * p.splits, kThreads, g.smem_bytes, stream>>>(p);
    record_timing_hook(1, stream);
    AC_CUDA_TRY(cudaGetLastError());
    if (p.splits > 1) return launch_splitk_reduce(partials, p.splits, p.dw_elems, dw, stream);
    (void)pl;
    return AC_OK;
}

}  // namespace ac
