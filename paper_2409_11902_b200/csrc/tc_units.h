// How the tensor-core weight-gradient kernels cut dW into accumulator tiles.
//
// An accumulator tile ("unit") is 128 rows x BN columns of fp32 in tensor memory:
// rows = one block of CB input channels of one filter tap (CB = 128, or 64 with
// the upper 64 rows unused), columns = BN output channels. A CTA owns up to
// 512 / BN units that share the same output-channel block, so that one
// output-gradient tile in shared memory feeds all of them. CTAs that own
// different units of the same K-slice form a "group".
#pragma once

namespace ac {

struct UnitPlan {
    int CB, ncgpc, ncib_total;   // input-channel block, its 8-channel planes, number of blocks
    int BN, ncob;                // output-channel block, number of blocks
    int taps_per_group, ntapgroups, cibs_per_group, ncibgroups;
    int groups;                  // CTAs per K-slice
    int units;                   // accumulator tiles per CTA (upper bound)
    unsigned tmem_cols;          // power of two >= units * BN
    int planesA;                 // 8-channel planes of the input tile a CTA keeps per phase
    bool ok;
};

// fill_rectangles: when the taps do not fit one CTA, let a CTA's tiles be any taps x channel-blocks
// rectangle (not only taps of one channel block), chosen so that as few CTAs as possible are left
// with fewer tiles than the others.
// bn_cap: widest output-channel block considered (a narrower one leaves more shared memory to the
// input tile).
inline UnitPlan plan_units(int Ci, int Co, int ntaps, int max_units, bool fill_rectangles = false,
                           int bn_cap = 256) {
    UnitPlan u{};
    u.ok = false;
    if (Ci % 64 != 0 || Co % 64 != 0) return u;
    u.CB = (Ci % 128 == 0) ? 128 : 64;
    u.ncgpc = u.CB / 8;
    u.ncib_total = Ci / u.CB;
    u.BN = Co <= 256 ? Co : (Co % 256 == 0 ? 256 : (Co % 128 == 0 ? 128 : 64));
    while (u.BN > bn_cap && u.BN % 128 == 0) u.BN /= 2;
    u.ncob = Co / u.BN;
    const int U = 512 / u.BN;
    if (ntaps <= U) {
        u.ntapgroups = 1;
        u.taps_per_group = ntaps;
        u.cibs_per_group = U / ntaps < u.ncib_total ? U / ntaps : u.ncib_total;
    } else {
        u.ntapgroups = (ntaps + U - 1) / U;
        u.taps_per_group = (ntaps + u.ntapgroups - 1) / u.ntapgroups;
        u.ntapgroups = (ntaps + u.taps_per_group - 1) / u.taps_per_group;
        u.cibs_per_group = 1;
        if (fill_rectangles) {
            // 9 taps in CTAs of 2 tiles: (2,2,2,2,1) taps of one block leaves every fifth CTA half
            // empty; 1 tap x 2 blocks fills them all. Ties go to more taps (a smaller input tile).
            long long best_slots = (long long)u.ntapgroups * u.taps_per_group * u.ncib_total;
            for (int t = U; t >= 1; --t) {
                int c = U / t < u.ncib_total ? U / t : u.ncib_total;
                if (c < 1 || t * c > max_units) continue;
                const int tg = (ntaps + t - 1) / t, cg = (u.ncib_total + c - 1) / c;
                const long long slots = (long long)tg * t * cg * c;      // tile slots over all CTAs
                if (slots < best_slots) {
                    best_slots = slots;
                    u.taps_per_group = t; u.ntapgroups = tg; u.cibs_per_group = c;
                }
            }
        }
    }
    u.units = u.cibs_per_group * u.taps_per_group;
    if (u.units > max_units) return u;
    u.ncibgroups = (u.ncib_total + u.cibs_per_group - 1) / u.cibs_per_group;
    u.groups = u.ncob * u.ncibgroups * u.ntapgroups;
    u.tmem_cols = 32;
    while (u.tmem_cols < (unsigned)(u.units * u.BN)) u.tmem_cols *= 2;
    if (u.tmem_cols > 512) return u;
    // an MMA with M = 128 always reads 16 planes: with CB = 64 the upper 8 belong to
    // rows whose results are discarded, but they must lie inside the allocation
    u.planesA = u.cibs_per_group * u.ncgpc + (u.CB == 64 ? 8 : 0);
    u.ok = true;
    return u;
}

__host__ __device__ inline int floor_div_i(int a, int b) {
    int q = a / b;
    return (a % b != 0 && ((a < 0) != (b < 0))) ? q - 1 : q;
}

}  // namespace ac
