// Work plans of the persistent kernels (host arithmetic only).
//
// A launch is a sequence of tiles, each a run of `nsteps` channel steps.  The steps of all tiles, laid end to end,
// are cut into one share per CTA of equal weight, so that a tile count that is not a multiple of the CTA count
// leaves no CTA idle in a last round.  A share is a list of segments (tile, steps [k0, k1)).  A tile that falls
// into several shares is a split tile: every part stores its partial sums in its own slot and counts itself in on the
// tile's counter; the part that arrives last adds the slots in part order and finishes the tile.
#pragma once

#include <stdint.h>

#include <algorithm>
#include <vector>

namespace sbnn {

struct ShareSeg {
    int tile;            // position of the tile in the launch's sequence
    int k0, k1;          // channel steps [k0, k1)
    int part, nparts;    // this segment's position among the tile's parts
    int slot, counter;   // first partial-sum slot and arrival counter of the tile (nparts > 1)
    int reserved;
};

struct SharePlan {
    std::vector<int32_t> cta_ptr;   // [ncta + 1]: CTA c owns segments cta_ptr[c] .. cta_ptr[c + 1] - 1
    std::vector<ShareSeg> segs;
    int ncta = 0, nslots = 0, ncounters = 0;
};

// weight(tile, k) > 0 is what step k of a tile costs.  At most ncta_max CTAs, never more than there are steps.
template <class Weight>
void plan_shares(long long ntiles, int nsteps, Weight weight, int ncta_max, SharePlan* out) {
    const long long steps = ntiles * nsteps;
    const int ncta = (int)std::max<long long>(1, std::min<long long>(ncta_max, steps));
    long long total = 0;
    for (long long t = 0; t < ntiles; ++t)
        for (int k = 0; k < nsteps; ++k) total += weight(t, k);
    std::vector<int32_t>& cta_ptr = out->cta_ptr;
    std::vector<ShareSeg>& segs = out->segs;
    cta_ptr.assign(ncta + 1, 0);
    segs.clear();
    long long cum = 0;
    int cur_cta = 0;
    for (long long t = 0; t < ntiles; ++t) {
        int part = 0, k = 0;
        while (k < nsteps) {
            // the CTA that owns the step starting at cumulative weight `cum`
            int c = total > 0 ? (int)std::min<long long>(ncta - 1, (long long)((__int128)cum * ncta / total)) : 0;
            if (c < cur_cta) c = cur_cta;
            while (cur_cta < c) cta_ptr[++cur_cta] = (int32_t)segs.size();
            // this CTA's share ends at weight (c + 1) * total / ncta: take steps while they start below it
            const long long lim = (long long)(((__int128)(c + 1) * total + ncta - 1) / ncta);
            const int k0 = k;
            while (k < nsteps && (k == k0 || cum < lim)) {
                cum += weight(t, k);
                ++k;
            }
            const ShareSeg sg = {(int)t, k0, k, part++, 0, 0, 0, 0};
            segs.push_back(sg);
        }
        for (int j = 0; j < part; ++j) segs[segs.size() - 1 - j].nparts = part;   // the tile's segments are the last `part` entries
    }
    while (cur_cta < ncta) cta_ptr[++cur_cta] = (int32_t)segs.size();
    out->ncta = ncta;
    out->nslots = out->ncounters = 0;
    for (size_t i = 0; i < segs.size(); ++i) {
        if (segs[i].nparts > 1 && segs[i].part == 0) {
            for (int j = 0; j < segs[i].nparts; ++j) {
                segs[i + j].slot = out->nslots;
                segs[i + j].counter = out->ncounters;
            }
            out->nslots += segs[i].nparts;
            out->ncounters += 1;
        }
    }
}

}  // namespace sbnn
