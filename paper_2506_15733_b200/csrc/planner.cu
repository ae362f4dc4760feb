// Host-side work-unit planner of the tensor-core scoring kernel (pure arithmetic, no CUDA calls):
// how the (row super tile x vocabulary tile) grid is cut into waves of persistent work units.
#include <cstring>

#include "specs_internal.h"

namespace specs {

// ---------------------------------------------------------------------------------- planner
namespace {

// Estimated duration of a plan, in seconds: per wave, the busiest unit's run of vocabulary
// tiles at the tensor rate the kernel reaches, or the HBM time of streaming W once, whichever
// is longer.  The constants only rank candidate plans; they are not performance claims.
constexpr double kPlanClockHz = 1.4e9;            // SM clock under sustained tensor load
constexpr double kPlanHbmBytesPerS = 6.0e12;
constexpr double kPlanL2Budget = 50.0e6;          // bytes of hidden-state tiles kept live per wave
constexpr double kPlanTensorEff1 = 0.76;          // one CTA per unit: bounded by L2 -> SM operand delivery
constexpr double kPlanTensorEff2 = 0.93;          // CTA pair: each CTA stages only half of the W tile

double fill_plan(ScorePlan* p, int32_t cta_group, int32_t units) {
    p->cta_group = cta_group;
    p->units = units;
    p->grid = units * cta_group;
    p->super_tiles = (p->row_tiles + cta_group - 1) / cta_group;
    const double tile_bytes = (double)kBlockM * cta_group * p->d * p->elem_bytes;
    const double t_tile = (double)p->k_blocks * 512.0 / (cta_group == 2 ? kPlanTensorEff2 : kPlanTensorEff1) /
                          kPlanClockHz;
    const double w_bytes = (double)p->V * p->d * p->elem_bytes;
    auto wave_time = [&](int gm, int s) {
        const int run = (p->vocab_tiles + s - 1) / s;          // vocabulary tiles of the busiest unit
        const double t_hbm = (w_bytes + gm * tile_bytes) / kPlanHbmBytesPerS;
        const double t_mma = run * t_tile;
        return t_mma > t_hbm ? t_mma : t_hbm;
    };
    double best = -1.0;
    const int s_max = units < p->vocab_tiles ? units : p->vocab_tiles;
    // super tiles whose hidden states fit the L2 budget together (at least one)
    int gm_cap = (int)(kPlanL2Budget / tile_bytes);
    if (gm_cap < 1) gm_cap = 1;
    for (int s = 1; s <= s_max; ++s) {
        // as many super tiles per wave as the units and the L2 budget allow; when the vocabulary has fewer tiles
        // than there are units, s cannot grow to use them all and some units stay idle
        int gm = units / s;
        if (gm > gm_cap) gm = gm_cap;
        const int full = p->super_tiles / gm;
        const int rem = p->super_tiles - full * gm;
        int s_rem = 0;
        double cost = full * wave_time(gm, s);
        if (rem > 0) {
            s_rem = units / rem;
            if (s_rem > p->vocab_tiles) s_rem = p->vocab_tiles;
            if (s_rem < 1) s_rem = 1;
            // The fewest chunks with the same longest run: every unit then carries that run (one of them may be
            // a tile short) and all finish together.  With more chunks a few units would carry one tile more
            // than the rest and stream it alone at the end, at one SM's rate instead of the memory system's
            // (measured on 64 rows, d = 3584: 148 chunks of 4 or 5 tiles 187 us, 119 chunks of 5 tiles 175 us).
            const int run_rem = (p->vocab_tiles + s_rem - 1) / s_rem;
            s_rem = (p->vocab_tiles + run_rem - 1) / run_rem;
            cost += wave_time(rem, s_rem);
        }
        if (best < 0.0 || cost < best * (1.0 - 1e-9)) {
            best = cost;
            p->group_m = gm; p->split_full = s; p->full_waves = full; p->rem_m = rem; p->split_rem = s_rem;
        }
    }
    p->waves = p->full_waves + (p->rem_m > 0 ? 1 : 0);
    return best;
}

}  // namespace

ScorePlan make_score_plan(int64_t rows, int32_t d, int32_t V, int32_t num_sms, int32_t pair_units,
                          int32_t cta_group, int32_t chunk_kblocks, bool adaptive, int32_t elem_bytes) {
    ScorePlan p;
    std::memset(&p, 0, sizeof(p));
    p.rows = rows; p.d = d; p.V = V;
    p.row_tiles = (int32_t)((rows + kBlockM - 1) / kBlockM);
    p.vocab_tiles = (V + kBlockN - 1) / kBlockN;
    p.elem_bytes = elem_bytes;
    const int32_t k_elems = kBlockK * 2 / elem_bytes;        // elements in a 128-byte k-block
    p.k_blocks = (d + k_elems - 1) / k_elems;
    p.chunk_kblocks = (chunk_kblocks > 0 && chunk_kblocks < p.k_blocks) ? chunk_kblocks : p.k_blocks;
    // A single row tile (at most 128 rows) is bound by streaming W from HBM, not by the tensor pipe: the
    // restarts of short accumulation chunks cost it nothing, so it keeps the base chunks and needs no second pass.
    p.adaptive = (adaptive && p.chunk_kblocks < p.k_blocks && p.row_tiles > 1) ? 1 : 0;
    if (pair_units <= 0 && cta_group == 2) cta_group = 1;      // pairs unavailable on this device
    if (cta_group == 1 || pair_units <= 0) {
        fill_plan(&p, 1, num_sms);
    } else if (cta_group == 2) {
        fill_plan(&p, 2, pair_units);
    } else {
        ScorePlan q = p;
        const double c1 = fill_plan(&p, 1, num_sms);
        const double c2 = fill_plan(&q, 2, pair_units);
        if (c2 < c1) p = q;
    }
    return p;
}

size_t plan_workspace_bytes(const ScorePlan& p) {
    return plan_layout(p).total;
}

}  // namespace specs

