// The small kernels after the LM-head pass:
//   merge_splits_kernel   combines the per-chunk (max, sum-exp, logit) triples of a row into
//                         log pi_target of the drafted token;
//   block_sums_kernel     warp-level segmented sum of per-token log-probabilities per drafted
//                         block (the block probability of Eq. (1) is the product over its tokens);
//   subsample_kernel      one warp per problem: scores of Eq. (1), the normalised weights of
//                         Algorithm 2, a Gumbel-max draw from caller-supplied uniforms and the
//                         switch test of Algorithm 1, Step III;
//   accept_kernel         the switch test alone;
//   fix_merge_kernel      writes the second scoring pass's results over those of the re-scored rows;
//   finish_step_kernel    block sums, SubSample and the switch test for one problem per CTA, for the
//                         fused beam step.
#include <cuda_bf16.h>

#include "specs_internal.h"

namespace specs {
namespace {

constexpr double kLn2 = 0.6931471805599453094;
constexpr unsigned kFull = 0xffffffffu;

// ------------------------------------------------------------------------------------ merge
// Workspace slot (wave * grid + cta) holds, for the 128 rows of that CTA's row tile and for each
// half of the tile's 256 columns (the two epilogue threads of a row), the running maximum in
// base-2 units (max logit * log2 e), the sum of 2^(logit*log2e - max) over that half of the CTA's
// vocabulary chunk, and the drafted id's logit if the id fell there (-inf otherwise).  A half
// that saw no valid column (vocabulary tail) carries max = -inf, sum = 0.  A NEGATIVE sum is the first
// pass's mark on a row whose logits outgrew its tile's accumulation chunks: its magnitude is the sum,
// and the row is re-scored by the second pass.
constexpr int kMergeBatch = 6;                              // splits whose six floats are loaded before any is used

// Fold of a row's per-split partials, in split order, into (max, sum) in base-2 units and the drafted
// id's logit.  The loads of a batch of splits are independent of the arithmetic and of each other, so a
// batch costs one trip to L2.
struct RowFold { float max2; double sum2; float logit; bool marked; };

// The fold takes the splits first, first + step, ...: all of them by default, or a lane's share of them.
__device__ __forceinline__ RowFold fold_row(const ScorePlan& plan, const float* __restrict__ workspace, int64_t row,
                                            int first = 0, int step = 1, uint32_t* status = nullptr) {
    const int mt = (int)(row / kBlockM), r = (int)(row % kBlockM);
    // the row tile's work unit: super tile (cta_group row tiles) and the CTA's rank inside the unit
    const int cg = plan.cta_group, sup = mt / cg, rank = mt % cg;
    int wave, i, gm, splits;
    if (sup < plan.full_waves * plan.group_m) {
        wave = sup / plan.group_m; i = sup % plan.group_m; gm = plan.group_m; splits = plan.split_full;
    } else {
        wave = plan.full_waves; i = sup - plan.full_waves * plan.group_m; gm = plan.rem_m; splits = plan.split_rem;
    }
    // slot of CTA (unit * cg + rank) with unit = chunk * gm + i
    const float* base = workspace + ((size_t)wave * plan.grid + (size_t)i * cg + rank) * kTripleFloats + r;
    const size_t stride = (size_t)gm * cg * kTripleFloats;  // next chunk of the same row tile
    constexpr int kHalf = 3 * kBlockM;                      // second half of the tile's columns

    RowFold f;
    f.max2 = -INFINITY; f.sum2 = 0.0; f.logit = -INFINITY; f.marked = false;
    // checked build: the last float this row's fold reads must lie inside the plan's slots
    if (status != nullptr && splits > 0 &&
        !SPECS_IN_BOUNDS((base - workspace) + (size_t)(splits - 1) * stride + kHalf + 2 * kBlockM,
                         plan_slot_bytes(plan) / sizeof(float), status))
        return f;
    for (int s0 = first; s0 < splits; s0 += kMergeBatch * step) {
        float v[kMergeBatch][6];
#pragma unroll
        for (int u = 0; u < kMergeBatch; ++u) {
            const bool live = s0 + u * step < splits;
            // (splits past the end are not loaded: the loads below are predicated, not redirected)
            float m0 = -INFINITY, s_0 = 0.0f, t0 = -INFINITY, m1 = -INFINITY, s_1 = 0.0f, t1 = -INFINITY;
            if (live) {
                const float* p = base + (size_t)(s0 + u * step) * stride;
                m0 = __ldcg(p); s_0 = __ldcg(p + kBlockM); t0 = __ldcg(p + 2 * kBlockM);
                m1 = __ldcg(p + kHalf); s_1 = __ldcg(p + kHalf + kBlockM); t1 = __ldcg(p + kHalf + 2 * kBlockM);
            }
            f.marked = f.marked || s_0 < 0.0f || s_1 < 0.0f;
            v[u][0] = m0; v[u][1] = fabsf(s_0); v[u][2] = t0;
            v[u][3] = m1; v[u][4] = fabsf(s_1); v[u][5] = t1;
        }
#pragma unroll
        for (int u = 0; u < kMergeBatch; ++u) {
            const float mn = fmaxf(f.max2, fmaxf(v[u][0], v[u][3]));
            if (mn != -INFINITY) {
                // exp2f(-inf) = 0 takes care of halves and states that have seen nothing yet
                f.sum2 = f.sum2 * (double)exp2f(f.max2 - mn) + (double)v[u][1] * (double)exp2f(v[u][0] - mn) +
                         (double)v[u][4] * (double)exp2f(v[u][3] - mn);
                f.max2 = mn;
            }
            f.logit = fmaxf(f.logit, fmaxf(v[u][2], v[u][5]));
        }
    }
    return f;
}

// Two folds over disjoint sets of splits into one.
__device__ __forceinline__ RowFold combine_folds(const RowFold& a, const RowFold& b) {
    RowFold f;
    f.max2 = fmaxf(a.max2, b.max2);
    f.sum2 = 0.0;
    if (f.max2 != -INFINITY)
        f.sum2 = a.sum2 * (double)exp2f(a.max2 - f.max2) + b.sum2 * (double)exp2f(b.max2 - f.max2);
    f.logit = fmaxf(a.logit, b.logit);
    f.marked = a.marked || b.marked;
    return f;
}

// log pi_target of the drafted token from a row's fold:  logit - (max + log2 sum) * ln 2.
__device__ __forceinline__ float fold_logprob(const RowFold& f, int32_t id, int32_t V, uint32_t* __restrict__ status) {
    if (id < 0 || id >= V) {
        atomicOr(status, SPECS_DEV_TOKEN_RANGE);
        return __int_as_float(0x7fc00000);                  // no such vocabulary entry: NaN
    }
    const double lse = ((double)f.max2 + log2(f.sum2)) * kLn2;   // natural-log normaliser
    return (float)((double)f.logit - lse);
}

// Lanes that share a row's splits: four, or as many (a power of two, at most a warp) as leave a lane no more than
// one batch of splits -- a plan for a few rows cuts the vocabulary into up to 148 chunks, and four lanes would fold
// them in five dependent round trips to L2.  A function of the plan alone, so that every route that merges a plan
// (merge kernel, finish kernel) combines the splits in the same order and gives the same bits.
__host__ __device__ inline int merge_lanes(const ScorePlan& plan) {
    // the split count of most rows: that of the full waves when there are any, else the last wave's
    const int splits = plan.full_waves > 0 ? plan.split_full : plan.split_rem;
    int lanes = 4;
    while (lanes < 32 && splits > lanes * kMergeBatch) lanes <<= 1;
    return lanes;
}

// A row's fold by `lanes` adjacent lanes of a warp: lane `sub` of the group takes every lanes-th split, shuffles
// combine them; every lane of the warp must call it, all lanes of a group receive the result.
// A group with `active` false loads nothing (its result is empty) but still takes part in the shuffles.
__device__ __forceinline__ RowFold fold_row_lanes(const ScorePlan& plan, const float* __restrict__ workspace,
                                                  int64_t row, int sub, int lanes, uint32_t* status,
                                                  bool active = true) {
    RowFold f = fold_row(plan, workspace, row, active ? sub : (1 << 30), lanes, status);
    for (int o = 1; o < lanes; o <<= 1) {
        RowFold g;
        g.max2 = __shfl_xor_sync(kFull, f.max2, o);
        g.sum2 = __shfl_xor_sync(kFull, f.sum2, o);
        g.logit = __shfl_xor_sync(kFull, f.logit, o);
        g.marked = __shfl_xor_sync(kFull, (int)f.marked, o) != 0;
        f = combine_folds(f, g);
    }
    return f;
}

// What the merge needs to collect the marked rows of an adaptive plan (ctl == NULL otherwise).
struct CollectArgs {
    FixCtl* ctl;
    int32_t* list;                // [cap_rows]
    uint8_t* compact;             // [cap_rows, row_bytes]
    float* compact_scale;         // [cap_rows], 8-bit operands only
    const uint8_t* hidden;        // [rows, row_bytes]
    const float* hidden_scale;    // [rows] or NULL
    int32_t row_bytes;            // a multiple of 16
    int32_t cap_rows;
};
constexpr int kMergeThreads = 128;
constexpr int kMergeMaxRows = kMergeThreads / 4;            // rows per CTA with the fewest lanes per row

// merge_lanes(plan) lanes per row, each folding its share of the row's splits, combined by shuffles; lane 0 of
// the group writes the row's log-probability (or, for a holder of one vocabulary shard, its partials: max in
// base-2 units, sum of 2^(x - max), drafted id's logit or -inf, 0).  A marked row also takes the next place in
// the list of rows to re-score; then the CTA's threads together copy the hidden states of the CTA's marked rows
// into the compact buffer.  Rows beyond the buffer's capacity are only counted: the second pass then works on
// all rows in place.
__global__ void __launch_bounds__(kMergeThreads)
merge_splits_kernel(const ScorePlan plan, const float* __restrict__ workspace,
                    const int32_t* __restrict__ token_ids, float* __restrict__ tok_logprob,
                    float4* __restrict__ partials, const CollectArgs col, uint32_t* __restrict__ status) {
    __shared__ int32_t marked_row[kMergeMaxRows], marked_at[kMergeMaxRows];
    __shared__ int marked_n;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 0) marked_n = 0;
    __syncthreads();
    asm volatile("griddepcontrol.wait;" ::: "memory");       // the scoring kernel's results
    const int lanes = merge_lanes(plan);
    const int sub = threadIdx.x % lanes;
    // rows past the end load nothing and write nothing (the shuffles need every lane)
    const int64_t row_raw = (int64_t)blockIdx.x * (kMergeThreads / lanes) + threadIdx.x / lanes;
    const int64_t row = row_raw < plan.rows ? row_raw : 0;
    const RowFold f = fold_row_lanes(plan, workspace, row, sub, lanes, status, row_raw < plan.rows);
    if (row_raw < plan.rows && sub == 0) {
        if (partials) partials[row] = make_float4(f.max2, (float)f.sum2, f.logit, 0.0f);
        else          tok_logprob[row] = fold_logprob(f, token_ids[row], plan.V, status);
        if (f.marked && col.ctl != nullptr) {
            // the magnitude that got the row marked is at most the larger of its maximum and its drafted logit
            float mag = fabsf(f.max2) * (float)kLn2;
            if (f.logit != -INFINITY) mag = fmaxf(mag, fabsf(f.logit));
            if (mag == mag) atomicMax(&col.ctl->max_mag_bits, __float_as_uint(fminf(mag, 3.0e38f)));
            const uint32_t at = atomicAdd(&col.ctl->count, 1u);
            if (at < (uint32_t)col.cap_rows) {
                col.list[at] = (int32_t)row;
                if (col.compact_scale) col.compact_scale[at] = col.hidden_scale[row];
                const int k = atomicAdd(&marked_n, 1);
                marked_row[k] = (int32_t)row;
                marked_at[k] = (int32_t)at;
            }
        }
    }
    if (col.ctl == nullptr) return;
    __syncthreads();
    const int n = marked_n;
    const int vecs = col.row_bytes / 16;
    for (int k = 0; k < n; ++k) {
        const uint4* src = reinterpret_cast<const uint4*>(col.hidden + (size_t)marked_row[k] * col.row_bytes);
        uint4* dst = reinterpret_cast<uint4*>(col.compact + (size_t)marked_at[k] * col.row_bytes);
        if (!SPECS_IN_BOUNDS(marked_at[k], col.cap_rows, status) || !SPECS_IN_BOUNDS(marked_row[k], plan.rows, status))
            continue;
        for (int v = threadIdx.x; v < vecs; v += kMergeThreads) dst[v] = __ldg(src + v);
    }
}

// How the second pass ran, from the number of marked rows: not at all, over the gathered rows, or over
// every row in place.  `*plan2` is then the plan its slots are laid out by.
__device__ __forceinline__ int second_pass_rows(const ScorePlan& plan, const FixView& fix, ScorePlan* plan2,
                                                bool* compact) {
    if (fix.ctl == nullptr) return 0;
    const uint32_t n = *reinterpret_cast<const volatile uint32_t*>(&fix.ctl->count);
    if (n == 0u) return 0;
    *compact = n <= (uint32_t)fix.cap_rows;
    // (the chunk length of the second pass does not enter the layout of its slots: any magnitude will do here)
    *plan2 = *compact ? make_compact_plan(plan, (int64_t)n, 0.0f) : make_inplace_fix_plan(plan, 0.0f);
    return *compact ? (int)n : (int)plan.rows;
}

// Results of the second pass over those of the re-scored rows: one thread per re-scored row.
__global__ void __launch_bounds__(kMergeThreads)
fix_merge_kernel(const ScorePlan plan, const FixView fix, const int32_t* __restrict__ token_ids,
                 float* __restrict__ tok_logprob, float4* __restrict__ partials, uint32_t* __restrict__ status) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    ScorePlan plan2;
    bool compact = false;
    const int n = second_pass_rows(plan, fix, &plan2, &compact);
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int64_t row = compact ? (int64_t)fix.list[i] : i;
    const RowFold f = fold_row(plan2, fix.slots, i, 0, 1, status);
    if (!SPECS_IN_BOUNDS(row, plan.rows, status)) return;
    if (partials) partials[row] = make_float4(f.max2, (float)f.sum2, f.logit, 0.0f);
    else          tok_logprob[row] = fold_logprob(f, token_ids[row], plan.V, status);
}

// The same fold over the shards' partials [shards, rows]: log pi_target of the drafted id.
__global__ void __launch_bounds__(128)
merge_partials_kernel(const float4* __restrict__ partials, int32_t shards, int64_t rows,
                      const int32_t* __restrict__ token_ids, int32_t V, float* __restrict__ tok_logprob,
                      uint32_t* __restrict__ status) {
    const int64_t row = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= rows) return;
    float m = -INFINITY, logit = -INFINITY;
    double sum = 0.0;
    for (int j = 0; j < shards; ++j) {
        const float4 v = partials[(size_t)j * rows + row];
        const float mn = fmaxf(m, v.x);
        if (mn != -INFINITY) {
            sum = sum * (double)exp2f(m - mn) + (double)v.y * (double)exp2f(v.x - mn);
            m = mn;
        }
        logit = fmaxf(logit, v.z);
    }
    const int32_t id = token_ids[row];
    if (id < 0 || id >= V) {
        tok_logprob[row] = __int_as_float(0x7fc00000);
        atomicOr(status, SPECS_DEV_TOKEN_RANGE);
        return;
    }
    tok_logprob[row] = (float)((double)logit - ((double)m + log2(sum)) * kLn2);
}

// ------------------------------------------------------------------------------------ block sums
__global__ void block_sums_kernel(const float* __restrict__ per_token, const int64_t* __restrict__ block_offsets,
                                  int32_t B, float* __restrict__ out, double* __restrict__ out_f64) {
    const int warp = (int)(((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
    const int lane = threadIdx.x & 31;
    if (warp >= B) return;
    const int64_t a = block_offsets[warp], b = block_offsets[warp + 1];
    double acc = 0.0;
    for (int64_t t = a + lane; t < b; t += 32) acc += (double)per_token[t];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(kFull, acc, o);
    if (lane == 0) {
        if (out) out[warp] = (float)acc;
        if (out_f64) out_f64[warp] = acc;
    }
}

// ------------------------------------------------------------------------------------ SubSample
template <typename LP>
__device__ __forceinline__ double score_of(const LP* lp_t, const LP* lp_g, const float* reward, float beta, int i) {
    const double br = __dmul_rn((double)beta, (double)reward[i]);
    if (lp_g == nullptr) return br;                          // pi_gen = pi_target: the ratio drops out
    return __dadd_rn(__dsub_rn((double)lp_t[i], (double)lp_g[i]), br);
}

// One warp, one problem with candidates [a, b): scores, weights, Gumbel-max pick, switch test.
template <typename LP>
__device__ __forceinline__ void subsample_problem(const LP* lp_t, const LP* lp_g, const float* __restrict__ reward,
                                                  int a, int b, int p, int lane, float beta,
                                                  const float* __restrict__ uniforms, int32_t* __restrict__ chosen,
                                                  float* __restrict__ weights, float tau,
                                                  uint8_t* __restrict__ accept) {
    if (b <= a) {
        if (lane == 0) {
            if (chosen) chosen[p] = -1;
            if (accept) accept[p] = 0;
        }
        return;
    }
    double smax = -INFINITY, best = -INFINITY;
    int best_i = 0x7fffffff;
    float rmax = -INFINITY;
    for (int i = a + lane; i < b; i += 32) {
        const double s = score_of(lp_t, lp_g, reward, beta, i);
        smax = fmax(smax, s);
        rmax = fmaxf(rmax, reward[i]);
        float u = uniforms[i];
        u = fminf(fmaxf(u, 2.98023223876953125e-8f), 0.99999994039535522461f);   // [2^-25, 1 - 2^-24]
        const double pert = s - log(-log((double)u));        // S_i + Gumbel(0,1)
        if (pert > best || best_i == 0x7fffffff) { best = pert; best_i = i; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        smax = fmax(smax, __shfl_xor_sync(kFull, smax, o));
        rmax = fmaxf(rmax, __shfl_xor_sync(kFull, rmax, o));
        const double ob = __shfl_xor_sync(kFull, best, o);
        const int oi = __shfl_xor_sync(kFull, best_i, o);
        if (oi != 0x7fffffff && (best_i == 0x7fffffff || ob > best || (ob == best && oi < best_i))) {
            best = ob; best_i = oi;
        }
    }
    if (weights) {
        double z = 0.0;
        for (int i = a + lane; i < b; i += 32) z += exp(score_of(lp_t, lp_g, reward, beta, i) - smax);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(kFull, z, o);
        const double lse = smax + log(z);
        for (int i = a + lane; i < b; i += 32)
            weights[i] = (float)exp(score_of(lp_t, lp_g, reward, beta, i) - lse);
    }
    if (lane == 0) {
        if (chosen) chosen[p] = best_i - a;
        if (accept) accept[p] = (rmax > tau) ? 1 : 0;
    }
}

template <typename LP>
__global__ void subsample_kernel(const LP* __restrict__ lp_t, const LP* __restrict__ lp_g,
                                 const float* __restrict__ reward, const int32_t* __restrict__ cand_offsets,
                                 int32_t P, float beta, const float* __restrict__ uniforms,
                                 int32_t* __restrict__ chosen, float* __restrict__ weights, float tau,
                                 uint8_t* __restrict__ accept) {
    const int p = (int)(((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
    const int lane = threadIdx.x & 31;
    if (p >= P) return;
    subsample_problem<LP>(lp_t, lp_g, reward, cand_offsets[p], cand_offsets[p + 1], p, lane, beta, uniforms, chosen,
                          weights, tau, accept);
}

// ------------------------------------------------------------------------------------ selection variants
// Algorithm 2 with its candidate set L explicit (mask), the "highest reward" rule of the beam-search
// and RSD++ baselines, the score without the log-ratio, and the three switch rules.  One warp per
// problem; scores in double like subsample_problem.
__global__ void select_kernel(const double* __restrict__ lp_t, const double* __restrict__ lp_g,
                              const float* __restrict__ reward, const uint8_t* __restrict__ mask,
                              const int32_t* __restrict__ cand_offsets, int32_t P, float beta,
                              const float* __restrict__ uniforms, int select_rule, int score_flags,
                              int switch_rule, float tau, int32_t* __restrict__ chosen,
                              float* __restrict__ weights, uint8_t* __restrict__ flag) {
    const int p = (int)(((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
    const int lane = threadIdx.x & 31;
    if (p >= P) return;
    const int a = cand_offsets[p], b = cand_offsets[p + 1];
    const double* lq = (score_flags & SPECS_SCORE_NO_LL) ? nullptr : lp_g;
    double smax = -INFINITY, best = -INFINITY;
    int best_i = 0x7fffffff;
    float rmax = -INFINITY;
    for (int i = a + lane; i < b; i += 32) {
        rmax = fmaxf(rmax, reward[i]);                       // the switch test sees every candidate
        if (mask && mask[i] == 0) continue;
        const double s = score_of(lp_t, lq, reward, beta, i);
        smax = fmax(smax, s);
        double key;
        if (select_rule == SPECS_SELECT_BEST_REWARD) {
            key = (double)reward[i];
        } else {
            float u = uniforms[i];
            u = fminf(fmaxf(u, 2.98023223876953125e-8f), 0.99999994039535522461f);
            key = s - log(-log((double)u));
        }
        if (key > best || best_i == 0x7fffffff) { best = key; best_i = i; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        smax = fmax(smax, __shfl_xor_sync(kFull, smax, o));
        rmax = fmaxf(rmax, __shfl_xor_sync(kFull, rmax, o));
        const double ob = __shfl_xor_sync(kFull, best, o);
        const int oi = __shfl_xor_sync(kFull, best_i, o);
        if (oi != 0x7fffffff && (best_i == 0x7fffffff || ob > best || (ob == best && oi < best_i))) {
            best = ob; best_i = oi;
        }
    }
    const bool none = best_i == 0x7fffffff;                  // empty problem, or nobody in L
    if (weights) {
        if (select_rule == SPECS_SELECT_BEST_REWARD || none) {
            for (int i = a + lane; i < b; i += 32) weights[i] = (i == best_i) ? 1.0f : 0.0f;
        } else {
            double z = 0.0;
            for (int i = a + lane; i < b; i += 32)
                if (!mask || mask[i]) z += exp(score_of(lp_t, lq, reward, beta, i) - smax);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(kFull, z, o);
            const double lse = smax + log(z);
            for (int i = a + lane; i < b; i += 32)
                weights[i] = (!mask || mask[i]) ? (float)exp(score_of(lp_t, lq, reward, beta, i) - lse) : 0.0f;
        }
    }
    if (lane == 0) {
        chosen[p] = none ? -1 : best_i - a;
        if (flag) {
            uint8_t f = 0;
            if (b > a) {
                if (switch_rule == SPECS_SWITCH_ANY_ABOVE) f = rmax > tau;
                else if (switch_rule == SPECS_SWITCH_NONE_ABOVE) f = !(rmax > tau);
                else f = !none && reward[best_i] < tau;
            }
            flag[p] = f;
        }
    }
}

// ------------------------------------------------------------------------------------ fused finish
// Everything after the merge for one problem per CTA: where a second scoring pass ran, its results go over
// those of the problem's re-scored rows first; then target and generator log-probabilities are summed per
// drafted block, then SubSample and the switch test on those sums.  The phases are separated by CTA
// barriers; the block sums travel through the output arrays blk_lp / gen_lp (double).
constexpr int kFinishThreads = 1024;

// Ids of the selected block of problem p into row p of chosen_ids [P, stride] (-1 beyond the block's
// length, the whole row -1 when nothing was selected) and its length into chosen_len[p]: what Step II
// of Algorithm 1 appends to the trace.  Executed by all threads of a CTA (or a warp with nthreads = 32).
__device__ __forceinline__ void gather_chosen_block(const int32_t* __restrict__ token_ids,
                                                    const int64_t* __restrict__ block_offsets, int a, int pick, int p,
                                                    int32_t* __restrict__ chosen_ids, int32_t* __restrict__ chosen_len,
                                                    int32_t stride, int tid, int nthreads) {
    int64_t t0 = 0, len = 0;
    if (pick >= 0) {
        t0 = block_offsets[a + pick];
        len = block_offsets[a + pick + 1] - t0;
        if (len > stride) len = stride;                      // the host has checked that no block is longer
    }
    for (int k = tid; k < stride; k += nthreads)
        chosen_ids[(size_t)p * stride + k] = k < len ? token_ids[t0 + k] : -1;
    if (tid == 0) chosen_len[p] = (int32_t)len;
}

__global__ void gather_chosen_kernel(const int32_t* __restrict__ token_ids, const int64_t* __restrict__ block_offsets,
                                     const int32_t* __restrict__ cand_offsets, const int32_t* __restrict__ chosen,
                                     int32_t* __restrict__ chosen_ids, int32_t* __restrict__ chosen_len,
                                     int32_t stride) {
    const int p = blockIdx.x;
    gather_chosen_block(token_ids, block_offsets, cand_offsets[p], chosen[p], p, chosen_ids, chosen_len, stride,
                        threadIdx.x, blockDim.x);
}

// Second-pass results of the rows [row_a, row_b) into `tok`.
__device__ __forceinline__ void apply_second_pass(const ScorePlan& plan, const FixView& fix, int64_t row_a,
                                                  int64_t row_b, const int32_t* __restrict__ token_ids, float* tok,
                                                  uint32_t* __restrict__ status, int tid, int nthreads) {
    ScorePlan plan2;
    bool compact = false;
    const int n = second_pass_rows(plan, fix, &plan2, &compact);
    if (n == 0) return;
    if (compact) {
        for (int i = tid; i < n; i += nthreads) {
            const int64_t row = fix.list[i];
            if (row >= row_a && row < row_b)
                tok[row] = fold_logprob(fold_row(plan2, fix.slots, i, 0, 1, status), token_ids[row], plan.V, status);
        }
    } else {
        for (int64_t row = row_a + tid; row < row_b; row += nthreads)
            tok[row] = fold_logprob(fold_row(plan2, fix.slots, row, 0, 1, status), token_ids[row], plan.V, status);
    }
}

// tok_logprob (and, with two scoring passes, gen_tok) hold the merged first-pass results; gen_tok may also
// be the caller's own array of generator log-probabilities (fix_g.ctl == NULL then), or NULL.
// With merge_slots the merge has not run: the CTA folds its problem's rows itself first (small steps without
// a second pass, where a merge launch of its own would cost more than it does).
__global__ void __launch_bounds__(kFinishThreads)
finish_step_kernel(const ScorePlan plan, const FixView fix_t, const ScorePlan plan_g, const FixView fix_g,
                   const int32_t* __restrict__ token_ids, const int64_t* __restrict__ block_offsets,
                   const int32_t* __restrict__ cand_offsets, float* gen_tok, const float* __restrict__ reward,
                   const float* __restrict__ uniforms, float beta, float tau, float* tok_logprob, double* blk_lp,
                   double* gen_lp, float* __restrict__ weights, int32_t* chosen, uint8_t* __restrict__ accept,
                   int32_t* __restrict__ chosen_ids, int32_t* __restrict__ chosen_len, int32_t chosen_stride,
                   const float* __restrict__ merge_slots, uint32_t* __restrict__ status) {
    // Launched with programmatic stream serialisation: wait here for the kernels before it.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // let the next kernel of the stream (the next step's scoring kernel) begin its prologue
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int p = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int a = cand_offsets[p], b = cand_offsets[p + 1];
    if (b > a) {
        const int64_t row_a = block_offsets[a], row_b = block_offsets[b];   // the problem's rows are contiguous
        if (merge_slots != nullptr) {
            const int lanes = merge_lanes(plan);
            const int sub = threadIdx.x % lanes;
            for (int64_t r0 = row_a; r0 < row_b; r0 += kFinishThreads / lanes) {
                const int64_t row_raw = r0 + threadIdx.x / lanes;
                const int64_t row = row_raw < row_b ? row_raw : row_a;      // idle groups: a valid row, no loads
                const RowFold f = fold_row_lanes(plan, merge_slots, row, sub, lanes, status, row_raw < row_b);
                if (row_raw < row_b && sub == 0) tok_logprob[row] = fold_logprob(f, token_ids[row], plan.V, status);
            }
            __syncthreads();
        }
        if (fix_t.ctl != nullptr || fix_g.ctl != nullptr) {
            apply_second_pass(plan, fix_t, row_a, row_b, token_ids, tok_logprob, status, threadIdx.x, kFinishThreads);
            apply_second_pass(plan_g, fix_g, row_a, row_b, token_ids, gen_tok, status, threadIdx.x, kFinishThreads);
            __syncthreads();
        }
        for (int i = a + warp; i < b; i += kFinishThreads / 32) {
            const int64_t t0 = block_offsets[i], t1 = block_offsets[i + 1];
            double lp = 0.0, lq = 0.0;
            for (int64_t t = t0 + lane; t < t1; t += 32) {
                lp += (double)tok_logprob[t];
                if (gen_tok) lq += (double)gen_tok[t];
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                lp += __shfl_xor_sync(kFull, lp, o);
                lq += __shfl_xor_sync(kFull, lq, o);
            }
            if (lane == 0) {
                blk_lp[i] = lp;
                if (gen_tok) gen_lp[i] = lq;
            }
        }
        __syncthreads();
    }
    if (warp == 0)
        subsample_problem<double>(blk_lp, gen_tok ? gen_lp : nullptr, reward, a, b, p, lane, beta, uniforms,
                                  chosen, weights, tau, accept);
    if (chosen_ids) {
        __syncthreads();                                      // chosen[p] was written by warp 0 of this CTA
        gather_chosen_block(token_ids, block_offsets, a, chosen[p], p, chosen_ids, chosen_len, chosen_stride,
                            threadIdx.x, kFinishThreads);
    }
}

// ------------------------------------------------------------------------------------ PRM head
// Reward of every drafted block from the process reward model's final hidden states: the value head
// (one weight vector, one bias) on the hidden state of the block's last token, through the logistic
// function.  One warp per block; 16-byte loads of eight bf16 at a time, fp32 products summed in fp32
// per lane and in double across the lanes.  HBM-bound on B rows of d bf16 (plus the head, from L2).
__global__ void prm_head_kernel(const __nv_bfloat16* __restrict__ prm_hidden, const int64_t* __restrict__ block_offsets,
                                int32_t B, int32_t d, const __nv_bfloat16* __restrict__ w_head, float bias,
                                float* __restrict__ reward) {
    const int i = (int)(((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
    const int lane = threadIdx.x & 31;
    if (i >= B) return;
    const int64_t a = block_offsets[i], e = block_offsets[i + 1];
    if (e <= a) {                                            // no last token
        if (lane == 0) reward[i] = __int_as_float(0x7fc00000);
        return;
    }
    const uint4* h = reinterpret_cast<const uint4*>(prm_hidden + (size_t)(e - 1) * d);
    const uint4* w = reinterpret_cast<const uint4*>(w_head);
    float acc = 0.0f;
    for (int v = lane; v < d / 8; v += 32) {
        const uint4 hv = __ldg(h + v), wv = __ldg(w + v);
        const __nv_bfloat162* hp = reinterpret_cast<const __nv_bfloat162*>(&hv);
        const __nv_bfloat162* wp = reinterpret_cast<const __nv_bfloat162*>(&wv);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 x = __bfloat1622float2(hp[j]), y = __bfloat1622float2(wp[j]);
            acc = fmaf(x.x, y.x, acc);
            acc = fmaf(x.y, y.y, acc);
        }
    }
    double z = (double)acc;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(kFull, z, o);
    if (lane == 0) reward[i] = (float)(1.0 / (1.0 + exp(-(z + (double)bias))));
}

__global__ void accept_kernel(const float* __restrict__ reward, const int32_t* __restrict__ cand_offsets, int32_t P,
                              float tau, uint8_t* __restrict__ accept) {
    const int p = (int)(((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
    const int lane = threadIdx.x & 31;
    if (p >= P) return;
    const int a = cand_offsets[p], b = cand_offsets[p + 1];
    float rmax = -INFINITY;
    for (int i = a + lane; i < b; i += 32) rmax = fmaxf(rmax, reward[i]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) rmax = fmaxf(rmax, __shfl_xor_sync(kFull, rmax, o));
    if (lane == 0) accept[p] = (b > a && rmax > tau) ? 1 : 0;
}

inline unsigned warps_grid(int64_t warps, int threads) {
    const int64_t per_block = threads / 32;
    return (unsigned)((warps + per_block - 1) / per_block);
}

}  // namespace

namespace {
// every kernel of a step is launched with programmatic stream serialisation and waits for its predecessor itself
template <typename... KArgs, typename... Args>
int launch_chained(void (*kernel)(KArgs...), unsigned blocks, unsigned threads, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks, 1, 1);
    cfg.blockDim = dim3(threads, 1, 1);
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cuda_status(cudaLaunchKernelEx(&cfg, kernel, args...));
}
}  // namespace

int launch_merge(specs_ctx* ctx, const ScorePlan& plan, void* workspace, const int32_t* token_ids,
                 float* tok_logprob, float* partials, const void* hidden, const float* hidden_scale,
                 cudaStream_t stream) {
    if (plan.rows == 0) return SPECS_OK;
    CollectArgs col = {};
    if (plan.adaptive) {
        const WsLayout lay = plan_layout(plan);
        uint8_t* ws = static_cast<uint8_t*>(workspace);
        col.ctl = reinterpret_cast<FixCtl*>(ws + lay.ctl);
        col.list = reinterpret_cast<int32_t*>(ws + lay.list);
        col.compact = ws + lay.compact;
        col.compact_scale = plan.elem_bytes == 1 ? reinterpret_cast<float*>(ws + lay.compact_scale) : nullptr;
        col.hidden = static_cast<const uint8_t*>(hidden);
        col.hidden_scale = hidden_scale;
        col.row_bytes = plan.d * plan.elem_bytes;
        col.cap_rows = lay.cap_rows;
    }
    const int rows_per_cta = kMergeThreads / merge_lanes(plan);
    const unsigned blocks = (unsigned)((plan.rows + rows_per_cta - 1) / rows_per_cta);
    return launch_chained(merge_splits_kernel, blocks, kMergeThreads, stream, plan,
                          static_cast<const float*>(workspace), token_ids, tok_logprob,
                          reinterpret_cast<float4*>(partials), col, ctx->d_status);
}

int launch_fix_merge(specs_ctx* ctx, const ScorePlan& plan, const void* workspace, const int32_t* token_ids,
                     float* tok_logprob, float* partials, cudaStream_t stream) {
    if (plan.rows == 0 || !plan.adaptive) return SPECS_OK;
    const unsigned blocks = (unsigned)((plan.rows + kMergeThreads - 1) / kMergeThreads);
    return launch_chained(fix_merge_kernel, blocks, kMergeThreads, stream, plan, fix_view(plan, workspace), token_ids,
                          tok_logprob, reinterpret_cast<float4*>(partials), ctx->d_status);
}

int launch_finish_step(specs_ctx* ctx, const ScorePlan& plan, const FixView& fix_t, const ScorePlan* plan_g,
                       const FixView& fix_g, const int32_t* token_ids, const int64_t* block_offsets,
                       const int32_t* cand_offsets, int32_t P, float* gen_tok, const float* reward,
                       const float* uniforms, float beta, float tau, float* tok_logprob, double* blk_lp, double* gen_lp,
                       float* weights, int32_t* chosen, uint8_t* accept, int32_t* chosen_ids, int32_t* chosen_len,
                       int32_t chosen_stride, const float* merge_slots, cudaStream_t stream) {
    if (P == 0) return SPECS_OK;
    const ScorePlan second = plan_g ? *plan_g : plan;
    return launch_chained(finish_step_kernel, (unsigned)P, kFinishThreads, stream, plan, fix_t, second, fix_g,
                          token_ids, block_offsets, cand_offsets, gen_tok, reward, uniforms, beta, tau, tok_logprob,
                          blk_lp, gen_lp, weights, chosen, accept, chosen_ids, chosen_len, chosen_stride, merge_slots,
                          ctx->d_status);
}

int launch_gather_chosen(const int32_t* token_ids, const int64_t* block_offsets, const int32_t* cand_offsets,
                         const int32_t* chosen, int32_t P, int32_t* chosen_ids, int32_t* chosen_len, int32_t stride,
                         cudaStream_t stream) {
    if (P == 0) return SPECS_OK;
    gather_chosen_kernel<<<(unsigned)P, 128, 0, stream>>>(token_ids, block_offsets, cand_offsets, chosen, chosen_ids,
                                                          chosen_len, stride);
    return cuda_status(cudaGetLastError());
}

int launch_merge_partials(specs_ctx* ctx, const float* partials, int32_t shards, int64_t rows, const int32_t* token_ids,
                          int32_t V, float* tok_logprob, cudaStream_t stream) {
    if (rows == 0) return SPECS_OK;
    merge_partials_kernel<<<(unsigned)((rows + 127) / 128), 128, 0, stream>>>(
        reinterpret_cast<const float4*>(partials), shards, rows, token_ids, V, tok_logprob, ctx->d_status);
    return cuda_status(cudaGetLastError());
}

int launch_block_sums(const float* per_token, const int64_t* block_offsets, int32_t B, float* out, double* out_f64,
                      cudaStream_t stream) {
    if (B == 0) return SPECS_OK;
    const int threads = 128;
    block_sums_kernel<<<warps_grid(B, threads), threads, 0, stream>>>(per_token, block_offsets, B, out, out_f64);
    return cuda_status(cudaGetLastError());
}

int launch_subsample(const void* lp_target, const void* lp_gen, bool lp_is_f64, const float* reward,
                     const int32_t* cand_offsets, int32_t P, float beta, const float* uniforms, int32_t* chosen,
                     float* weights, float tau, uint8_t* accept, cudaStream_t stream) {
    if (P == 0) return SPECS_OK;
    const int threads = 128;
    const unsigned blocks = warps_grid(P, threads);
    if (lp_is_f64)
        subsample_kernel<double><<<blocks, threads, 0, stream>>>(
            static_cast<const double*>(lp_target), static_cast<const double*>(lp_gen), reward, cand_offsets, P, beta,
            uniforms, chosen, weights, tau, accept);
    else
        subsample_kernel<float><<<blocks, threads, 0, stream>>>(
            static_cast<const float*>(lp_target), static_cast<const float*>(lp_gen), reward, cand_offsets, P, beta,
            uniforms, chosen, weights, tau, accept);
    return cuda_status(cudaGetLastError());
}

int launch_select(const double* lp_target, const double* lp_gen, const float* reward, const uint8_t* mask,
                  const int32_t* cand_offsets, int32_t P, float beta, const float* uniforms, int select_rule,
                  int score_flags, int switch_rule, float tau, int32_t* chosen, float* weights, uint8_t* flag,
                  cudaStream_t stream) {
    if (P == 0) return SPECS_OK;
    const int threads = 128;
    select_kernel<<<warps_grid(P, threads), threads, 0, stream>>>(lp_target, lp_gen, reward, mask, cand_offsets, P,
                                                                   beta, uniforms, select_rule, score_flags,
                                                                   switch_rule, tau, chosen, weights, flag);
    return cuda_status(cudaGetLastError());
}

int launch_prm_head(const void* prm_hidden, const int64_t* block_offsets, int32_t B, int32_t d, const void* w_head,
                    float bias, float* reward, cudaStream_t stream) {
    if (B == 0) return SPECS_OK;
    const int threads = 128;
    prm_head_kernel<<<warps_grid(B, threads), threads, 0, stream>>>(
        static_cast<const __nv_bfloat16*>(prm_hidden), block_offsets, B, d, static_cast<const __nv_bfloat16*>(w_head),
        bias, reward);
    return cuda_status(cudaGetLastError());
}

int launch_accept(const float* reward, const int32_t* cand_offsets, int32_t P, float tau, uint8_t* accept,
                  cudaStream_t stream) {
    if (P == 0) return SPECS_OK;
    const int threads = 128;
    accept_kernel<<<warps_grid(P, threads), threads, 0, stream>>>(reward, cand_offsets, P, tau, accept);
    return cuda_status(cudaGetLastError());
}

}  // namespace specs
