// Internal declarations shared by the translation units of the library.
// Nothing here is part of the C ABI (see include/specs.h for that).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <vector>

#include "specs.h"

namespace specs {

// ---- index checks of the checked build (-DSPECS_DEBUG) ------------------------------------------
// SPECS_IN_BOUNDS(index, extent, status) is true when 0 <= index < extent.  In the checked build a
// failing index raises SPECS_DEV_BOUNDS in the status word and the caller skips the access; in the
// default build the macro is the constant true and costs nothing.
#ifdef SPECS_DEBUG
__device__ __forceinline__ bool index_in_bounds(int64_t index, int64_t extent, uint32_t* status) {
    if (index >= 0 && index < extent) return true;
    atomicOr(status, SPECS_DEV_BOUNDS);
    return false;
}
#define SPECS_IN_BOUNDS(index, extent, status) ::specs::index_in_bounds((int64_t)(index), (int64_t)(extent), (status))
#else
#define SPECS_IN_BOUNDS(index, extent, status) true
#endif

// ---- tile geometry of the tensor-core scoring kernel -----------------------------------------
constexpr int kBlockM = 128;   // drafted rows per tile   (= TMEM lanes, one epilogue thread per row)
constexpr int kBlockN = 256;   // vocabulary entries per tile (= fp32 TMEM columns of one accumulator)
constexpr int kBlockK = 64;    // bf16 elements per k-block: 128 bytes, one swizzle-128B row
constexpr int kTripleFloats = 2 * 3 * kBlockM;   // one workspace slot: for each half of the 256 columns, max[128], sumexp[128], logit[128]
constexpr int kDefaultChunkKBlocks = 8;      // k-blocks (of 64) per accumulation chunk: 512 elements of d

// How the (row tile x vocab tile) grid is cut into persistent work units.
//
// A work unit is run by `cta_group` CTAs: one CTA (128 rows), or a pair of CTAs in one
// cluster (256 rows: the pair issues one tcgen05.mma over both CTAs' shared memory, each CTA
// stages its own 128 rows of hidden states and only HALF of the 256 W rows of a tile, which
// cuts the L2 -> shared-memory operand traffic per CTA from 48 KB to 32 KB per k-block).
// A "super tile" is the cta_group * 128 rows of one unit.
//
// Time is cut into waves.  In one wave `gm` consecutive super tiles are live and the
// vocabulary is cut into `s` contiguous chunks, gm * s <= units; unit u owns super tile
// (u % gm) of the wave and chunk (u / gm).  Units that share a chunk stream the same W tiles
// at the same pace, so each W tile is fetched from HBM once per wave and hits L2 for the
// other super tiles, while the wave's hidden-state tiles stay L2-resident.  Every wave but
// the last is "full" (gm = group_m, s = split_full); the last takes the remaining super tiles.
struct ScorePlan {
    int64_t rows;
    int32_t d, V;
    int32_t row_tiles;     // ceil(rows / 128)
    int32_t vocab_tiles;   // ceil(V / 256)
    int32_t k_blocks;      // ceil(d / elements per k-block): 128-byte k-blocks, 64 bf16 or 128 E4M3 elements
    int32_t elem_bytes;    // 2: bf16 operands; 1: E4M3 operands with per-row scales
    int32_t cta_group;     // CTAs per work unit: 1, or 2 (cluster pair)
    int32_t units;         // work units per wave
    int32_t grid;          // CTAs launched = units * cta_group (also workspace slots per wave)
    int32_t super_tiles;   // ceil(row_tiles / cta_group)
    int32_t group_m;       // super tiles per full wave
    int32_t split_full;    // vocab chunks per full wave
    int32_t full_waves;
    int32_t rem_m;         // super tiles of the last wave (0: none)
    int32_t split_rem;     // vocab chunks of the last wave
    int32_t waves;         // full_waves + (rem_m > 0)
    int32_t chunk_kblocks; // k-blocks per fresh tensor-core accumulator (chunks are summed in registers)
    int32_t lead_tiles;    // > 0: a unit starts vocabulary tile t of a wave only once every unit that streams the
                           //      same W chunk has started tile t - lead_tiles (advisory, bounded wait)
    int32_t pace_points;   // pace points per vocabulary tile (1: the tile's start only); lead_tiles counts these
    int32_t id_offset;     // vocabulary index of W_vocab's first row (a shard of a larger vocabulary); 0 normally
    uint32_t epoch;        // distinguishes this launch's progress words from older contents of the workspace
    int32_t adaptive;      // 1: from the third vocabulary tile of a run on, lengthen the chunks as far as the
                           //    logit magnitude seen in the run's first tile allows (see score_tcgen05.cu)
};

// cta_group argument of make_score_plan: 0 lets the planner choose between 1 and 2.
constexpr int kCtaGroupAuto = 0;

// Host-side planner (pure arithmetic, no CUDA calls).  `pair_units` is the number of CTA
// pairs the device can keep resident (<= num_sms / 2; 0: pairs unavailable).
ScorePlan make_score_plan(int64_t rows, int32_t d, int32_t V, int32_t num_sms, int32_t pair_units,
                          int32_t cta_group = kCtaGroupAuto, int32_t chunk_kblocks = kDefaultChunkKBlocks,
                          bool adaptive = true, int32_t elem_bytes = 2);
size_t plan_workspace_bytes(const ScorePlan& p);
__host__ __device__ inline size_t plan_slot_bytes(const ScorePlan& p) {
    return (size_t)(p.waves > 0 ? p.waves : 1) * (size_t)p.grid * kTripleFloats * sizeof(float);
}

// ---- second pass over the rows whose logits outgrew their tile's accumulation chunks --------------
// With adaptive chunks the first pass marks every row in which a logit that matters (the row's
// maximum or the drafted id's) lies beyond the magnitude its tile's chunks were sized for.  The merge
// collects those rows (a count and a list), copies their hidden states into a compact buffer, and a
// second launch of the scoring kernel re-scores them with the base chunks.  More marked rows than
// the compact buffer holds: the second launch re-scores every row in place instead.
struct FixCtl {
    uint32_t count;        // rows marked by the merge (may exceed the compact capacity)
    uint32_t max_mag_bits; // largest |logit| that mattered in a marked row, as the bits of a non-negative float
    uint32_t pad[2];
};

// Magnitude up to which the base chunk (32 accumulations) keeps the accumulated truncation under 2e-3: rows
// beyond it are marked even where the base chunk was kept, and the second pass shortens its chunks for them.
constexpr float kBaseChunkBound = 1024.0f;

// k-blocks per accumulation chunk of the second pass, from the largest magnitude among the marked rows: as many
// accumulations (four per k-block) as keep count x fp32 spacing at that magnitude under 2e-3, at most `base`,
// at least one k-block.
__host__ __device__ inline int second_pass_chunk_kblocks(float mag, int base) {
    if (!(mag >= kBaseChunkBound)) return base;
    int kb = base;
    for (float bound = kBaseChunkBound; mag >= bound && kb > 1; bound *= 2.0f) kb >>= 1;
    return kb < 1 ? 1 : kb;
}

// The workspace: triple slots [waves x grid], one 64-bit progress word per unit, and for adaptive
// plans the control block, the list of marked rows, their gathered hidden states (and, for 8-bit
// operands, row scales), and the slots + progress words of the second pass.
struct WsLayout {
    size_t progress;       // = plan_slot_bytes(plan)
    size_t ctl, list, compact, compact_scale, fix_slots;   // 0 when the plan is not adaptive
    size_t total;
    int32_t cap_rows;      // rows the compact buffer holds (a multiple of the super tile)
};
inline WsLayout plan_layout(const ScorePlan& p) {
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    WsLayout L = {};
    L.progress = plan_slot_bytes(p);
    const size_t first = L.progress + (size_t)p.units * sizeof(uint64_t);
    if (!p.adaptive) { L.total = first; return L; }
    int cap_super = (p.super_tiles + 7) / 8;
    if (cap_super > 32) cap_super = 32;
    if (cap_super > p.units) cap_super = p.units;
    if (cap_super < 1) cap_super = 1;
    L.cap_rows = cap_super * kBlockM * p.cta_group;
    size_t off = up(first);
    L.ctl = off;            off += 256;
    L.list = off;           off += up((size_t)L.cap_rows * sizeof(int32_t));
    L.compact = off;        off += up((size_t)L.cap_rows * p.d * p.elem_bytes);
    L.compact_scale = off;  off += p.elem_bytes == 1 ? up((size_t)L.cap_rows * sizeof(float)) : 0;
    L.fix_slots = off;      off += up(first);
    L.total = off;
    return L;
}

// Plan of the second pass over `n` gathered rows (n <= cap_rows, so one wave): same tile shape and
// vocabulary as `base`, every super tile live at once, the units shared out over vocabulary chunks,
// base chunks throughout.
__host__ __device__ inline ScorePlan make_compact_plan(const ScorePlan& base, int64_t n, float mag) {
    ScorePlan p = base;
    p.chunk_kblocks = second_pass_chunk_kblocks(mag, base.chunk_kblocks);
    p.rows = n;
    p.row_tiles = (int32_t)((n + kBlockM - 1) / kBlockM);
    p.super_tiles = (p.row_tiles + p.cta_group - 1) / p.cta_group;
    int s = p.super_tiles > 0 ? p.units / p.super_tiles : 1;
    if (s > p.vocab_tiles) s = p.vocab_tiles;
    if (s < 1) s = 1;
    p.group_m = p.super_tiles; p.split_full = s; p.full_waves = p.super_tiles > 0 ? 1 : 0;
    p.rem_m = 0; p.split_rem = 0; p.waves = p.full_waves;
    p.adaptive = 0;
    return p;
}
// The second pass over all rows in place: the first pass's geometry with the base chunks.
__host__ __device__ inline ScorePlan make_inplace_fix_plan(const ScorePlan& base, float mag) {
    ScorePlan p = base;
    p.chunk_kblocks = second_pass_chunk_kblocks(mag, base.chunk_kblocks);
    p.adaptive = 0;
    return p;
}

// Work unit `unit` in wave `wave`: returns false when the unit idles in that wave.
__host__ __device__ inline bool plan_unit(const ScorePlan& p, int wave, int unit,
                                          int* super_tile, int* n_begin, int* n_end) {
    int gm, s, base;
    if (wave < p.full_waves) { gm = p.group_m; s = p.split_full; base = wave * p.group_m; }
    else                     { gm = p.rem_m;   s = p.split_rem;  base = p.full_waves * p.group_m; }
    if (gm <= 0 || unit >= gm * s) return false;
    const int i = unit % gm, c = unit / gm;
    *super_tile = base + i;
    *n_begin = (int)(((int64_t)c * p.vocab_tiles) / s);
    *n_end   = (int)(((int64_t)(c + 1) * p.vocab_tiles) / s);
    return true;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TimedLaunch { cudaEvent_t start, stop; bool second_pass; };

// A tensor map the context has encoded before, found again by what it describes.
struct CachedMap {
    const void* base; uint64_t inner, outer; uint32_t box_inner, box_outer; int elem_bytes;
    CUtensorMap map;
};
constexpr size_t kMapCacheSize = 16;

// What the kernels after the first scoring pass need to know about the second one.
struct FixView {
    const FixCtl* ctl;        // NULL: the plan is not adaptive, there is no second pass
    const int32_t* list;      // marked rows in the order of the compact buffer
    const float* slots;       // triple slots of the second pass
    int32_t cap_rows;
};

// One host-buffer step in flight: a grow-only device arena (hidden states, small inputs, outputs, scoring
// workspace), a pinned mirror of the arena's small-input and output blocks, the events that order its copies
// and kernels, and where its results go once it is waited for.
struct HostSlot {
    void* arena = nullptr;
    size_t arena_bytes = 0;
    void* h_stage = nullptr;
    size_t stage_bytes = 0;
    cudaEvent_t ev_in = nullptr, ev_done = nullptr, ev_out = nullptr;
    bool busy = false;
    uint32_t ticket = 0;
    size_t in0 = 0, o_tok = 0, o_blk = 0, o_wts = 0, o_cho = 0, o_acc = 0;
    int64_t rows = 0;
    int32_t B = 0, P = 0;
    float* h_tok = nullptr; double* h_blk = nullptr; float* h_wts = nullptr; int32_t* h_cho = nullptr;
    uint8_t* h_acc = nullptr;
};

}  // namespace specs

struct specs_ctx {
    int device = 0;
    int num_sms = 0;
    int engine = SPECS_ENGINE_TCGEN05;
    int pair_units = 0;                    // resident CTA pairs of the pair kernel (0: not available)
    int chunk_kblocks = specs::kDefaultChunkKBlocks;   // see specs_set_accum_chunk
    bool accum_adaptive = true;
    int lead_tiles = 1;                    // see specs_set_tile_lead
    uint32_t* d_status = nullptr;          // device status word (SPECS_DEV_* bits)
    specs::EncodeTiledFn encode_tiled = nullptr;
    // the host-buffer step: two slots, so that one step's copies run under the other's kernels
    specs::HostSlot host_slots[2];
    cudaStream_t copy_in = nullptr, copy_out = nullptr;   // created on first use
    uint32_t next_ticket = 0;
    std::vector<specs::CachedMap> maps;    // tensor maps of recent operands (round robin)
    size_t maps_next = 0;
    // optional per-launch timing of the tensor-core kernel
    bool timing = false;
    std::vector<specs::TimedLaunch> timed;
    size_t timed_used = 0;
};

namespace specs {

// ---- kernel launchers (each enqueues on `stream`, returns a specs_status) ---------------------
// CTA pairs of the pair kernel that the current device keeps resident at once (cached per
// device; also opts both kernels in to their dynamic shared memory).  0 if pairs cannot launch.
int query_pair_units(int device, int num_sms);
// First pass: scores every row; `workspace` is laid out by plan_layout(plan).
int launch_score_tcgen05(specs_ctx* ctx, const ScorePlan& plan, const void* hidden, const void* w_vocab,
                         const int32_t* token_ids, void* workspace, cudaStream_t stream, int32_t id_offset = 0,
                         const float* hidden_scale = nullptr, const float* w_scale = nullptr);
// Second pass (adaptive plans only; a no-op launch when the merge marked no row): re-scores the marked
// rows with the base chunks.  Must follow launch_merge on the same workspace.
int launch_score_second_pass(specs_ctx* ctx, const ScorePlan& plan, const void* hidden, const void* w_vocab,
                             const int32_t* token_ids, void* workspace, cudaStream_t stream, int32_t id_offset = 0,
                             const float* hidden_scale = nullptr, const float* w_scale = nullptr);
FixView fix_view(const ScorePlan& plan, const void* workspace);
int launch_quantize_rows(const void* x_bf16, int64_t n, int32_t d, uint8_t* codes, float* scale, cudaStream_t stream);
int launch_wait_expiry_probe(specs_ctx* ctx, unsigned long long limit_ns, cudaStream_t stream);
int launch_score_simt(specs_ctx* ctx, const void* hidden, const void* w_vocab, const int32_t* token_ids,
                      int64_t rows, int32_t d, int32_t V, float* tok_logprob, cudaStream_t stream);
// Merge of the first pass's splits into tok_logprob (or, with `partials`, into per-row shard partials);
// for adaptive plans it also collects the marked rows and gathers their hidden states.
int launch_merge(specs_ctx* ctx, const ScorePlan& plan, void* workspace, const int32_t* token_ids,
                 float* tok_logprob, float* partials, const void* hidden, const float* hidden_scale,
                 cudaStream_t stream);
// Results of the second pass written over those of the marked rows.
int launch_fix_merge(specs_ctx* ctx, const ScorePlan& plan, const void* workspace, const int32_t* token_ids,
                     float* tok_logprob, float* partials, cudaStream_t stream);
// Block sums of both per-token arrays, SubSample, the switch test and the gather of the chosen block, one CTA
// per problem.  fix_t / fix_g: second-pass results still to be written over tok_logprob / gen_tok first.
// merge_slots: the first pass's slots when no merge kernel ran (the CTAs then merge their own rows first).
int launch_finish_step(specs_ctx* ctx, const ScorePlan& plan, const FixView& fix_t, const ScorePlan* plan_g,
                       const FixView& fix_g, const int32_t* token_ids, const int64_t* block_offsets,
                       const int32_t* cand_offsets, int32_t P, float* gen_tok, const float* reward,
                       const float* uniforms, float beta, float tau, float* tok_logprob, double* blk_lp, double* gen_lp,
                       float* weights, int32_t* chosen, uint8_t* accept, int32_t* chosen_ids, int32_t* chosen_len,
                       int32_t chosen_stride, const float* merge_slots, cudaStream_t stream);
// Steps whose merge the finish kernel does itself (merge_slots): no second pass to wait for, and so few partial
// triples (rows x vocabulary chunks) that one CTA per problem folds them faster than another launch would take
// (64 rows x 4 chunks: 28 us per step instead of 32; 64 rows x 119 chunks: no gain, 128 x 119: 3 us slower).
inline bool merge_in_finish(const ScorePlan& plan) {
    const int splits = plan.split_full > plan.split_rem ? plan.split_full : plan.split_rem;
    return !plan.adaptive && plan.rows * splits <= 2048;
}
int launch_gather_chosen(const int32_t* token_ids, const int64_t* block_offsets, const int32_t* cand_offsets,
                         const int32_t* chosen, int32_t P, int32_t* chosen_ids, int32_t* chosen_len, int32_t stride,
                         cudaStream_t stream);
int launch_merge_partials(specs_ctx* ctx, const float* partials, int32_t shards, int64_t rows, const int32_t* token_ids,
                          int32_t V, float* tok_logprob, cudaStream_t stream);
int launch_block_sums(const float* per_token, const int64_t* block_offsets, int32_t B,
                      float* out, double* out_f64, cudaStream_t stream);
int launch_subsample(const void* lp_target, const void* lp_gen, bool lp_is_f64, const float* reward,
                     const int32_t* cand_offsets, int32_t P, float beta, const float* uniforms,
                     int32_t* chosen, float* weights, float tau, uint8_t* accept, cudaStream_t stream);
int launch_select(const double* lp_target, const double* lp_gen, const float* reward, const uint8_t* mask,
                  const int32_t* cand_offsets, int32_t P, float beta, const float* uniforms, int select_rule,
                  int score_flags, int switch_rule, float tau, int32_t* chosen, float* weights, uint8_t* flag,
                  cudaStream_t stream);
int launch_prm_head(const void* prm_hidden, const int64_t* block_offsets, int32_t B, int32_t d, const void* w_head,
                    float bias, float* reward, cudaStream_t stream);
int launch_accept(const float* reward, const int32_t* cand_offsets, int32_t P, float tau,
                  uint8_t* accept, cudaStream_t stream);

inline int cuda_status(cudaError_t e) { return e == cudaSuccess ? SPECS_OK : SPECS_ERR_CUDA; }

}  // namespace specs
