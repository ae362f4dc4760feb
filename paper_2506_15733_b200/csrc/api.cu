// C ABI of the library: argument validation, the work-unit planner, context management and
// the host-buffer convenience entry point.  All arithmetic of the method runs in the kernels
// of the other translation units.
#include <cstring>
#include <new>

#include "specs_internal.h"

using namespace specs;

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_offsets64(const int64_t* off, int64_t count, int64_t total) {
    if (off[0] != 0) return SPECS_ERR_OFFSETS;
    for (int64_t i = 0; i < count; ++i)
        if (off[i + 1] < off[i]) return SPECS_ERR_OFFSETS;
    return off[count] == total ? SPECS_OK : SPECS_ERR_OFFSETS;
}
int check_offsets32(const int32_t* off, int64_t count, int64_t total) {
    if (off[0] != 0) return SPECS_ERR_OFFSETS;
    for (int64_t i = 0; i < count; ++i)
        if (off[i + 1] < off[i]) return SPECS_ERR_OFFSETS;
    return off[count] == total ? SPECS_OK : SPECS_ERR_OFFSETS;
}

int check_score_shapes(int64_t rows, int32_t d, int32_t V, int32_t B) {
    if (rows < 0 || d <= 0 || (d % 8) != 0 || V <= 0 || B < 0) return SPECS_ERR_SHAPE;
    if (rows > (int64_t)1 << 31) return SPECS_ERR_LIMIT;
    return SPECS_OK;
}

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
        if (prev == dev) prev = -1;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

// The scoring launches for one LM head: the first pass over all rows, the merge of its vocabulary splits
// into `tok_logprob` (or into shard `partials`), and -- for plans with adaptive accumulation chunks -- the
// second pass over the rows the first one marked.  With `defer_fix` the caller's next kernel (the finish
// kernel of a fused step) writes the second pass's results over the marked rows; otherwise a last small
// launch does.
int score_rows(specs_ctx* ctx, const ScorePlan& plan, const void* hidden, const void* w_vocab,
               const int32_t* token_ids, void* workspace, cudaStream_t stream, int32_t id_offset,
               const float* hidden_scale, const float* w_scale, float* tok_logprob, float* partials, bool defer_fix,
               bool finish_may_merge = false) {
    int st = launch_score_tcgen05(ctx, plan, hidden, w_vocab, token_ids, workspace, stream, id_offset, hidden_scale,
                                  w_scale);
    if (st != SPECS_OK) return st;
    if (finish_may_merge && merge_in_finish(plan)) return SPECS_OK;   // the finish kernel merges; no second pass exists
    st = launch_merge(ctx, plan, workspace, token_ids, tok_logprob, partials, hidden, hidden_scale, stream);
    if (st != SPECS_OK || !plan.adaptive) return st;
    st = launch_score_second_pass(ctx, plan, hidden, w_vocab, token_ids, workspace, stream, id_offset, hidden_scale,
                                  w_scale);
    if (st != SPECS_OK || defer_fix) return st;
    return launch_fix_merge(ctx, plan, workspace, token_ids, tok_logprob, partials, stream);
}

const FixView kNoFix = {nullptr, nullptr, nullptr, 0};

}  // namespace

extern "C" {

const char* specs_status_string(int status) {
    switch (status) {
        case SPECS_OK: return "ok";
        case SPECS_ERR_NULL: return "a required pointer is NULL";
        case SPECS_ERR_SHAPE: return "invalid shape (negative size, d not a positive multiple of 8, ...)";
        case SPECS_ERR_ALIGN: return "pointer not 16-byte aligned";
        case SPECS_ERR_WORKSPACE: return "workspace too small";
        case SPECS_ERR_OFFSETS: return "offsets must start at 0, be non-decreasing and end at the total";
        case SPECS_ERR_ARCH: return "device is not an sm_100-class GPU";
        case SPECS_ERR_CUDA: return "a CUDA call failed";
        case SPECS_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel expired";
        case SPECS_ERR_TOKEN_RANGE: return "a drafted token id was outside [0, V)";
        case SPECS_ERR_LIMIT: return "a size exceeds a documented maximum";
        case SPECS_ERR_DEVICE_BOUNDS: return "an index check inside a kernel failed (checked build)";
        default: return "unknown status";
    }
}

int specs_debug_build(void) {
#ifdef SPECS_DEBUG
    return 1;
#else
    return 0;
#endif
}

int specs_create(specs_ctx** out, int device) {
    if (!out) return SPECS_ERR_NULL;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
        cudaGetLastError();
        return SPECS_ERR_CUDA;
    }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return SPECS_ERR_CUDA;
    if (prop.major != 10) return SPECS_ERR_ARCH;
    DeviceGuard guard(device);
    if (!guard.ok) return SPECS_ERR_CUDA;

    specs_ctx* ctx = new (std::nothrow) specs_ctx();
    if (!ctx) return SPECS_ERR_CUDA;
    ctx->device = device;
    ctx->num_sms = prop.multiProcessorCount;

    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || fn == nullptr) {
        delete ctx;
        return SPECS_ERR_CUDA;
    }
    ctx->encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
    if (cudaMalloc(&ctx->d_status, sizeof(uint32_t)) != cudaSuccess ||
        cudaMemset(ctx->d_status, 0, sizeof(uint32_t)) != cudaSuccess) {
        if (ctx->d_status) cudaFree(ctx->d_status);
        delete ctx;
        return SPECS_ERR_CUDA;
    }
    ctx->pair_units = query_pair_units(device, ctx->num_sms);
    *out = ctx;
    return SPECS_OK;
}

int specs_destroy(specs_ctx* ctx) {
    if (!ctx) return SPECS_OK;
    DeviceGuard guard(ctx->device);
    for (auto& t : ctx->timed) { cudaEventDestroy(t.start); cudaEventDestroy(t.stop); }
    for (HostSlot& slot : ctx->host_slots) {
        if (slot.ev_out && slot.busy) cudaEventSynchronize(slot.ev_out);
        if (slot.arena) cudaFree(slot.arena);
        if (slot.h_stage) cudaFreeHost(slot.h_stage);
        if (slot.ev_in) cudaEventDestroy(slot.ev_in);
        if (slot.ev_done) cudaEventDestroy(slot.ev_done);
        if (slot.ev_out) cudaEventDestroy(slot.ev_out);
    }
    if (ctx->copy_in) cudaStreamDestroy(ctx->copy_in);
    if (ctx->copy_out) cudaStreamDestroy(ctx->copy_out);
    if (ctx->d_status) cudaFree(ctx->d_status);
    delete ctx;
    return SPECS_OK;
}

int specs_set_engine(specs_ctx* ctx, int engine) {
    if (!ctx) return SPECS_ERR_NULL;
    if (engine != SPECS_ENGINE_TCGEN05 && engine != SPECS_ENGINE_SIMT && engine != SPECS_ENGINE_TCGEN05_1CTA &&
        engine != SPECS_ENGINE_TCGEN05_2CTA)
        return SPECS_ERR_SHAPE;
#ifndef SPECS_DEBUG
    if (engine == SPECS_ENGINE_SIMT) return SPECS_ERR_SHAPE;     // the bisecting aid exists in the checked build only
#endif
    if (engine == SPECS_ENGINE_TCGEN05_2CTA && ctx->pair_units <= 0) return SPECS_ERR_CUDA;
    ctx->engine = engine;
    return SPECS_OK;
}

int specs_set_accum_chunk(specs_ctx* ctx, int32_t k_elements) {
    if (!ctx) return SPECS_ERR_NULL;
    if (k_elements == SPECS_ACCUM_ADAPTIVE) {
        ctx->chunk_kblocks = kDefaultChunkKBlocks;
        ctx->accum_adaptive = true;
        return SPECS_OK;
    }
    if (k_elements < 0 || (k_elements % kBlockK) != 0) return SPECS_ERR_SHAPE;
    ctx->chunk_kblocks = k_elements / kBlockK;               // 0: one accumulator over the whole of d
    ctx->accum_adaptive = false;
    return SPECS_OK;
}

int specs_set_tile_lead(specs_ctx* ctx, int32_t tiles) {
    if (!ctx) return SPECS_ERR_NULL;
    if (tiles < 0 || tiles > 1024) return SPECS_ERR_SHAPE;
    ctx->lead_tiles = tiles;
    return SPECS_OK;
}

int specs_sm_count(const specs_ctx* ctx) { return ctx ? ctx->num_sms : 0; }

size_t specs_score_workspace_bytes(const specs_ctx* ctx, int64_t rows, int32_t d, int32_t V) {
    if (!ctx || check_score_shapes(rows, d, V, 0) != SPECS_OK) return 0;
    // enough for whichever tile shape the engine setting selects at call time
    const size_t one = plan_workspace_bytes(make_score_plan(rows, d, V, ctx->num_sms, ctx->pair_units, 1));
    const size_t two = plan_workspace_bytes(make_score_plan(rows, d, V, ctx->num_sms, ctx->pair_units, 2));
    return one > two ? one : two;
}

int specs_score_plan(int64_t rows, int32_t d, int32_t V, int32_t num_sms, int32_t cta_group, int32_t* h_out16) {
    if (!h_out16) return SPECS_ERR_NULL;
    if (check_score_shapes(rows, d, V, 0) != SPECS_OK || num_sms <= 0 || cta_group < 0 || cta_group > 2)
        return SPECS_ERR_SHAPE;
    const ScorePlan p = make_score_plan(rows, d, V, num_sms, num_sms / 2, cta_group);
    const size_t ws = plan_workspace_bytes(p);
    const int32_t v[16] = {p.row_tiles, p.vocab_tiles, p.k_blocks, p.grid, p.group_m, p.split_full,
                           p.full_waves, p.rem_m, p.split_rem, p.waves,
                           (int32_t)(ws & 0x7fffffff), (int32_t)(ws >> 31),
                           p.cta_group, p.units, p.super_tiles, p.chunk_kblocks};
    std::memcpy(h_out16, v, sizeof(v));
    return SPECS_OK;
}

int specs_score_plan_unit(int64_t rows, int32_t d, int32_t V, int32_t num_sms, int32_t cta_group, int32_t wave,
                          int32_t cta, int32_t* h_out3) {
    if (!h_out3) return SPECS_ERR_NULL;
    if (check_score_shapes(rows, d, V, 0) != SPECS_OK || num_sms <= 0 || cta_group < 0 || cta_group > 2)
        return SPECS_ERR_SHAPE;
    const ScorePlan p = make_score_plan(rows, d, V, num_sms, num_sms / 2, cta_group);
    int st = -1, nb = 0, ne = 0;
    h_out3[0] = -1; h_out3[1] = 0; h_out3[2] = 0;
    if (wave < 0 || wave >= p.waves || cta < 0 || cta >= p.grid ||
        !plan_unit(p, wave, cta / p.cta_group, &st, &nb, &ne))
        return SPECS_OK;
    const int mt = st * p.cta_group + cta % p.cta_group;     // the CTA's own 128-row tile
    if (mt >= p.row_tiles) return SPECS_OK;                  // second CTA of a pair past the last row tile
    h_out3[0] = mt; h_out3[1] = nb; h_out3[2] = ne;
    return SPECS_OK;
}

int specs_score_blocks(specs_ctx* ctx, const void* hidden, const void* W_vocab, const int32_t* token_ids,
                       const int64_t* block_offsets, int64_t rows, int32_t d, int32_t V, int32_t B,
                       float* tok_logprob, float* blk_logprob, double* blk_logprob_f64, void* workspace,
                       size_t workspace_bytes, void* cuda_stream) {
    if (!ctx) return SPECS_ERR_NULL;
    int st = check_score_shapes(rows, d, V, B);
    if (st != SPECS_OK) return st;
    if (!W_vocab || (B > 0 && !block_offsets)) return SPECS_ERR_NULL;
    if (rows > 0 && (!hidden || !token_ids || !tok_logprob)) return SPECS_ERR_NULL;
    if (!aligned16(hidden) || !aligned16(W_vocab) || !aligned16(workspace)) return SPECS_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SPECS_ERR_CUDA;

    if (rows > 0) {
#ifdef SPECS_DEBUG
        if (ctx->engine == SPECS_ENGINE_SIMT) {
            st = launch_score_simt(ctx, hidden, W_vocab, token_ids, rows, d, V, tok_logprob, stream);
            if (st != SPECS_OK) return st;
        } else
#endif
        {
            const int cta_group = ctx->engine == SPECS_ENGINE_TCGEN05_1CTA ? 1
                                : ctx->engine == SPECS_ENGINE_TCGEN05_2CTA ? 2 : kCtaGroupAuto;
            const ScorePlan plan = make_score_plan(rows, d, V, ctx->num_sms, ctx->pair_units, cta_group,
                                                   ctx->chunk_kblocks, ctx->accum_adaptive);
            if (!workspace) return SPECS_ERR_NULL;
            if (workspace_bytes < plan_workspace_bytes(plan)) return SPECS_ERR_WORKSPACE;
            st = score_rows(ctx, plan, hidden, W_vocab, token_ids, workspace, stream, 0, nullptr, nullptr, tok_logprob,
                            nullptr, false);
            if (st != SPECS_OK) return st;
        }
    }
    if (B > 0 && (blk_logprob || blk_logprob_f64))
        return launch_block_sums(tok_logprob, block_offsets, B, blk_logprob, blk_logprob_f64, stream);
    return SPECS_OK;
}

int specs_score_partials(specs_ctx* ctx, const void* hidden, const void* W_shard, const int32_t* token_ids,
                         int32_t id_offset, int64_t rows, int32_t d, int32_t V_shard, float* partials,
                         void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!ctx) return SPECS_ERR_NULL;
    int st = check_score_shapes(rows, d, V_shard, 0);
    if (st != SPECS_OK) return st;
    if (id_offset < 0) return SPECS_ERR_SHAPE;
    if (rows == 0) return SPECS_OK;
    if (!hidden || !W_shard || !token_ids || !partials || !workspace) return SPECS_ERR_NULL;
    if (!aligned16(hidden) || !aligned16(W_shard) || !aligned16(workspace) || !aligned16(partials))
        return SPECS_ERR_ALIGN;
    if (ctx->engine == SPECS_ENGINE_SIMT) return SPECS_ERR_SHAPE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SPECS_ERR_CUDA;
    const int cta_group = ctx->engine == SPECS_ENGINE_TCGEN05_1CTA ? 1
                        : ctx->engine == SPECS_ENGINE_TCGEN05_2CTA ? 2 : kCtaGroupAuto;
    const ScorePlan plan = make_score_plan(rows, d, V_shard, ctx->num_sms, ctx->pair_units, cta_group,
                                           ctx->chunk_kblocks, ctx->accum_adaptive);
    if (workspace_bytes < plan_workspace_bytes(plan)) return SPECS_ERR_WORKSPACE;
    return score_rows(ctx, plan, hidden, W_shard, token_ids, workspace, stream, id_offset, nullptr, nullptr, nullptr,
                      partials, false);
}

int specs_merge_partials(specs_ctx* ctx, const float* partials, int32_t shards, int64_t rows,
                         const int32_t* token_ids, int32_t V, float* tok_logprob, void* cuda_stream) {
    if (!ctx) return SPECS_ERR_NULL;
    if (shards <= 0 || rows < 0 || V <= 0) return SPECS_ERR_SHAPE;
    if (rows == 0) return SPECS_OK;
    if (!partials || !token_ids || !tok_logprob) return SPECS_ERR_NULL;
    if (!aligned16(partials)) return SPECS_ERR_ALIGN;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SPECS_ERR_CUDA;
    return launch_merge_partials(ctx, partials, shards, rows, token_ids, V, tok_logprob,
                                 static_cast<cudaStream_t>(cuda_stream));
}

int specs_quantize_rows_e4m3(specs_ctx* ctx, const void* x_bf16, int64_t n, int32_t d, uint8_t* codes, float* scale,
                             void* cuda_stream) {
    if (!ctx) return SPECS_ERR_NULL;
    if (n < 0 || d <= 0 || (d % 16) != 0) return SPECS_ERR_SHAPE;
    if (n == 0) return SPECS_OK;
    if (!x_bf16 || !codes || !scale) return SPECS_ERR_NULL;
    if (!aligned16(x_bf16) || !aligned16(codes)) return SPECS_ERR_ALIGN;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SPECS_ERR_CUDA;
    return launch_quantize_rows(x_bf16, n, d, codes, scale, static_cast<cudaStream_t>(cuda_stream));
}

static ScorePlan fp8_plan(const specs_ctx* ctx, int64_t rows, int32_t d, int32_t V) {
    const int cta_group = ctx->engine == SPECS_ENGINE_TCGEN05_1CTA ? 1
                        : ctx->engine == SPECS_ENGINE_TCGEN05_2CTA ? 2 : kCtaGroupAuto;
    return make_score_plan(rows, d, V, ctx->num_sms, ctx->pair_units, cta_group, ctx->chunk_kblocks,
                           ctx->accum_adaptive, 1);
}

size_t specs_score_workspace_bytes_fp8(const specs_ctx* ctx, int64_t rows, int32_t d, int32_t V) {
    if (!ctx || check_score_shapes(rows, d, V, 0) != SPECS_OK || (d % 16) != 0) return 0;
    const size_t one = plan_workspace_bytes(make_score_plan(rows, d, V, ctx->num_sms, ctx->pair_units, 1,
                                                            kDefaultChunkKBlocks, true, 1));
    const size_t two = plan_workspace_bytes(make_score_plan(rows, d, V, ctx->num_sms, ctx->pair_units, 2,
                                                            kDefaultChunkKBlocks, true, 1));
    return one > two ? one : two;
}

int specs_score_blocks_fp8(specs_ctx* ctx, const uint8_t* hidden_q, const float* hidden_scale, const uint8_t* W_q,
                           const float* W_scale, const int32_t* token_ids, const int64_t* block_offsets, int64_t rows,
                           int32_t d, int32_t V, int32_t B, float* tok_logprob, float* blk_logprob,
                           double* blk_logprob_f64, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!ctx) return SPECS_ERR_NULL;
    int st = check_score_shapes(rows, d, V, B);
    if (st != SPECS_OK) return st;
    if ((d % 16) != 0) return SPECS_ERR_SHAPE;               // rows of 8-bit codes must start on 16-byte boundaries
    if (!W_q || !W_scale || (B > 0 && !block_offsets)) return SPECS_ERR_NULL;
    if (rows > 0 && (!hidden_q || !hidden_scale || !token_ids || !tok_logprob || !workspace)) return SPECS_ERR_NULL;
    if (!aligned16(hidden_q) || !aligned16(W_q) || !aligned16(workspace)) return SPECS_ERR_ALIGN;
    if (ctx->engine == SPECS_ENGINE_SIMT) return SPECS_ERR_SHAPE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SPECS_ERR_CUDA;
    if (rows > 0) {
        const ScorePlan plan = fp8_plan(ctx, rows, d, V);
        if (workspace_bytes < plan_workspace_bytes(plan)) return SPECS_ERR_WORKSPACE;
        st = score_rows(ctx, plan, hidden_q, W_q, token_ids, workspace, stream, 0, hidden_scale, W_scale, tok_logprob,
                        nullptr, false);
        if (st != SPECS_OK) return st;
    }
    if (B > 0 && (blk_logprob || blk_logprob_f64))
        return launch_block_sums(tok_logprob, block_offsets, B, blk_logprob, blk_logprob_f64, stream);
    return SPECS_OK;
}

// layout of the fused 8-bit step's workspace: [codes of the hidden states | their scales | scoring workspace]
static size_t fp8_step_offsets(int64_t rows, int32_t d, size_t* off_scale, size_t* off_ws) {
    const size_t codes = ((size_t)rows * d + 255) & ~(size_t)255;
    const size_t scales = ((size_t)rows * sizeof(float) + 255) & ~(size_t)255;
    *off_scale = codes;
    *off_ws = codes + scales;
    return codes + scales;
}

size_t specs_beam_step_fp8_workspace_bytes(const specs_ctx* ctx, int64_t rows, int32_t d, int32_t V) {
    const size_t ws = specs_score_workspace_bytes_fp8(ctx, rows, d, V);
    if (ws == 0) return 0;
    size_t o1, o2;
    return fp8_step_offsets(rows, d, &o1, &o2) + ws;
}

int specs_beam_step_fp8(specs_ctx* ctx, const void* hidden, const uint8_t* W_q, const float* W_scale,
                        const int32_t* token_ids, const int64_t* block_offsets, const int32_t* cand_offsets,
                        const float* gen_tok_logprob, const float* reward, const float* uniforms, int64_t rows,
                        int32_t d, int32_t V, int32_t B, int32_t P, float beta, float tau, float* tok_logprob,
                        double* blk_logprob_f64, double* gen_blk_logprob_f64, float* weights, int32_t* chosen,
                        uint8_t* accept, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!ctx) return SPECS_ERR_NULL;
    int st = check_score_shapes(rows, d, V, B);
    if (st != SPECS_OK) return st;
    if (P < 0 || (d % 16) != 0) return SPECS_ERR_SHAPE;
    if (P == 0) return SPECS_OK;
    if (!W_q || !W_scale || !block_offsets || !cand_offsets || !chosen) return SPECS_ERR_NULL;
    if (rows > 0 && (!hidden || !token_ids || !tok_logprob || !workspace)) return SPECS_ERR_NULL;
    if (B > 0 && (!reward || !uniforms || !blk_logprob_f64 || (gen_tok_logprob && !gen_blk_logprob_f64)))
        return SPECS_ERR_NULL;
    if (!aligned16(hidden) || !aligned16(W_q) || !aligned16(workspace)) return SPECS_ERR_ALIGN;
    if (ctx->engine == SPECS_ENGINE_SIMT) return SPECS_ERR_SHAPE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SPECS_ERR_CUDA;

    const ScorePlan plan = fp8_plan(ctx, rows, d, V);
    size_t off_scale, off_ws;
    const size_t head = fp8_step_offsets(rows, d, &off_scale, &off_ws);
    uint8_t* base = static_cast<uint8_t*>(workspace);
    uint8_t* ws = base + off_ws;
    if (rows > 0) {
        if (workspace_bytes < head + plan_workspace_bytes(plan)) return SPECS_ERR_WORKSPACE;
        float* h_scale = reinterpret_cast<float*>(base + off_scale);
        st = launch_quantize_rows(hidden, rows, d, base, h_scale, stream);
        if (st != SPECS_OK) return st;
        st = score_rows(ctx, plan, base, W_q, token_ids, ws, stream, 0, h_scale, W_scale, tok_logprob, nullptr, true,
                        true);
        if (st != SPECS_OK) return st;
    }
    return launch_finish_step(ctx, plan, rows > 0 ? fix_view(plan, ws) : kNoFix, nullptr, kNoFix, token_ids,
                              block_offsets, cand_offsets, P,
                              const_cast<float*>(gen_tok_logprob), reward, uniforms, beta, tau, tok_logprob,
                              blk_logprob_f64, gen_blk_logprob_f64, weights, chosen, accept, nullptr, nullptr, 0,
                              rows > 0 && merge_in_finish(plan) ? reinterpret_cast<const float*>(ws) : nullptr, stream);
}

int specs_block_sums(specs_ctx* ctx, const float* per_token, const int64_t* block_offsets, int32_t B, float* out,
                     double* out_f64, void* cuda_stream) {
    if (!ctx) return SPECS_ERR_NULL;
    if (B < 0) return SPECS_ERR_SHAPE;
    if (B == 0) return SPECS_OK;
    if (!block_offsets || (!out && !out_f64)) return SPECS_ERR_NULL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SPECS_ERR_CUDA;
    return launch_block_sums(per_token, block_offsets, B, out, out_f64, static_cast<cudaStream_t>(cuda_stream));
}

static int subsample_common(specs_ctx* ctx, const void* lp_t, const void* lp_g, bool f64, const float* reward,
                            const int32_t* cand_offsets, int32_t P, float beta, const float* uniforms,
                            int32_t* chosen, float* weights, float tau, uint8_t* accept, void* cuda_stream) {
    if (!ctx) return SPECS_ERR_NULL;
    if (P < 0) return SPECS_ERR_SHAPE;
    if (P == 0) return SPECS_OK;
    if (!reward || !cand_offsets || !uniforms || !chosen) return SPECS_ERR_NULL;
    if (lp_g && !lp_t) return SPECS_ERR_NULL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SPECS_ERR_CUDA;
    return launch_subsample(lp_t, lp_g, f64, reward, cand_offsets, P, beta, uniforms, chosen, weights, tau, accept,
                            static_cast<cudaStream_t>(cuda_stream));
}

int specs_subsample(specs_ctx* ctx, const float* blk_lp_target, const float* blk_lp_gen, const float* reward,
                    const int32_t* cand_offsets, int32_t P, float beta, const float* uniforms, int32_t* chosen,
                    float* weights, float tau, uint8_t* accept, void* cuda_stream) {
    return subsample_common(ctx, blk_lp_target, blk_lp_gen, false, reward, cand_offsets, P, beta, uniforms, chosen,
                            weights, tau, accept, cuda_stream);
}

int specs_subsample_f64(specs_ctx* ctx, const double* blk_lp_target, const double* blk_lp_gen, const float* reward,
                        const int32_t* cand_offsets, int32_t P, float beta, const float* uniforms, int32_t* chosen,
                        float* weights, float tau, uint8_t* accept, void* cuda_stream) {
    return subsample_common(ctx, blk_lp_target, blk_lp_gen, true, reward, cand_offsets, P, beta, uniforms, chosen,
                            weights, tau, accept, cuda_stream);
}

int specs_select(specs_ctx* ctx, const double* blk_lp_target, const double* blk_lp_gen, const float* reward,
                 const uint8_t* mask, const int32_t* cand_offsets, int32_t P, float beta, const float* uniforms,
                 int select_rule, int score_flags, int switch_rule, float tau, int32_t* chosen, float* weights,
                 uint8_t* flag, void* cuda_stream) {
    if (!ctx) return SPECS_ERR_NULL;
    if (P < 0) return SPECS_ERR_SHAPE;
    if (select_rule != SPECS_SELECT_SUBSAMPLE && select_rule != SPECS_SELECT_BEST_REWARD) return SPECS_ERR_SHAPE;
    if (switch_rule < SPECS_SWITCH_ANY_ABOVE || switch_rule > SPECS_SWITCH_CHOSEN_BELOW) return SPECS_ERR_SHAPE;
    if (score_flags & ~SPECS_SCORE_NO_LL) return SPECS_ERR_SHAPE;
    if (P == 0) return SPECS_OK;
    if (!reward || !cand_offsets || !chosen) return SPECS_ERR_NULL;
    if (select_rule == SPECS_SELECT_SUBSAMPLE && !uniforms) return SPECS_ERR_NULL;
    if (blk_lp_gen && !blk_lp_target) return SPECS_ERR_NULL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SPECS_ERR_CUDA;
    return launch_select(blk_lp_target, blk_lp_gen, reward, mask, cand_offsets, P, beta, uniforms, select_rule,
                         score_flags, switch_rule, tau, chosen, weights, flag, static_cast<cudaStream_t>(cuda_stream));
}

int specs_prm_rewards(specs_ctx* ctx, const void* prm_hidden, const int64_t* block_offsets, int32_t B, int32_t d,
                      const void* w_head, float bias, float* reward, void* cuda_stream) {
    if (!ctx) return SPECS_ERR_NULL;
    if (B < 0 || d <= 0 || (d % 8) != 0) return SPECS_ERR_SHAPE;
    if (B == 0) return SPECS_OK;
    if (!prm_hidden || !block_offsets || !w_head || !reward) return SPECS_ERR_NULL;
    if (!aligned16(prm_hidden) || !aligned16(w_head)) return SPECS_ERR_ALIGN;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SPECS_ERR_CUDA;
    return launch_prm_head(prm_hidden, block_offsets, B, d, w_head, bias, reward,
                           static_cast<cudaStream_t>(cuda_stream));
}

int specs_accept(specs_ctx* ctx, const float* reward, const int32_t* cand_offsets, int32_t P, float tau,
                 uint8_t* accept, void* cuda_stream) {
    if (!ctx) return SPECS_ERR_NULL;
    if (P < 0) return SPECS_ERR_SHAPE;
    if (P == 0) return SPECS_OK;
    if (!reward || !cand_offsets || !accept) return SPECS_ERR_NULL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SPECS_ERR_CUDA;
    return launch_accept(reward, cand_offsets, P, tau, accept, static_cast<cudaStream_t>(cuda_stream));
}

int specs_beam_step(specs_ctx* ctx, const void* hidden, const void* W_vocab, const int32_t* token_ids,
                    const int64_t* block_offsets, const int32_t* cand_offsets, const float* gen_tok_logprob,
                    const float* reward, const float* uniforms, int64_t rows, int32_t d, int32_t V, int32_t B,
                    int32_t P, float beta, float tau, float* tok_logprob, double* blk_logprob_f64,
                    double* gen_blk_logprob_f64, float* weights, int32_t* chosen, uint8_t* accept, void* workspace,
                    size_t workspace_bytes, void* cuda_stream) {
    if (!ctx) return SPECS_ERR_NULL;
    int st = check_score_shapes(rows, d, V, B);
    if (st != SPECS_OK) return st;
    if (P < 0) return SPECS_ERR_SHAPE;
    if (P == 0) return SPECS_OK;
    if (!W_vocab || !block_offsets || !cand_offsets || !chosen) return SPECS_ERR_NULL;
    if (rows > 0 && (!hidden || !token_ids || !tok_logprob || !workspace)) return SPECS_ERR_NULL;
    if (B > 0 && (!reward || !uniforms || !blk_logprob_f64 || (gen_tok_logprob && !gen_blk_logprob_f64)))
        return SPECS_ERR_NULL;
    if (!aligned16(hidden) || !aligned16(W_vocab) || !aligned16(workspace)) return SPECS_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SPECS_ERR_CUDA;
    if (ctx->engine == SPECS_ENGINE_SIMT) return SPECS_ERR_SHAPE;         // the fused step is tensor-core only

    const int cta_group = ctx->engine == SPECS_ENGINE_TCGEN05_1CTA ? 1
                        : ctx->engine == SPECS_ENGINE_TCGEN05_2CTA ? 2 : kCtaGroupAuto;
    const ScorePlan plan = make_score_plan(rows, d, V, ctx->num_sms, ctx->pair_units, cta_group, ctx->chunk_kblocks,
                                           ctx->accum_adaptive);
    if (rows > 0) {
        if (workspace_bytes < plan_workspace_bytes(plan)) return SPECS_ERR_WORKSPACE;
        st = score_rows(ctx, plan, hidden, W_vocab, token_ids, workspace, stream, 0, nullptr, nullptr, tok_logprob,
                        nullptr, true, true);
        if (st != SPECS_OK) return st;
    }
    // the finish kernel only reads the generator's log-probabilities on this route
    return launch_finish_step(ctx, plan, rows > 0 ? fix_view(plan, workspace) : kNoFix, nullptr, kNoFix, token_ids,
                              block_offsets, cand_offsets, P, const_cast<float*>(gen_tok_logprob), reward, uniforms,
                              beta, tau, tok_logprob, blk_logprob_f64, gen_blk_logprob_f64, weights, chosen, accept,
                              nullptr, nullptr, 0,
                              rows > 0 && merge_in_finish(plan) ? static_cast<const float*>(workspace) : nullptr, stream);
}

size_t specs_beam_step_dual_workspace_bytes(const specs_ctx* ctx, int64_t rows, int32_t d_target, int32_t d_gen,
                                            int32_t V) {
    const size_t t = specs_score_workspace_bytes(ctx, rows, d_target, V);
    const size_t g = specs_score_workspace_bytes(ctx, rows, d_gen, V);
    if (t == 0 || g == 0) return 0;
    return ((t + 255) & ~(size_t)255) + g;
}

int specs_beam_step_dual(specs_ctx* ctx, const void* hidden_target, const void* W_target, int32_t d_target,
                         const void* hidden_gen, const void* W_gen, int32_t d_gen, const int32_t* token_ids,
                         const int64_t* block_offsets, const int32_t* cand_offsets, const float* reward,
                         const float* uniforms, int64_t rows, int32_t V, int32_t B, int32_t P, float beta, float tau,
                         float* tok_logprob, float* gen_tok_logprob, double* blk_logprob_f64,
                         double* gen_blk_logprob_f64, float* weights, int32_t* chosen, uint8_t* accept,
                         int32_t* chosen_ids, int32_t* chosen_len, int32_t chosen_stride, void* workspace,
                         size_t workspace_bytes, void* cuda_stream) {
    if (!ctx) return SPECS_ERR_NULL;
    int st = check_score_shapes(rows, d_target, V, B);
    if (st != SPECS_OK) return st;
    if ((st = check_score_shapes(rows, d_gen, V, B)) != SPECS_OK) return st;
    if (P < 0 || (chosen_ids && chosen_stride <= 0)) return SPECS_ERR_SHAPE;
    if (P == 0) return SPECS_OK;
    if (!W_target || !W_gen || !block_offsets || !cand_offsets || !chosen || (chosen_ids && !chosen_len))
        return SPECS_ERR_NULL;
    if (rows > 0 && (!hidden_target || !hidden_gen || !token_ids || !tok_logprob || !gen_tok_logprob || !workspace))
        return SPECS_ERR_NULL;
    if (B > 0 && (!reward || !uniforms || !blk_logprob_f64 || !gen_blk_logprob_f64)) return SPECS_ERR_NULL;
    if (!aligned16(hidden_target) || !aligned16(W_target) || !aligned16(hidden_gen) || !aligned16(W_gen) ||
        !aligned16(workspace))
        return SPECS_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SPECS_ERR_CUDA;
    if (ctx->engine == SPECS_ENGINE_SIMT) return SPECS_ERR_SHAPE;

    const int cta_group = ctx->engine == SPECS_ENGINE_TCGEN05_1CTA ? 1
                        : ctx->engine == SPECS_ENGINE_TCGEN05_2CTA ? 2 : kCtaGroupAuto;
    const ScorePlan plan_t = make_score_plan(rows, d_target, V, ctx->num_sms, ctx->pair_units, cta_group,
                                             ctx->chunk_kblocks, ctx->accum_adaptive);
    const ScorePlan plan_g = make_score_plan(rows, d_gen, V, ctx->num_sms, ctx->pair_units, cta_group,
                                             ctx->chunk_kblocks, ctx->accum_adaptive);
    const size_t off_g = (plan_workspace_bytes(plan_t) + 255) & ~(size_t)255;
    uint8_t* ws_t = static_cast<uint8_t*>(workspace);
    uint8_t* ws_g = ws_t + off_g;
    if (rows > 0) {
        if (workspace_bytes < off_g + plan_workspace_bytes(plan_g)) return SPECS_ERR_WORKSPACE;
        // the generator's (smaller) head first; both heads are done when the finish kernel starts
        st = score_rows(ctx, plan_g, hidden_gen, W_gen, token_ids, ws_g, stream, 0, nullptr, nullptr, gen_tok_logprob,
                        nullptr, true);
        if (st != SPECS_OK) return st;
        st = score_rows(ctx, plan_t, hidden_target, W_target, token_ids, ws_t, stream, 0, nullptr, nullptr,
                        tok_logprob, nullptr, true);
        if (st != SPECS_OK) return st;
    }
    return launch_finish_step(ctx, plan_t, rows > 0 ? fix_view(plan_t, ws_t) : kNoFix, &plan_g,
                              rows > 0 ? fix_view(plan_g, ws_g) : kNoFix, token_ids, block_offsets,
                              cand_offsets, P, gen_tok_logprob, reward, uniforms, beta, tau, tok_logprob,
                              blk_logprob_f64, gen_blk_logprob_f64, weights, chosen, accept, chosen_ids, chosen_len,
                              chosen_stride, nullptr, stream);
}

int specs_gather_chosen(specs_ctx* ctx, const int32_t* token_ids, const int64_t* block_offsets,
                        const int32_t* cand_offsets, const int32_t* chosen, int32_t P, int32_t* chosen_ids,
                        int32_t* chosen_len, int32_t chosen_stride, void* cuda_stream) {
    if (!ctx) return SPECS_ERR_NULL;
    if (P < 0 || chosen_stride <= 0) return SPECS_ERR_SHAPE;
    if (P == 0) return SPECS_OK;
    if (!block_offsets || !cand_offsets || !chosen || !chosen_ids || !chosen_len) return SPECS_ERR_NULL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SPECS_ERR_CUDA;
    return launch_gather_chosen(token_ids, block_offsets, cand_offsets, chosen, P, chosen_ids, chosen_len,
                                chosen_stride, static_cast<cudaStream_t>(cuda_stream));
}

int specs_device_status(specs_ctx* ctx, uint32_t* h_bits, void* cuda_stream) {
    if (!ctx) return SPECS_ERR_NULL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SPECS_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    uint32_t bits = 0;
    if (cudaMemcpyAsync(&bits, ctx->d_status, sizeof(bits), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaMemsetAsync(ctx->d_status, 0, sizeof(bits), stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess)
        return SPECS_ERR_CUDA;
    if (h_bits) *h_bits = bits;
    if (bits & SPECS_DEV_TIMEOUT) return SPECS_ERR_DEVICE_TIMEOUT;
    if (bits & SPECS_DEV_BOUNDS) return SPECS_ERR_DEVICE_BOUNDS;
    if (bits & SPECS_DEV_TOKEN_RANGE) return SPECS_ERR_TOKEN_RANGE;
    return SPECS_OK;
}

int specs_probe_wait_expiry(specs_ctx* ctx, int64_t limit_us, void* cuda_stream) {
    if (!ctx) return SPECS_ERR_NULL;
    if (limit_us <= 0 || limit_us > 1000000) return SPECS_ERR_SHAPE;   // at most one second
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SPECS_ERR_CUDA;
    return launch_wait_expiry_probe(ctx, (unsigned long long)limit_us * 1000ull, static_cast<cudaStream_t>(cuda_stream));
}

int specs_set_timing(specs_ctx* ctx, int enabled) {
    if (!ctx) return SPECS_ERR_NULL;
    if (enabled < 0 || enabled > 2) return SPECS_ERR_SHAPE;
    ctx->timing = enabled != 0;
    if (enabled == 1) ctx->timed_used = 0;                   // a fresh start forgets earlier records
    return SPECS_OK;
}

float specs_score_kernel_ms(specs_ctx* ctx, int32_t* h_launches) {
    if (h_launches) *h_launches = 0;
    if (!ctx || ctx->timed_used == 0) return -1.0f;
    DeviceGuard guard(ctx->device);
    double total = 0.0;
    size_t first_passes = 0;
    for (size_t i = 0; i < ctx->timed_used; ++i) {
        float ms = 0.0f;
        if (cudaEventSynchronize(ctx->timed[i].stop) != cudaSuccess ||
            cudaEventElapsedTime(&ms, ctx->timed[i].start, ctx->timed[i].stop) != cudaSuccess)
            return -1.0f;
        total += ms;
        if (!ctx->timed[i].second_pass) ++first_passes;
    }
    if (first_passes == 0) first_passes = 1;
    if (h_launches) *h_launches = (int32_t)first_passes;
    // per scoring call: its pass over all rows plus its second pass over the re-scored rows
    const float mean = (float)(total / (double)first_passes);
    ctx->timed_used = 0;
    return mean;
}

int specs_beam_step_host_submit(specs_ctx* ctx, const void* h_hidden, const void* W_vocab, const int32_t* h_token_ids,
                                const int64_t* h_block_offsets, const int32_t* h_cand_offsets,
                                const float* h_gen_tok_logprob, const float* h_reward, const float* h_uniforms,
                                int64_t rows, int32_t d, int32_t V, int32_t B, int32_t P, float beta, float tau,
                                float* h_tok_logprob, double* h_blk_logprob, float* h_weights, int32_t* h_chosen,
                                uint8_t* h_accept, void* cuda_stream, int32_t* h_ticket) {
    if (!ctx || !h_ticket) return SPECS_ERR_NULL;
    int st = check_score_shapes(rows, d, V, B);
    if (st != SPECS_OK) return st;
    if (P < 0) return SPECS_ERR_SHAPE;
    if (!W_vocab || !h_block_offsets || !h_cand_offsets || !h_chosen) return SPECS_ERR_NULL;
    if (rows > 0 && (!h_hidden || !h_token_ids)) return SPECS_ERR_NULL;
    if (B > 0 && (!h_reward || !h_uniforms)) return SPECS_ERR_NULL;
    if (!aligned16(W_vocab)) return SPECS_ERR_ALIGN;
    if ((st = check_offsets64(h_block_offsets, B, rows)) != SPECS_OK) return st;
    if ((st = check_offsets32(h_cand_offsets, P, B)) != SPECS_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SPECS_ERR_CUDA;

    HostSlot& slot = ctx->host_slots[ctx->next_ticket & 1u];
    if (slot.busy) return SPECS_ERR_LIMIT;                   // two steps in flight at most: wait for the older one
    if (!ctx->copy_in && (cudaStreamCreateWithFlags(&ctx->copy_in, cudaStreamNonBlocking) != cudaSuccess ||
                          cudaStreamCreateWithFlags(&ctx->copy_out, cudaStreamNonBlocking) != cudaSuccess))
        return SPECS_ERR_CUDA;
    if (!slot.ev_in && (cudaEventCreateWithFlags(&slot.ev_in, cudaEventDisableTiming) != cudaSuccess ||
                        cudaEventCreateWithFlags(&slot.ev_done, cudaEventDisableTiming) != cudaSuccess ||
                        cudaEventCreateWithFlags(&slot.ev_out, cudaEventDisableTiming) != cudaSuccess))
        return SPECS_ERR_CUDA;

    // Carve the arena (every piece 256-byte aligned): hidden states, then one block of the small inputs, then
    // one block of the outputs, then what never crosses the bus.  The two blocks are mirrored in a pinned
    // staging buffer so that each crosses in ONE copy instead of one copy per array.
    size_t off = 0;
    auto carve = [&off](size_t bytes) { const size_t at = off; off += (bytes + 255) & ~(size_t)255; return at; };
    const size_t o_hidden = carve((size_t)rows * d * 2);
    const size_t in0 = off;
    const size_t o_ids = carve((size_t)rows * 4), o_boff = carve((size_t)(B + 1) * 8), o_coff = carve((size_t)(P + 1) * 4);
    const size_t o_gen = carve((size_t)rows * 4), o_rew = carve((size_t)B * 4), o_uni = carve((size_t)B * 4);
    const size_t out0 = off;
    const size_t o_tok = carve((size_t)rows * 4), o_blk_t = carve((size_t)B * 8), o_wts = carve((size_t)B * 4);
    const size_t o_cho = carve((size_t)P * 4), o_acc = carve((size_t)P);
    const size_t out1 = off;
    const size_t o_blk_g = carve((size_t)B * 8);
    const size_t ws_bytes = specs_score_workspace_bytes(ctx, rows, d, V);
    const size_t o_ws = carve(ws_bytes);
    // the slot is idle (its last step was waited for), so its buffers may be replaced
    if (off > slot.arena_bytes) {
        if (slot.arena) { cudaFree(slot.arena); slot.arena = nullptr; slot.arena_bytes = 0; }
        if (cudaMalloc(&slot.arena, off) != cudaSuccess) return SPECS_ERR_CUDA;
        slot.arena_bytes = off;
    }
    const size_t stage_bytes = out1 - in0;
    if (stage_bytes > slot.stage_bytes) {
        if (slot.h_stage) { cudaFreeHost(slot.h_stage); slot.h_stage = nullptr; slot.stage_bytes = 0; }
        if (cudaMallocHost(&slot.h_stage, stage_bytes) != cudaSuccess) return SPECS_ERR_CUDA;
        slot.stage_bytes = stage_bytes;
    }
    uint8_t* A = static_cast<uint8_t*>(slot.arena);
    uint8_t* S = static_cast<uint8_t*>(slot.h_stage) - in0;          // S + offset mirrors A + offset
    auto put = [&](size_t at, const void* src, size_t bytes) { if (src && bytes) std::memcpy(S + at, src, bytes); };
    put(o_ids, h_token_ids, (size_t)rows * 4);
    put(o_boff, h_block_offsets, (size_t)(B + 1) * 8);
    put(o_coff, h_cand_offsets, (size_t)(P + 1) * 4);
    put(o_gen, h_gen_tok_logprob, (size_t)rows * 4);
    put(o_rew, h_reward, (size_t)B * 4);
    put(o_uni, h_uniforms, (size_t)B * 4);
    // inputs on the inbound copy stream, kernels on the caller's stream, results on the outbound copy stream
    if (rows > 0 && cudaMemcpyAsync(A + o_hidden, h_hidden, (size_t)rows * d * 2, cudaMemcpyHostToDevice,
                                    ctx->copy_in) != cudaSuccess)
        return SPECS_ERR_CUDA;
    if (cudaMemcpyAsync(A + in0, S + in0, out0 - in0, cudaMemcpyHostToDevice, ctx->copy_in) != cudaSuccess ||
        cudaEventRecord(slot.ev_in, ctx->copy_in) != cudaSuccess ||
        cudaStreamWaitEvent(stream, slot.ev_in, 0) != cudaSuccess)
        return SPECS_ERR_CUDA;

    st = specs_beam_step(ctx, A + o_hidden, W_vocab, reinterpret_cast<int32_t*>(A + o_ids),
                         reinterpret_cast<int64_t*>(A + o_boff), reinterpret_cast<int32_t*>(A + o_coff),
                         h_gen_tok_logprob ? reinterpret_cast<float*>(A + o_gen) : nullptr,
                         reinterpret_cast<float*>(A + o_rew), reinterpret_cast<float*>(A + o_uni), rows, d, V, B, P,
                         beta, tau, reinterpret_cast<float*>(A + o_tok), reinterpret_cast<double*>(A + o_blk_t),
                         reinterpret_cast<double*>(A + o_blk_g), reinterpret_cast<float*>(A + o_wts),
                         reinterpret_cast<int32_t*>(A + o_cho), reinterpret_cast<uint8_t*>(A + o_acc), A + o_ws,
                         ws_bytes, cuda_stream);
    if (st != SPECS_OK) return st;
    if (cudaEventRecord(slot.ev_done, stream) != cudaSuccess ||
        cudaStreamWaitEvent(ctx->copy_out, slot.ev_done, 0) != cudaSuccess ||
        cudaMemcpyAsync(S + out0, A + out0, out1 - out0, cudaMemcpyDeviceToHost, ctx->copy_out) != cudaSuccess ||
        cudaEventRecord(slot.ev_out, ctx->copy_out) != cudaSuccess)
        return SPECS_ERR_CUDA;
    slot.busy = true;
    slot.ticket = ctx->next_ticket++;
    slot.in0 = in0; slot.o_tok = o_tok; slot.o_blk = o_blk_t; slot.o_wts = o_wts; slot.o_cho = o_cho; slot.o_acc = o_acc;
    slot.rows = rows; slot.B = B; slot.P = P;
    slot.h_tok = h_tok_logprob; slot.h_blk = h_blk_logprob; slot.h_wts = h_weights; slot.h_cho = h_chosen;
    slot.h_acc = h_accept;
    *h_ticket = (int32_t)(slot.ticket & 0x7fffffffu);
    return SPECS_OK;
}

int specs_beam_step_host_wait(specs_ctx* ctx, int32_t ticket) {
    if (!ctx) return SPECS_ERR_NULL;
    HostSlot& slot = ctx->host_slots[(uint32_t)ticket & 1u];
    if (!slot.busy || (int32_t)(slot.ticket & 0x7fffffffu) != ticket) return SPECS_ERR_SHAPE;   // no such step in flight
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SPECS_ERR_CUDA;
    slot.busy = false;
    if (cudaEventSynchronize(slot.ev_out) != cudaSuccess) return SPECS_ERR_CUDA;
    const uint8_t* S = static_cast<const uint8_t*>(slot.h_stage) - slot.in0;
    auto get = [&](void* dst, size_t at, size_t bytes) { if (dst && bytes) std::memcpy(dst, S + at, bytes); };
    get(slot.h_tok, slot.o_tok, (size_t)slot.rows * 4);
    get(slot.h_blk, slot.o_blk, (size_t)slot.B * 8);
    get(slot.h_wts, slot.o_wts, (size_t)slot.B * 4);
    get(slot.h_cho, slot.o_cho, (size_t)slot.P * 4);
    get(slot.h_acc, slot.o_acc, (size_t)slot.P);
    return SPECS_OK;
}

int specs_beam_step_host(specs_ctx* ctx, const void* h_hidden, const void* W_vocab, const int32_t* h_token_ids,
                         const int64_t* h_block_offsets, const int32_t* h_cand_offsets,
                         const float* h_gen_tok_logprob, const float* h_reward, const float* h_uniforms,
                         int64_t rows, int32_t d, int32_t V, int32_t B, int32_t P, float beta, float tau,
                         float* h_tok_logprob, double* h_blk_logprob, float* h_weights, int32_t* h_chosen,
                         uint8_t* h_accept, void* cuda_stream) {
    int32_t ticket = 0;
    const int st = specs_beam_step_host_submit(ctx, h_hidden, W_vocab, h_token_ids, h_block_offsets, h_cand_offsets,
                                               h_gen_tok_logprob, h_reward, h_uniforms, rows, d, V, B, P, beta, tau,
                                               h_tok_logprob, h_blk_logprob, h_weights, h_chosen, h_accept,
                                               cuda_stream, &ticket);
    if (st != SPECS_OK) return st;
    return specs_beam_step_host_wait(ctx, ticket);
}

}  // extern "C"
