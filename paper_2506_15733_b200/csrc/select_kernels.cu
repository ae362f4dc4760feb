// The small kernels after the LM-head pass:
//   merge_splits_kernel   combines the per-chunk (max, sum-exp, logit) triples of a row into
//                         log pi_target of the drafted token;
//   block_sums_kernel     warp-level segmented sum of per-token log-probabilities per drafted
//                         block (the block probability of Eq. (1) is the product over its tokens);
//   subsample_kernel      one warp per problem: scores of Eq. (1), the normalised weights of
//                         Algorithm 2, a Gumbel-max draw from caller-supplied uniforms and the
//                         switch test of Algorithm 1, Step III;
//   accept_kernel         the switch test alone.
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
// that saw no valid column (vocabulary tail) carries max = -inf, sum = 0.
constexpr int kMergeWarps = 8;                              // warps per block: each takes every 8th split

__global__ void __launch_bounds__(32 * kMergeWarps)
merge_splits_kernel(const ScorePlan plan, const float* __restrict__ workspace,
                    const int32_t* __restrict__ token_ids, float* __restrict__ tok_logprob,
                    uint32_t* __restrict__ status) {
    // A block owns 32 consecutive rows (lane = row, so loads are coalesced); its warps share the
    // vocabulary splits of those rows and combine their partial (max, sum, logit) in shared memory.
    __shared__ float sh_max[kMergeWarps][32], sh_logit[kMergeWarps][32];
    __shared__ double sh_sum[kMergeWarps][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row = (int64_t)blockIdx.x * 32 + lane;
    const bool live = row < plan.rows;
    const int64_t row_c = live ? row : plan.rows - 1;
    const int mt = (int)(row_c / kBlockM), r = (int)(row_c % kBlockM);
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

    float m = -INFINITY, logit = -INFINITY;
    double sum = 0.0;
    for (int s = warp; s < splits; s += kMergeWarps) {
        const float* p = base + s * stride;
        const float m0 = p[0], s0 = p[kBlockM], t0 = p[2 * kBlockM];
        const float m1 = p[kHalf], s1 = p[kHalf + kBlockM], t1 = p[kHalf + 2 * kBlockM];
        const float mn = fmaxf(m, fmaxf(m0, m1));
        if (mn != -INFINITY) {
            // exp2f(-inf) = 0 takes care of halves and states that have seen nothing yet
            sum = sum * (double)exp2f(m - mn) + (double)s0 * (double)exp2f(m0 - mn) +
                  (double)s1 * (double)exp2f(m1 - mn);
            m = mn;
        }
        logit = fmaxf(logit, fmaxf(t0, t1));
    }
    sh_max[warp][lane] = m; sh_sum[warp][lane] = sum; sh_logit[warp][lane] = logit;
    __syncthreads();
    if (warp != 0 || !live) return;
    float gmax = sh_max[0][lane];
#pragma unroll
    for (int w = 1; w < kMergeWarps; ++w) gmax = fmaxf(gmax, sh_max[w][lane]);
    double total = 0.0;
    float picked = -INFINITY;
#pragma unroll
    for (int w = 0; w < kMergeWarps; ++w) {
        if (sh_max[w][lane] != -INFINITY) total += sh_sum[w][lane] * (double)exp2f(sh_max[w][lane] - gmax);
        picked = fmaxf(picked, sh_logit[w][lane]);
    }
    const int32_t id = token_ids[row];
    if (id < 0 || id >= plan.V) {
        tok_logprob[row] = __int_as_float(0x7fc00000);      // no such vocabulary entry: NaN
        atomicOr(status, SPECS_DEV_TOKEN_RANGE);
        return;
    }
    const double lse = ((double)gmax + log2(total)) * kLn2; // natural-log normaliser
    tok_logprob[row] = (float)((double)picked - lse);
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

template <typename LP>
__global__ void subsample_kernel(const LP* __restrict__ lp_t, const LP* __restrict__ lp_g,
                                 const float* __restrict__ reward, const int32_t* __restrict__ cand_offsets,
                                 int32_t P, float beta, const float* __restrict__ uniforms,
                                 int32_t* __restrict__ chosen, float* __restrict__ weights, float tau,
                                 uint8_t* __restrict__ accept) {
    const int p = (int)(((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
    const int lane = threadIdx.x & 31;
    if (p >= P) return;
    const int a = cand_offsets[p], b = cand_offsets[p + 1];
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

int launch_merge(specs_ctx* ctx, const ScorePlan& plan, const float* workspace, const int32_t* token_ids,
                 float* tok_logprob, cudaStream_t stream) {
    if (plan.rows == 0) return SPECS_OK;
    const unsigned blocks = (unsigned)((plan.rows + 31) / 32);
    merge_splits_kernel<<<blocks, 32 * kMergeWarps, 0, stream>>>(plan, workspace, token_ids, tok_logprob,
                                                                 ctx->d_status);
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

int launch_accept(const float* reward, const int32_t* cand_offsets, int32_t P, float tau, uint8_t* accept,
                  cudaStream_t stream) {
    if (P == 0) return SPECS_OK;
    const int threads = 128;
    accept_kernel<<<warps_grid(P, threads), threads, 0, stream>>>(reward, cand_offsets, P, tau, accept);
    return cuda_status(cudaGetLastError());
}

}  // namespace specs
