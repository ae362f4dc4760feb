// Plain CUDA-core scoring kernel: one thread block per drafted row walks the whole vocabulary,
// computing each logit as an fp32 dot product and keeping an online (max, sum-exp, drafted
// logit) state.  It exists to bring the library up and to bisect the tensor-core path on sizes
// the CPU cannot check quickly; it is selected only by an explicit specs_set_engine() call.
// Compiled into the checked build (-DSPECS_DEBUG) only.
#ifdef SPECS_DEBUG
#include <cuda_bf16.h>

#include "specs_internal.h"

namespace specs {
namespace {

constexpr int kSimtThreads = 256;

__device__ __forceinline__ void online_merge(float& m, float& s, float m2, float s2) {
    const float mn = fmaxf(m, m2);
    if (mn == -INFINITY) { m = mn; s = 0.0f; return; }
    s = s * expf(m - mn) + s2 * expf(m2 - mn);
    m = mn;
}

__global__ void __launch_bounds__(kSimtThreads)
score_rows_simt_kernel(const __nv_bfloat16* __restrict__ hidden, const __nv_bfloat16* __restrict__ w_vocab,
                       const int32_t* __restrict__ token_ids, int64_t rows, int32_t d, int32_t V,
                       float* __restrict__ tok_logprob, uint32_t* __restrict__ status) {
    extern __shared__ float h_row[];                 // d floats
    __shared__ float red_m[kSimtThreads / 32], red_s[kSimtThreads / 32], red_t[kSimtThreads / 32];
    const int64_t row = blockIdx.x;
    if (row >= rows) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = kSimtThreads / 32;
    for (int k = threadIdx.x; k < d; k += kSimtThreads) h_row[k] = __bfloat162float(hidden[row * d + k]);
    __syncthreads();

    const int32_t id = token_ids[row];
    float m = -INFINITY, s = 0.0f, t = -INFINITY;
    const int chunks = d / 8;                        // d % 8 == 0: 16-byte loads of 8 bf16
    for (int v = warp; v < V; v += nwarps) {
        const uint4* wrow = reinterpret_cast<const uint4*>(w_vocab + (size_t)v * d);
        float acc = 0.0f;
        for (int c = lane; c < chunks; c += 32) {
            const uint4 q = wrow[c];
            const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&q);
            const float* h = h_row + c * 8;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 f = __bfloat1622float2(p[j]);
                acc = fmaf(f.x, h[2 * j], acc);
                acc = fmaf(f.y, h[2 * j + 1], acc);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        // every lane now holds the logit z_v; lane 0's copy of the state is the one that counts
        if (acc > m) { s = s * expf(m - acc) + 1.0f; m = acc; }
        else         { s += expf(acc - m); }
        if (v == id) t = acc;
    }
    if (lane == 0) { red_m[warp] = m; red_s[warp] = s; red_t[warp] = t; }
    __syncthreads();
    if (threadIdx.x == 0) {
        float M = red_m[0], S = red_s[0], T = red_t[0];
        for (int i = 1; i < nwarps; ++i) {
            online_merge(M, S, red_m[i], red_s[i]);
            T = fmaxf(T, red_t[i]);
        }
        if (id < 0 || id >= V) {
            tok_logprob[row] = __int_as_float(0x7fc00000);
            atomicOr(status, SPECS_DEV_TOKEN_RANGE);
        } else {
            tok_logprob[row] = (float)((double)T - ((double)M + log((double)S)));
        }
    }
}

}  // namespace

int launch_score_simt(specs_ctx* ctx, const void* hidden, const void* w_vocab, const int32_t* token_ids,
                      int64_t rows, int32_t d, int32_t V, float* tok_logprob, cudaStream_t stream) {
    if (rows == 0) return SPECS_OK;
    const size_t smem = (size_t)d * sizeof(float);
    if (smem > 48 * 1024) {
        if (smem > 200 * 1024) return SPECS_ERR_LIMIT;
        if (cudaFuncSetAttribute(score_rows_simt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
            cudaSuccess)
            return SPECS_ERR_CUDA;
    }
    if (rows > 0x7fffffffLL) return SPECS_ERR_LIMIT;
    score_rows_simt_kernel<<<(unsigned)rows, kSimtThreads, smem, stream>>>(
        static_cast<const __nv_bfloat16*>(hidden), static_cast<const __nv_bfloat16*>(w_vocab), token_ids, rows, d, V,
        tok_logprob, ctx->d_status);
    return cuda_status(cudaGetLastError());
}

}  // namespace specs
#endif  // SPECS_DEBUG
