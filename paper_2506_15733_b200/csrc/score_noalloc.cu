// specs_score_blocks_noalloc: block scoring for callers that cannot allocate device memory.
//
// The regular entry point needs a context (whose creation calls cudaMalloc for its status
// word) and a caller-allocated workspace.  Some hosts can give neither: an inference server
// that handed the whole device to its own memory pool at start-up has nothing left for
// cudaMalloc to return, and a latency-critical step loop must not run into the device-wide
// synchronisation that cudaMalloc / cudaFree imply.  For them the scratch of the scoring
// kernel (the per-chunk (max, sum-exp, logit) triples) lives in a fixed array in the
// library's own device image, and the call needs no context at all.
//
// Consequences of the fixed array, all part of the contract in specs.h:
//   * every GPU that loads the library carries SPECS_NOALLOC_SCRATCH_BYTES of it until exit;
//   * problems whose plan needs more scratch are refused with SPECS_ERR_LIMIT;
//   * all calls on a device share the array, which still holds the previous call's triples.
//     Nothing in it has to start at zero -- every slot the merge reads is written earlier in
//     the same call -- but two calls whose kernels overlap on the GPU (different streams)
//     would overwrite each other's triples: callers must serialise them.
#include <mutex>

#include "specs_internal.h"

namespace {

// The scratch itself.  In host code this name is only a handle for the runtime, never a
// device address: the address is fetched once per device with cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_noalloc_scratch[SPECS_NOALLOC_SCRATCH_BYTES];
// Sticky status bits for calls that pass no status word of their own (zero at module load).
static __device__ uint32_t g_noalloc_status;

struct DeviceSetup {
    bool ready = false;
    void* scratch = nullptr;
    uint32_t* status = nullptr;
    int num_sms = 0;
    int pair_units = 0;
    specs::EncodeTiledFn encode_tiled = nullptr;
};

constexpr int kMaxDevices = 64;
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

// One-time set-up for the CURRENT device: resolve the device addresses of the two symbols,
// the SM count and the driver's tensor-map encoder.  None of these allocates.
int setup_current_device(int device, DeviceSetup* out) {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    DeviceSetup& s = g_setup[device];
    if (!s.ready) {
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return SPECS_ERR_CUDA;
        if (prop.major != 10) return SPECS_ERR_ARCH;
        void* scratch = nullptr;
        void* status = nullptr;
        if (cudaGetSymbolAddress(&scratch, g_noalloc_scratch) != cudaSuccess || scratch == nullptr)
            return SPECS_ERR_CUDA;
        if (cudaGetSymbolAddress(&status, g_noalloc_status) != cudaSuccess || status == nullptr)
            return SPECS_ERR_CUDA;
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess || fn == nullptr)
            return SPECS_ERR_CUDA;
        s.scratch = scratch;
        s.status = static_cast<uint32_t*>(status);
        s.num_sms = prop.multiProcessorCount;
        s.pair_units = specs::query_pair_units(device, s.num_sms);   // occupancy query and attributes only
        s.encode_tiled = reinterpret_cast<specs::EncodeTiledFn>(fn);
        s.ready = true;
    }
    *out = s;
    return SPECS_OK;
}

}  // namespace

extern "C" int specs_score_blocks_noalloc(const void* hidden, const void* W_vocab, const int32_t* token_ids,
                                          const int64_t* block_offsets, int64_t rows, int32_t d, int32_t V,
                                          int32_t B, float* tok_logprob, float* blk_logprob,
                                          double* blk_logprob_f64, uint32_t* status_word, void* cuda_stream) {
    if (rows < 0 || d <= 0 || (d % 8) != 0 || V <= 0 || B < 0) return SPECS_ERR_SHAPE;
    if (rows > (int64_t)1 << 31) return SPECS_ERR_LIMIT;
    if (!W_vocab || (B > 0 && !block_offsets)) return SPECS_ERR_NULL;
    if (rows > 0 && (!hidden || !token_ids || !tok_logprob)) return SPECS_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(hidden) & 15u) || (reinterpret_cast<uintptr_t>(W_vocab) & 15u))
        return SPECS_ERR_ALIGN;

    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) return SPECS_ERR_CUDA;
    if (device < 0 || device >= kMaxDevices) return SPECS_ERR_LIMIT;
    DeviceSetup setup;
    int st = setup_current_device(device, &setup);
    if (st != SPECS_OK) return st;

    // Fixed 512-element accumulation chunks: exact enough for any logit magnitude without the second
    // pass (and the buffer of gathered rows) that adaptive chunks need, so the scratch stays small.
    const specs::ScorePlan plan = specs::make_score_plan(rows, d, V, setup.num_sms, setup.pair_units,
                                                         specs::kCtaGroupAuto, specs::kDefaultChunkKBlocks, false);
    if (specs::plan_workspace_bytes(plan) > (size_t)SPECS_NOALLOC_SCRATCH_BYTES) return SPECS_ERR_LIMIT;

    // A context that lives on this stack frame only: it carries what the launchers read
    // (device, SM count, encoder, status word) and owns nothing.
    specs_ctx local;
    local.device = device;
    local.num_sms = setup.num_sms;
    local.pair_units = setup.pair_units;
    local.encode_tiled = setup.encode_tiled;
    local.d_status = status_word ? status_word : setup.status;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    if (rows > 0) {
        void* scratch = setup.scratch;
        st = specs::launch_score_tcgen05(&local, plan, hidden, W_vocab, token_ids, scratch, stream);
        if (st != SPECS_OK) return st;
        st = specs::launch_merge(&local, plan, scratch, token_ids, tok_logprob, nullptr, hidden, nullptr, stream);
        if (st != SPECS_OK) return st;
    }
    if (B > 0 && (blk_logprob || blk_logprob_f64))
        return specs::launch_block_sums(tok_logprob, block_offsets, B, blk_logprob, blk_logprob_f64, stream);
    return SPECS_OK;
}
