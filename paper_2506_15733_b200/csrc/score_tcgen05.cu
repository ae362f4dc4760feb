// LM-head scoring kernel for sm_100a: hidden[rows,d] x W_vocab[V,d]^T on the 5th-generation
// tensor cores with a fused online log-sum-exp + drafted-logit gather epilogue.  The rows x V
// logits live only in tensor memory (TMEM); what reaches HBM is one (max, sum-exp, logit)
// triple per row and per vocabulary chunk.
//
// This is the "computing logits of each token" step of scoring a drafted block with the
// target model (Section 2 of the paper; Appendix E.3 restricts it to the new block's tokens).
//
// Persistent CTAs, one per SM, 384 threads (three warpgroups), three roles:
//   warp 0      TMA producer: cp.async.bulk.tensor loads of a 128x64 hidden tile and a W tile
//               per k-block into a ring of 128-byte-swizzled shared-memory stages (lane 0).
//               Before each vocabulary tile the warp paces itself against the other units
//               that stream the same W chunk (see "pacing" below), so that a W tile is
//               fetched from HBM once and found in L2 by the rest.
//   warp 1      MMA issuer: one thread issues tcgen05.mma (N=256, K=16, bf16 -> fp32) into one
//               of two 128-lane x 256-column TMEM buffers.  The reduction over d is cut into
//               chunks of plan.chunk_kblocks k-blocks; every chunk starts a fresh accumulator
//               and alternates between the two buffers.
//   warps 4-11  epilogue: thread = one row (TMEM lane) x one half (128 columns) of the tile.
//               After each chunk it adds the chunk's partial logits into fp32 registers
//               (round-to-nearest), which releases the TMEM buffer for the chunk after next;
//               after the last chunk it runs, on those registers, the online update of
//               running max / rescaled sum of 2^x / select of the drafted id's logit.  The
//               state stays in registers across the CTA's run of vocabulary tiles.
//
// Two tile shapes share that body (template parameter kCg = CTAs per work unit):
//   kCg = 1  one CTA owns a 128-row x 256-column tile: 16 KB of hidden states + 32 KB of W per
//            k-block, 4 stages.  At 512 tensor clocks per k-block this needs 96 B/clk/SM from
//            L2, more than the SMs get when all of them stream, so it tops out near 76 % of
//            the tensor pipe; it remains for problems with a single row tile.
//   kCg = 2  two CTAs of one cluster own a 256-row x 256-column tile and the leader (cluster
//            rank 0) issues tcgen05.mma.cta_group::2 over both CTAs' shared memory: each CTA
//            stages its own 128 hidden rows and only its HALF (128 rows) of the W tile, 32 KB
//            per k-block (64 B/clk/SM), 6 stages.  Each CTA's TMEM receives its own 128 rows
//            x 256 columns, so the epilogue is the same.  Barrier traffic across the pair:
//            the peer's TMA loads complete on the leader's "full" barrier; the leader's
//            tcgen05.commit arrives on both CTAs' "empty" and "accumulator full" barriers;
//            both CTAs' epilogue warps arrive on the leader's "accumulator drained" barrier.
//            W tiles are never multicast: each CTA fetches its own half.
//
// Why chunks: the tensor core adds each K=16 group of products into its fp32 accumulator with
// truncation, so a long reduction carries a bias proportional to the accumulator's magnitude
// times the number of accumulations (about -5e-3 on logits near 700 at d = 5120).  Restarting
// the accumulator every 512 elements and summing the chunks in registers with round-to-nearest
// divides that bias by the number of chunks.  Each restart costs a read of the accumulator out
// of TMEM, which holds up the tensor pipe for about 500 clocks, so chunks are only as short as
// the logits demand: with plan.adaptive the first two vocabulary tiles of a run use the base
// chunk; the epilogue warps publish how their rows' largest |logit| of the first tile spread over
// magnitude classes, and from the third tile on the MMA issuer and the epilogue both derive the
// chunk length from the class that all but 1/32 of the tile's samples stay within
// (adaptive_chunk_kblocks).  The hand-over is a barrier ("mode") on which every epilogue warp of
// the unit arrives after writing its counts into every CTA of the unit.
//
// Two passes: a row in which a logit that matters lies beyond the magnitude its chunks were sized
// for (or beyond 1024, the base chunk's own range) leaves the first pass marked (a negative sum).
// The merge collects the marked rows and gathers their hidden states; the same kernel body,
// instantiated as the second pass (template parameter kSecond), re-scores them with short chunks:
// it reads the count first and returns at once when it is zero, derives its plan from the count on
// the device, and scores either the gathered rows or, when they outnumber the gather buffer,
// every row in place.
//
// Pacing: the units (CTAs or pairs) that own the same vocabulary chunk in a wave read the same W
// tiles.  Only while they stay within about a tile of each other does a tile come from HBM once and
// from L2 for the others; left alone they drift apart within milliseconds and every tile is fetched
// several times.  Each unit therefore publishes its progress in a 64-bit word behind the workspace's
// slots and does not pass pace point t before all units of its chunk have passed point t - lead;
// a pace point is the start of a vocabulary tile, or one of several evenly spaced k-blocks of a tile
// where the wave's working set would otherwise outgrow L2 (plan.pace_points).  The wait is advisory
// (bounded, gives up for good after a few expiries).
//
// 8-bit operands (template parameter kFp8): the same kernel on E4M3 codes with per-row scales,
// 128 elements per k-block, tcgen05.mma kind::f8f6f4; the epilogue applies the column scales (staged
// in shared memory per tile) to the accumulators and folds the row's scale into the exponent.
//
// Every mbarrier wait is bounded; on expiry the CTA raises SPECS_DEV_TIMEOUT, all roles leave
// their loops, the producer waits (bounded) for its copies in flight, TMEM is freed and the
// kernel returns.
#include <cuda_bf16.h>

#include <atomic>
#include <map>
#include <mutex>

#include "specs_internal.h"

namespace specs {
namespace {

constexpr int kUmmaK = 16;
constexpr int kMaxStages = 8;
constexpr uint32_t kABytes = kBlockM * kBlockK * 2;      // 16 KB: 128 hidden rows x 64 k
constexpr int kThreads = 384;                            // three warpgroups: control, epilogue, epilogue
// Registers per thread after the warpgroups re-balance them (setmaxnreg).  The increase waits,
// without bound, until the CTA's own allocation (launch registers x threads) has that much to
// give, so the two budgets must fit into it.
constexpr int kLaunchRegs = 168;                         // what __launch_bounds__(384, 1) yields
constexpr int kControlRegs = 120;
constexpr int kEpilogueRegs = 184;
static_assert(128 * kControlRegs + 256 * kEpilogueRegs <= kThreads * kLaunchRegs,
              "setmaxnreg budgets exceed the CTA's register allocation: the increase would never return");
constexpr int kEpilogueWarps = 8;
constexpr int kHalfN = kBlockN / 2;                      // columns per epilogue thread
constexpr uint32_t kTmemCols = 512;                      // two 256-column accumulators
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s per wait
constexpr unsigned long long kDrainLimitNs = 20000000ull;    // 20 ms per stage when draining after an abort
constexpr float kLog2e = 1.4426950408889634f;

constexpr size_t kControlBytes = 5120;                   // barriers, published magnitudes, staged column scales
constexpr int kScaleBufs = 4;                            // vocabulary tiles whose column scales are staged at once

// Per tile shape: W rows staged per CTA and k-block, stage size, ring depth, shared memory.
template <int kCg> struct Shape {
    static constexpr int kBRows = kBlockN / kCg;                         // 256, or this CTA's half
    static constexpr uint32_t kBBytes = kBRows * kBlockK * 2;            // 32 KB / 16 KB
    static constexpr uint32_t kStageBytes = kABytes + kBBytes;           // 48 KB / 32 KB
    static constexpr int kStages = kCg == 1 ? 4 : 6;
    static constexpr size_t kSmemBytes = 1024 /*alignment slack*/ + (size_t)kStages * kStageBytes + kControlBytes;
};

// ---- thin PTX wrappers -------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// ---- cluster helpers (pair kernel) ----
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n"
                 "barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void st_cluster_u32(uint32_t cluster_addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}

// try_wait whose acquire covers writes made by the other CTA of the pair before its arrival
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ void st_cluster_u64(uint32_t cluster_addr, uint64_t v) {
    asm volatile("st.shared::cluster.u64 [%0], %1;" ::"r"(cluster_addr), "l"(v) : "memory");
}

// The abort flag of this CTA and, in the pair kernel, the shared::cluster address of the
// peer's (0: none): a wait that gives up raises both so that the whole unit winds down.
struct AbortFlags {
    volatile uint32_t* own;
    uint32_t peer;
};
// Bounded wait.  Returns false if the abort flag is (or becomes) set.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const AbortFlags& ab,
                                          unsigned long long limit_ns, bool raise, bool cluster_acquire = false) {
    if (cluster_acquire ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    uint32_t spins = 0;
    for (;;) {
        if (cluster_acquire ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
        if ((++spins & 0xFFu) == 0u) {
            if (raise && *ab.own) return false;
            if (global_timer_ns() - t0 > limit_ns) {
                if (raise) {
                    *ab.own = 1u;
                    if (ab.peer) st_cluster_u32(ab.peer, 1u);
                }
                return false;
            }
        }
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c_inner, int c_outer,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c_inner), "r"(c_outer), "r"(bar)
        : "memory");
}
// The same load issued by a CTA of a pair: the data lands in this CTA's shared memory, the bytes
// are counted on the barrier at shared::cluster address `cluster_bar` (the leader's).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c_inner, int c_outer,
                                                 uint32_t cluster_bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c_inner), "r"(c_outer), "r"(cluster_bar)
        : "memory");
}
// 2^x on the special-function unit (relative error about 2^-22; 2^-inf = 0).
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// Commit of the pair's MMAs: arrives on the barrier at this shared-memory offset in BOTH CTAs.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The same two instructions for 8-bit operands (kind::f8f6f4, K = 32 per instruction).
__device__ __forceinline__ void tc_mma_f8_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n"
        "}\n"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_mma_f8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n"
        "}\n"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread i of the warp gets lane (base lane + i).
// The load and its completion wait sit in one statement so that the registers are
// valid as soon as the statement has executed.
__device__ __forceinline__ void tmem_ld_32cols(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
        "tcgen05.wait::ld.sync.aligned;\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
}

// The same for 16 consecutive columns, straight into float registers.
__device__ __forceinline__ void tmem_ld_16cols(uint32_t taddr, float (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n"
        "tcgen05.wait::ld.sync.aligned;\n"
        : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7]), "=f"(v[8]), "=f"(v[9]), "=f"(v[10]), "=f"(v[11]), "=f"(v[12]), "=f"(v[13]), "=f"(v[14]), "=f"(v[15])
        : "r"(taddr)
        : "memory");
}

// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes (64
// elements) long, written by TMA with the 128-byte swizzle: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_k_major_sw128(uint32_t saddr) {
    uint64_t desc = 0;
    desc |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);   // bits  0-13 start address / 16
    desc |= static_cast<uint64_t>(1) << 16;                   // bits 16-29 leading byte offset (unused here)
    desc |= static_cast<uint64_t>(1024 >> 4) << 32;           // bits 32-45 stride byte offset / 16
    desc |= static_cast<uint64_t>(1) << 46;                   // bits 46-47 descriptor version (sm_100)
    desc |= static_cast<uint64_t>(2) << 61;                   // bits 61-63 swizzle mode: 128 bytes
    return desc;
}
// Instruction descriptor of kind::f8f6f4: dense, fp32 accumulate, A and B E4M3 (format code 0), K-major.
__host__ __device__ constexpr uint32_t instr_desc_e4m3(int m, int n) {
    return (1u << 4) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(m >> 4) << 24);
}
// Instruction descriptor: dense, fp32 accumulate, A and B bf16, both K-major, M x N.
__host__ __device__ constexpr uint32_t instr_desc_bf16(int m, int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) |
           (static_cast<uint32_t>(m >> 4) << 24);
}

// ---- pacing of the units that stream the same W chunk ------------------------------------------
// Units that share a vocabulary chunk read the same W tiles; only while they stay within a few
// tiles of each other does each tile come from HBM once and from L2 for the rest.  Every unit's
// producer publishes (epoch, wave, tile) when it starts a tile and, before starting tile t, waits
// until no unit of its group is further back than t - lead.  The wait is advisory: it gives up
// after a short time, and for good after a few expiries, so stale or foreign workspace contents
// can only cost time.
constexpr unsigned long long kPaceLimitNs = 40000ull;       // per tile
constexpr int kPaceMaxExpiries = 4;
__device__ __forceinline__ unsigned long long pace_key(uint32_t epoch, int wave, int tile) {
    return ((unsigned long long)(epoch & 0xffffu) << 48) | ((unsigned long long)(wave & 0xffffff) << 24) |
           (unsigned long long)(tile & 0xffffff);
}
__device__ __forceinline__ unsigned long long ld_progress(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_progress(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

struct SharedLayout {
    uint64_t full[kMaxStages];   // TMA -> MMA: stage holds data (pair: only the leader's is used)
    uint64_t empty[kMaxStages];  // MMA -> TMA: stage may be overwritten
    uint64_t acc_full[2];        // MMA -> epilogue: accumulator complete
    uint64_t acc_empty[2];       // epilogue -> MMA: accumulator drained (pair: only the leader's is used)
    uint64_t mode;               // epilogue warps -> MMA issuer and epilogue: magnitude counts published
    uint64_t mag_counts[2 * kEpilogueWarps];   // per epilogue warp of the unit: see pack_magnitude_counts
    ScorePlan plan2;             // second pass: the plan derived from the number of marked rows
    // 8-bit operands: the scales of a vocabulary tile's 256 columns, staged by the epilogue warps (32 columns
    // each) when they start the tile.  Four buffers: the warps of a CTA are never more than three tiles apart
    // (a warp starts tile t + 2 only after every warp has drained tile t - 1 from tensor memory).
    uint64_t wscale_full[kScaleBufs];
    alignas(16) float wscale[kScaleBufs][kBlockN];
    uint32_t tmem_base;
    uint32_t abort_flag;
};

// Magnitude class of a thread's largest |logit| in the run's first tile: the e with max(2 |logit|, 1) in
// [2^(e-1), 2^e), 1..10; 11 from 1024 on (and for NaN).  The factor two is margin: the maximum over the
// whole vocabulary lies above the maximum over one tile.
__device__ __forceinline__ int magnitude_class(float absmax) {
    const float a = fmaxf(2.0f * absmax, 1.0f);
    if (!(a < 1024.0f)) return 11;
    return ((__float_as_int(a) >> 23) & 0xff) - 126;         // a = m * 2^e with m in [0.5, 1)
}
// One word per warp: for t = 1..10, six bits holding how many of the warp's lanes have a class above t.
__device__ __forceinline__ uint64_t pack_magnitude_counts(int cls) {
    uint64_t w = 0;
#pragma unroll
    for (int t = 1; t <= 10; ++t)
        w |= (uint64_t)__popc(__ballot_sync(0xffffffffu, cls > t)) << (6 * (t - 1));
    return w;
}
// The class the unit's chunks are sized for: the smallest one that all but 1/32 of the unit's (row, column
// half) samples stay within.  A few rows with far larger logits than the rest (which the merge will send to
// the second pass anyway) therefore do not shorten the chunks of their whole tile.
template <int kCg>
__device__ __forceinline__ int read_magnitude_class(const SharedLayout* sh) {
    const volatile uint64_t* p = sh->mag_counts;
    uint32_t above[10];
#pragma unroll
    for (int t = 0; t < 10; ++t) above[t] = 0;
#pragma unroll
    for (int i = 0; i < kEpilogueWarps * kCg; ++i) {
        const uint64_t w = p[i];
#pragma unroll
        for (int t = 0; t < 10; ++t) above[t] += (uint32_t)(w >> (6 * t)) & 63u;
    }
    constexpr uint32_t kBudget = 8 * kCg;                    // of 256 * kCg samples
    int cls = 11;
#pragma unroll
    for (int t = 9; t >= 0; --t) cls = (above[t] <= kBudget) ? t + 1 : cls;
    return cls;
}

// Chunk length (in k-blocks) for logits of magnitude class `cls`, i.e. below 2^cls.
// One accumulation (one MMA instruction along K) truncates the fp32 accumulator toward zero by at most
// one spacing of its magnitude.  The chunk gets as many accumulations as keep (count x spacing below 2^cls)
// under 1e-3, half of the 2e-3 tolerance on a token log-probability.  That product is a worst case: the
// loss per accumulation averages half a spacing, and of the partial sum's magnitude, not the final one's;
// measured, the bias is about a quarter of it (-5e-3 at |logit| = 700, d = 5120, one chunk: bound 2e-2).
// The chunk is never shorter than `base`.  `*bound` receives the magnitude up to which that holds (2^cls),
// the base chunk's own bound when the base chunk is kept (the second pass has shorter chunks for rows beyond it).
__device__ __forceinline__ int adaptive_chunk_kblocks(int cls, int base, int k_blocks, float* bound) {
    *bound = kBaseChunkBound;
    if (cls > 10) return base;
    const float n_acc = ldexpf(1.0e-3f, 24 - cls);           // spacing of [2^(cls-1), 2^cls) is 2^(cls-24)
    int kb = (int)fminf(n_acc * 0.25f, 1.0e6f);              // four accumulations per k-block
    if (kb <= base) return base;
    *bound = ldexpf(1.0f, cls);
    if (kb >= k_blocks) return k_blocks;
    const int chunks = (k_blocks + kb - 1) / kb;             // equal chunks
    return (k_blocks + chunks - 1) / chunks;
}

// What links the two passes of an adaptive plan (see FixCtl): the first pass resets the count of marked
// rows; the second reads it, the list of marked rows and, for 8-bit operands, their gathered scales.
struct PassArgs {
    FixCtl* ctl;
    const int32_t* list;
    const float* scale_compact;
    int32_t cap_rows;
};

// kFp8: operands are E4M3 codes (128 elements per 128-byte k-block, K = 32 per MMA) and the epilogue
// multiplies every accumulator by hidden_scale[row] * w_scale[column] before anything else.
// kSecond: the second pass.  It returns at once when no row was marked; otherwise it scores, with the base
// chunks, either the marked rows gathered in the compact buffer (map_compact, plan derived from their
// number) or, when they outnumber that buffer, every row in place (map_hidden, the first pass's plan).
template <int kCg, bool kFp8, bool kSecond>
__device__ __forceinline__ void score_tiles_body(const CUtensorMap& map_hidden, const CUtensorMap& map_compact,
                                                 const CUtensorMap& map_w, const ScorePlan& plan_in,
                                                 const int32_t* __restrict__ token_ids,
                                                 float* __restrict__ workspace, uint32_t* __restrict__ status,
                                                 const float* __restrict__ hidden_scale,
                                                 const float* __restrict__ w_scale, const PassArgs pass) {
    constexpr int kElemsK = kFp8 ? 2 * kBlockK : kBlockK;    // elements in a 128-byte k-block
    using S = Shape<kCg>;
    constexpr int kStages = S::kStages;
    constexpr uint32_t kStageBytes = S::kStageBytes;
    extern __shared__ uint8_t smem_raw[];
    // 128-byte-swizzled TMA destinations and UMMA operands must sit on 1024-byte boundaries.
    // (The dynamic shared-memory window starts at the same offset in both CTAs of a pair, so
    // the layout below is identical in the two, as the pair's MMA descriptors require.)
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
    uint8_t* tiles = smem_raw + pad;
    SharedLayout* sh = reinterpret_cast<SharedLayout*>(tiles + (size_t)kStages * kStageBytes);
    const uint32_t tiles_addr = smem_u32(tiles);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int cta = blockIdx.x;
    const uint32_t rank = (kCg == 2) ? cluster_ctarank() : 0u;   // 0: leader of the pair
    const int unit = cta / kCg;
    AbortFlags ab;
    ab.own = &sh->abort_flag;
    ab.peer = (kCg == 2) ? mapa_shared(smem_u32(&sh->abort_flag), rank ^ 1u) : 0u;

    bool compact = false;                                    // second pass: gathered rows rather than all rows
    if (kSecond) {
        // the next kernel of the stream may set itself up from now on (it waits for this one's end itself)
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        // the count is the merge kernel's: wait for it before anything else, and leave when there is no work
        asm volatile("griddepcontrol.wait;" ::: "memory");
        const uint32_t marked = *reinterpret_cast<const volatile uint32_t*>(&pass.ctl->count);
        if (marked == 0u) return;                            // every CTA of the grid takes the same decision
        compact = marked <= (uint32_t)pass.cap_rows;
        if (threadIdx.x == 0) {
            const float mag = __uint_as_float(*reinterpret_cast<const volatile uint32_t*>(&pass.ctl->max_mag_bits));
            sh->plan2 = compact ? make_compact_plan(plan_in, (int64_t)marked, mag) : make_inplace_fix_plan(plan_in, mag);
        }
    }
    const ScorePlan& plan = kSecond ? sh->plan2 : plan_in;   // (plan2 is read after the barrier below)

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&sh->full[s]), 1);
            mbar_init(smem_u32(&sh->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&sh->acc_full[b]), 1);
            mbar_init(smem_u32(&sh->acc_empty[b]), kEpilogueWarps * kCg);   // one arrival per epilogue warp
        }
        mbar_init(smem_u32(&sh->mode), kEpilogueWarps * kCg);
        for (int b = 0; b < kScaleBufs; ++b) mbar_init(smem_u32(&sh->wscale_full[b]), kEpilogueWarps);
        sh->abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        // in the pair kernel warp 1 of BOTH CTAs executes the allocation, with the same arguments
        if (kCg == 1) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(&sh->tmem_base)), "r"(kTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(&sh->tmem_base)), "r"(kTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    __syncwarp();
    if (kCg == 2) cluster_sync_all();     // the peer's barriers are initialised before anything reaches them
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&sh->tmem_base);
    if (!kSecond) {
        // the kernel may have been launched while its predecessor in the stream still ran: wait for it here
        asm volatile("griddepcontrol.wait;" ::: "memory");
        // (No early launch of the dependents here: set up while this kernel still runs, the small kernels behind
        // it made a step about 4 us slower than when they are launched at its end.)
        if (pass.ctl != nullptr && blockIdx.x == 0 && threadIdx.x == 0) {
            pass.ctl->count = 0u;
            pass.ctl->max_mag_bits = 0u;
        }
    }

    // Registers move from the control warpgroup (which needs few) to the two epilogue warpgroups
    // (128 fp32 partial logits per thread).  Each setmaxnreg sits at the
    // top of the code it governs so that the register allocator sees which budget applies where.
    if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kControlRegs));
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        // Lane 0 waits for free stages and issues the loads; the whole warp takes part in the pacing
        // poll before each vocabulary tile (one progress word per lane, one trip to L2).
        // pair: every load of either CTA is counted on the leader's barrier of the stage
        const uint32_t full0 = (kCg == 2) ? mapa_shared(smem_u32(&sh->full[0]), 0u) : smem_u32(&sh->full[0]);
        unsigned long long* progress = reinterpret_cast<unsigned long long*>(
            reinterpret_cast<char*>(workspace) + plan_slot_bytes(plan));
        bool pace = plan.lead_tiles > 0 && rank == 0;
        int expiries = 0;
        uint32_t stage = 0, phase = 0;           // meaningful in lane 0 only
        uint32_t issued = 0;
        bool ok = true;                          // warp-uniform
        const CUtensorMap* map_rows = (kSecond && compact) ? &map_compact : &map_hidden;
        for (int w = 0; w < plan.waves && ok; ++w) {
            int st, nb, ne;
            if (!plan_unit(plan, w, unit, &st, &nb, &ne)) continue;
            const int row0 = (st * kCg + (int)rank) * kBlockM;
            // the units of this wave that stream the same vocabulary chunk
            const int gm_w = w < plan.full_waves ? plan.group_m : plan.rem_m;
            const int group0 = (unit / gm_w) * gm_w;
            // pace points: the start of a vocabulary tile and, where the plan asks for more than one per tile,
            // evenly spaced k-blocks inside it
            const int points = plan.pace_points > 1 ? plan.pace_points : 1;
            const int seg = (plan.k_blocks + points - 1) / points;
            for (int n = nb; n < ne && ok; ++n) {
                const int wrow0 = n * kBlockN + (int)rank * S::kBRows;
                for (int kb0 = 0, sidx = 0; kb0 < plan.k_blocks && ok; kb0 += seg, ++sidx) {
                    if (pace && gm_w > 1) {
                        const int t = (n - nb) * points + sidx;
                        if (lane == 0 && SPECS_IN_BOUNDS(unit, plan.units, status))
                            st_progress(progress + unit, pace_key(plan.epoch, w, t));
                        if (t >= plan.lead_tiles) {
                            const unsigned long long need = pace_key(plan.epoch, w, t - plan.lead_tiles);
                            const unsigned long long t0 = global_timer_ns();
                            for (;;) {
                                unsigned long long lo = ~0ull;
                                for (int i = lane; i < gm_w; i += 32) {
                                    const unsigned long long v = ld_progress(progress + group0 + i);
                                    // a word of another launch counts as "not started"
                                    const unsigned long long cur = (v >> 48) == (plan.epoch & 0xffffu) ? v : 0ull;
                                    lo = cur < lo ? cur : lo;
                                }
#pragma unroll
                                for (int o = 16; o > 0; o >>= 1) {
                                    const unsigned long long other = __shfl_xor_sync(0xffffffffu, lo, o);
                                    lo = other < lo ? other : lo;
                                }
                                const bool expired =
                                    __shfl_sync(0xffffffffu, global_timer_ns() - t0 > kPaceLimitNs, 0);
                                if (lo >= need) { expiries = 0; break; }
                                if (expired) {
                                    if (++expiries >= kPaceMaxExpiries) pace = false;
                                    break;
                                }
                            }
                        }
                    }
                    if (lane == 0) {
                        const int kb1 = min(kb0 + seg, plan.k_blocks);
                        for (int kb = kb0; kb < kb1; ++kb) {
                            if (!mbar_wait(smem_u32(&sh->empty[stage]), phase ^ 1u, ab, kWaitLimitNs, true)) {
                                ok = false;
                                break;
                            }
                            const uint32_t a_dst = tiles_addr + stage * kStageBytes;
                            const uint32_t bar = full0 + stage * 8u;
                            if (kCg == 1) {
                                mbar_arrive_expect_tx(bar, kStageBytes);
                                tma_load_2d(a_dst, map_rows, kb * kElemsK, row0, bar);
                                tma_load_2d(a_dst + kABytes, &map_w, kb * kElemsK, wrow0, bar);
                            } else {
                                // the leader expects both CTAs' bytes; the peer's may be counted first
                                if (rank == 0) mbar_arrive_expect_tx(smem_u32(&sh->full[stage]), 2u * kStageBytes);
                                tma_load_2d_pair(a_dst, map_rows, kb * kElemsK, row0, bar);
                                tma_load_2d_pair(a_dst + kABytes, &map_w, kb * kElemsK, wrow0, bar);
                            }
                            ++issued;
                            if (++stage == kStages) { stage = 0; phase ^= 1u; }
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                }
            }
        }
        if (lane == 0) {
            if (ok) {
                // Tail: wait until the MMAs that read the last stages have retired, so that no
                // barrier arrival (in the pair kernel: from the other CTA) is still on its way
                // to this CTA's shared memory when the CTA exits.
                for (int i = 0; i < kStages; ++i) {
                    if (!mbar_wait(smem_u32(&sh->empty[stage]), phase ^ 1u, ab, kWaitLimitNs, true)) break;
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
            } else if (kCg == 1 || rank == 0) {
                // Drain: the last min(issued, kStages) loads may still be landing in shared memory.
                const uint32_t pending = issued < (uint32_t)kStages ? issued : (uint32_t)kStages;
                uint32_t s = stage, ph = phase;
                for (uint32_t i = 0; i < pending; ++i) {
                    if (s == 0) { s = kStages - 1; ph ^= 1u; } else { --s; }
                    mbar_wait(smem_u32(&sh->full[s]), ph, ab, kDrainLimitNs, false);
                }
            } else {
                // The peer cannot poll the leader's barriers: give its own loads in flight a fixed time.
                const unsigned long long t0 = global_timer_ns();
                while (global_timer_ns() - t0 < kDrainLimitNs) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (pair: the leader's)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = kFp8 ? instr_desc_e4m3(kBlockM * kCg, kBlockN)
                                            : instr_desc_bf16(kBlockM * kCg, kBlockN);
            uint32_t stage = 0, phase = 0;
            uint32_t chunk_count = 0;                        // accumulator hand-overs so far
            uint32_t mode_runs = 0;                          // completed phases of the "mode" barrier
            bool ok = true;
            for (int w = 0; w < plan.waves && ok; ++w) {
                int st, nb, ne;
                if (!plan_unit(plan, w, unit, &st, &nb, &ne)) continue;
                const bool adapt_run = plan.adaptive && (ne - nb) >= 3;
                int ck = plan.chunk_kblocks;                 // k-blocks per chunk of the current tile
                for (int n = nb; n < ne && ok; ++n) {
                    if (adapt_run && n == nb + 2) {
                        if (!mbar_wait(smem_u32(&sh->mode), mode_runs & 1u, ab, kWaitLimitNs, true, true)) {
                            ok = false;
                            break;
                        }
                        ++mode_runs;
                        float bound;
                        ck = adaptive_chunk_kblocks(read_magnitude_class<kCg>(sh), plan.chunk_kblocks, plan.k_blocks,
                                                    &bound);
                    }
                    for (int kb0 = 0; kb0 < plan.k_blocks && ok; kb0 += ck, ++chunk_count) {
                        const uint32_t buf = chunk_count & 1u;
                        const uint32_t use_phase = (chunk_count >> 1) & 1u;
                        if (!mbar_wait(smem_u32(&sh->acc_empty[buf]), use_phase ^ 1u, ab, kWaitLimitNs, true)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint32_t d_tmem = tmem_base + buf * kBlockN;
                        const int kb1 = min(kb0 + ck, plan.k_blocks);
                        for (int kb = kb0; kb < kb1; ++kb) {
                            if (!mbar_wait(smem_u32(&sh->full[stage]), phase, ab, kWaitLimitNs, true)) {
                                ok = false;
                                break;
                            }
                            tc_fence_after();
                            const uint32_t a_addr = tiles_addr + stage * kStageBytes;
                            const uint64_t a_desc = smem_desc_k_major_sw128(a_addr);
                            const uint64_t b_desc = smem_desc_k_major_sw128(a_addr + kABytes);
#pragma unroll
                            for (int k = 0; k < kBlockK / kUmmaK; ++k) {
                                // advancing 32 bytes (16 bf16 or 32 E4M3) along K inside the swizzled row: +2
                                // in the 16-byte units of the descriptor's start-address field
                                const uint32_t accumulate = (kb != kb0 || k != 0) ? 1u : 0u;
                                const uint64_t a_k = a_desc + (uint64_t)(2 * k), b_k = b_desc + (uint64_t)(2 * k);
                                if (kFp8) {
                                    if (kCg == 1) tc_mma_f8(d_tmem, a_k, b_k, idesc, accumulate);
                                    else          tc_mma_f8_pair(d_tmem, a_k, b_k, idesc, accumulate);
                                } else {
                                    if (kCg == 1) tc_mma_bf16(d_tmem, a_k, b_k, idesc, accumulate);
                                    else          tc_mma_bf16_pair(d_tmem, a_k, b_k, idesc, accumulate);
                                }
                            }
                            // frees the stage (in both CTAs of a pair) once these MMAs retire
                            if (kCg == 1) tc_commit(smem_u32(&sh->empty[stage]));
                            else          tc_commit_pair(smem_u32(&sh->empty[stage]));
                            if (++stage == kStages) { stage = 0; phase ^= 1u; }
                        }
                        if (ok) {                            // chunk ready for the epilogue(s)
                            if (kCg == 1) tc_commit(smem_u32(&sh->acc_full[buf]));
                            else          tc_commit_pair(smem_u32(&sh->acc_full[buf]));
                        }
                    }
                }
            }
        }
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kEpilogueRegs));
        // ------------------------------------------------------------------ epilogue (warps 4..11)
        const int quarter = warp & 3;                        // TMEM lanes 32*quarter .. +31 belong to this warp
        const int half = (warp - 4) >> 2;                    // which 128 columns of the tile
        const int row_in_tile = quarter * 32 + lane;
        const uint32_t lane_field = static_cast<uint32_t>(quarter * 32) << 16;
        // "accumulator drained" is counted on the leader's barrier
        const uint32_t acc_empty0 = (kCg == 2) ? mapa_shared(smem_u32(&sh->acc_empty[0]), 0u) : 0u;
        uint32_t chunk_count = 0;
        uint32_t mode_runs = 0;
        uint32_t tile_count = 0;                             // vocabulary tiles so far (8-bit operands: scale buffers)
        bool ok = true;
        for (int w = 0; w < plan.waves && ok; ++w) {
            int st, nb, ne;
            if (!plan_unit(plan, w, unit, &st, &nb, &ne)) continue;
            const bool adapt_run = plan.adaptive && (ne - nb) >= 3;
            int ck = plan.chunk_kblocks;                     // k-blocks per chunk of the current tile
            // magnitude up to which the chunks in use keep the tolerance: the base chunk's own bound until (and
            // unless) the run lengthens its chunks; no claim, and no marking, outside adaptive plans
            float assumed = (!kSecond && plan.adaptive) ? kBaseChunkBound : INFINITY;
            const int64_t row = (int64_t)(st * kCg + (int)rank) * kBlockM + row_in_tile;
            // the row of the caller's arrays behind this one: itself, or the marked row gathered here
            int64_t src = row;
            if (kSecond && compact && row < plan.rows && SPECS_IN_BOUNDS(row, pass.cap_rows, status))
                src = (int64_t)pass.list[row];
            // ids are indices into the whole vocabulary; this W holds rows id_offset .. id_offset + V - 1
            const int32_t id = (row < plan.rows && SPECS_IN_BOUNDS(src, plan_in.rows, status))
                                   ? token_ids[src] - plan.id_offset : -1;
            float row_scale = 0.0f;
            if (kFp8 && row < plan.rows) row_scale = (kSecond && compact) ? pass.scale_compact[row] : hidden_scale[src];
            // what turns the values of `acc` below into base-2 exponents: log2(e), times the row's scale for 8-bit
            // operands (whose column scales are applied first, the row's only here, in the same multiply-add)
            const float to_exp2 = kFp8 ? row_scale * kLog2e : kLog2e;
            // state in base-2 units: run_max = max(z) * log2(e), run_sum = sum 2^(z*log2e - run_max)
            float run_max = -INFINITY, run_sum = 0.0f, picked = -INFINITY;
            for (int n = nb; n < ne && ok; ++n) {
                if (adapt_run && n == nb + 2) {
                    if (!__all_sync(0xffffffffu,
                                    mbar_wait(smem_u32(&sh->mode), mode_runs & 1u, ab, kWaitLimitNs, true, true))) {
                        ok = false;
                        break;
                    }
                    ++mode_runs;
                    ck = adaptive_chunk_kblocks(read_magnitude_class<kCg>(sh), plan.chunk_kblocks, plan.k_blocks,
                                                &assumed);
                }
                const uint32_t sbuf = tile_count % kScaleBufs;
                if (kFp8) {
                    // this warp's 32 of the tile's 256 column scales into shared memory (hidden behind the MMAs)
                    const int c = (warp - 4) * 32 + lane, col = n * kBlockN + c;
                    sh->wscale[sbuf][c] = col < plan.V ? __ldg(w_scale + col) : 0.0f;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&sh->wscale_full[sbuf]));
                }
                float acc[kHalfN];                           // this thread's 128 logits of the tile
                for (int kb0 = 0; kb0 < plan.k_blocks; kb0 += ck, ++chunk_count) {
                    const uint32_t buf = chunk_count & 1u;
                    const uint32_t use_phase = (chunk_count >> 1) & 1u;
                    // the whole warp takes the same decision: __syncwarp below needs every lane
                    if (!__all_sync(0xffffffffu,
                                    mbar_wait(smem_u32(&sh->acc_full[buf]), use_phase, ab, kWaitLimitNs, true))) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t taddr = tmem_base + lane_field + buf * kBlockN + half * kHalfN;
                    if (kb0 == 0) {
#pragma unroll
                        for (int g = 0; g < kHalfN / 32; ++g) {
                            float v[32];
                            tmem_ld_32cols(taddr + g * 32, v);
#pragma unroll
                            for (int j = 0; j < 32; ++j) acc[g * 32 + j] = v[j];
                        }
                    } else {
                        // 16 columns at a time: with 128 running sums live, a 32-register landing area spills
#pragma unroll
                        for (int g = 0; g < kHalfN / 16; ++g) {
                            float v[16];
                            tmem_ld_16cols(taddr + g * 16, v);
#pragma unroll
                            for (int j = 0; j < 16; ++j) acc[g * 16 + j] += v[j];
                        }
                    }
                    // the warp's loads are complete: one arrival per warp lets the MMA issuer reuse the buffer
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        if (kCg == 1) mbar_arrive(smem_u32(&sh->acc_empty[buf]));
                        else          mbar_arrive_cluster(acc_empty0 + buf * 8u);
                    }
                }
                if (!ok) break;
                const int col_base = n * kBlockN + half * kHalfN;
                if (kFp8) {
                    // de-quantise: the sums are over codes; logit = sum * scale of the column * scale of the row.
                    // The column scales come from shared memory, four at a time and the same for every lane; the
                    // row's scale is folded into the exponent's multiply-add (to_exp2).
                    if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&sh->wscale_full[sbuf]),
                                                           (tile_count / kScaleBufs) & 1u, ab, kWaitLimitNs, true))) {
                        ok = false;
                        break;
                    }
                    const float4* ws4 = reinterpret_cast<const float4*>(&sh->wscale[sbuf][half * kHalfN]);
#pragma unroll
                    for (int q = 0; q < kHalfN / 4; ++q) {
                        const float4 sc = ws4[q];
                        acc[4 * q] *= sc.x; acc[4 * q + 1] *= sc.y; acc[4 * q + 2] *= sc.z; acc[4 * q + 3] *= sc.w;
                    }
                }
                ++tile_count;
                if (adapt_run && n == nb) {
                    // first tile of the run: publish how this warp's rows are spread over the magnitude classes
                    // to every CTA of the unit
                    float amax = 0.0f;
#pragma unroll
                    for (int j = 0; j < kHalfN; ++j)
                        amax = (col_base + j < plan.V) ? fmaxf(amax, fabsf(acc[j])) : amax;
                    if (kFp8) amax *= row_scale;
                    const uint64_t counts = pack_magnitude_counts(magnitude_class(amax));
                    if (lane == 0) {
                        const int slot = (int)rank * kEpilogueWarps + (warp - 4);
                        if (kCg == 1) {
                            *reinterpret_cast<volatile uint64_t*>(&sh->mag_counts[slot]) = counts;
                            mbar_arrive(smem_u32(&sh->mode));
                        } else {
#pragma unroll
                            for (uint32_t r = 0; r < 2; ++r) {
                                st_cluster_u64(mapa_shared(smem_u32(&sh->mag_counts[slot]), r), counts);
                                mbar_arrive_cluster(mapa_shared(smem_u32(&sh->mode), r));
                            }
                        }
                    }
                }
#pragma unroll
                for (int g = 0; g < kHalfN / 32; ++g) {
                    const int col0 = col_base + g * 32;
                    const int valid = plan.V - col0;         // columns of this group inside the vocabulary
                    if (valid > 0) {
                        float* v = acc + g * 32;
                        if (valid < 32) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] = (j < valid) ? v[j] : -INFINITY;
                        }
                        const uint32_t rel = static_cast<uint32_t>(id - col0);
                        if (rel < 32u) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) picked = (rel == (uint32_t)j) ? v[j] : picked;
                            if (kFp8) picked *= row_scale;
                        }
                        float cmax = v[0];
#pragma unroll
                        for (int j = 1; j < 32; ++j) cmax = fmaxf(cmax, v[j]);
                        const float new_max = fmaxf(run_max, cmax * to_exp2);
                        run_sum *= ex2_approx(run_max - new_max);  // 2^-inf = 0 on the first group
                        run_max = new_max;
                        float acc0 = 0.0f, acc1 = 0.0f;
#pragma unroll
                        for (int j = 0; j < 32; j += 2) {
                            acc0 += ex2_approx(fmaf(v[j], to_exp2, -new_max));
                            acc1 += ex2_approx(fmaf(v[j + 1], to_exp2, -new_max));
                        }
                        run_sum += acc0 + acc1;
                    }
                }
            }
            if (ok) {
                // A logit that matters -- this part's maximum (the terms of the sum that count lie next to it)
                // or the drafted id's -- beyond the magnitude the lengthened chunks were sized for: the row is
                // marked by the sign of its sum (which is positive otherwise) and re-scored in the second pass.
                const bool over = run_sum > 0.0f && (fabsf(run_max) > assumed * kLog2e ||
                                                     (picked != -INFINITY && fabsf(picked) > assumed));
                if (__any_sync(0xffffffffu, over) && lane == 0) atomicOr(status, SPECS_DEV_ACCUM_RANGE);
                const size_t at = ((size_t)w * plan.grid + cta) * kTripleFloats + half * 3 * kBlockM;
                float* slot = workspace + at;
                if (SPECS_IN_BOUNDS(at + 2 * kBlockM + row_in_tile, plan_slot_bytes(plan) / sizeof(float), status)) {
                    slot[row_in_tile] = run_max;
                    slot[kBlockM + row_in_tile] = over ? -run_sum : run_sum;
                    slot[2 * kBlockM + row_in_tile] = picked;
                }
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    __syncwarp();
    if (kCg == 2) cluster_sync_all();     // neither CTA frees TMEM or exits while the other still works
    if (threadIdx.x == 0 && sh->abort_flag != 0u) atomicOr(status, SPECS_DEV_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        if (kCg == 1)
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// The kernels: {one CTA, CTA pair} x {bf16, E4M3} x {first pass, second pass}, one body.
#define SPECS_SCORE_KERNEL(name, cluster_attr, kCg, kFp8, kSecond)                                                  \
    __global__ void cluster_attr __launch_bounds__(kThreads, 1)                                                     \
    name(const __grid_constant__ CUtensorMap map_hidden, const __grid_constant__ CUtensorMap map_compact,           \
         const __grid_constant__ CUtensorMap map_w, const ScorePlan plan, const int32_t* __restrict__ token_ids,    \
         float* __restrict__ workspace, uint32_t* __restrict__ status, const float* __restrict__ hidden_scale,      \
         const float* __restrict__ w_scale, const PassArgs pass) {                                                  \
        score_tiles_body<kCg, kFp8, kSecond>(map_hidden, map_compact, map_w, plan, token_ids, workspace, status,    \
                                             hidden_scale, w_scale, pass);                                          \
    }
#define SPECS_NO_CLUSTER
SPECS_SCORE_KERNEL(score_tiles_kernel, SPECS_NO_CLUSTER, 1, false, false)
SPECS_SCORE_KERNEL(score_tiles_pair_kernel, __cluster_dims__(2, 1, 1), 2, false, false)
SPECS_SCORE_KERNEL(score_tiles_fp8_kernel, SPECS_NO_CLUSTER, 1, true, false)
SPECS_SCORE_KERNEL(score_tiles_pair_fp8_kernel, __cluster_dims__(2, 1, 1), 2, true, false)
SPECS_SCORE_KERNEL(score_tiles_second_kernel, SPECS_NO_CLUSTER, 1, false, true)
SPECS_SCORE_KERNEL(score_tiles_pair_second_kernel, __cluster_dims__(2, 1, 1), 2, false, true)
SPECS_SCORE_KERNEL(score_tiles_fp8_second_kernel, SPECS_NO_CLUSTER, 1, true, true)
SPECS_SCORE_KERNEL(score_tiles_pair_fp8_second_kernel, __cluster_dims__(2, 1, 1), 2, true, true)
#undef SPECS_NO_CLUSTER
#undef SPECS_SCORE_KERNEL

using ScoreKernel = void (*)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const ScorePlan, const int32_t*,
                             float*, uint32_t*, const float*, const float*, const PassArgs);
ScoreKernel score_kernel_for(bool pair, bool fp8, bool second) {
    if (second) {
        if (fp8) return pair ? score_tiles_pair_fp8_second_kernel : score_tiles_fp8_second_kernel;
        return pair ? score_tiles_pair_second_kernel : score_tiles_second_kernel;
    }
    if (fp8) return pair ? score_tiles_pair_fp8_kernel : score_tiles_fp8_kernel;
    return pair ? score_tiles_pair_kernel : score_tiles_kernel;
}

// Row-wise quantisation to E4M3: one warp per row.  scale = absmax / 448; code = nearest E4M3 of
// x * (448 / absmax), all in float32 with round-to-nearest operations (the codes are integers decided
// by this arithmetic, so it is spelled out); a row of zeros gets scale 1 and codes 0.
__global__ void quantize_rows_kernel(const __nv_bfloat16* __restrict__ x, int64_t n, int32_t d,
                                     uint8_t* __restrict__ codes, float* __restrict__ scale) {
    const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (row >= n) return;
    const __nv_bfloat16* xr = x + (size_t)row * d;
    float amax = 0.0f;
    for (int k = lane; k < d; k += 32) amax = fmaxf(amax, fabsf(__bfloat162float(xr[k])));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    const bool live = amax > 0.0f;
    const float inv = live ? __fdiv_rn(448.0f, amax) : 1.0f;
    if (lane == 0) scale[row] = live ? __fdiv_rn(amax, 448.0f) : 1.0f;
    uint8_t* cr = codes + (size_t)row * d;
    for (int k = 2 * lane; k < d; k += 64) {                 // d is even: two codes per conversion
        const float y0 = __fmul_rn(__bfloat162float(xr[k]), inv), y1 = __fmul_rn(__bfloat162float(xr[k + 1]), inv);
        uint16_t pair;
        // the first source operand lands in the upper byte, the second in the lower
        asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(pair) : "f"(y1), "f"(y0));
        *reinterpret_cast<uint16_t*>(cr + k) = pair;
    }
}

// One CTA waits, with the kernel's own bounded wait, on a barrier that nothing ever completes:
// the wait must give up after limit_ns, raise the abort flag and report SPECS_DEV_TIMEOUT, and
// the kernel must return.  This is the expiry path of every wait in the scoring kernel,
// exercised without a stuck scoring kernel.
__global__ void wait_expiry_probe_kernel(unsigned long long limit_ns, uint32_t* __restrict__ status) {
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    AbortFlags ab;
    ab.own = &abort_flag;
    ab.peer = 0u;
    const bool completed = mbar_wait(smem_u32(&bar), 0u, ab, limit_ns, true);
    __syncthreads();
    if (threadIdx.x == 0 && (!completed || abort_flag != 0u)) atomicOr(status, SPECS_DEV_TIMEOUT);
}

// Tensor map of a row-major [outer, inner] matrix with 128-byte-swizzled boxes; maps the context has
// encoded before are found again by what they describe (the weight's map is the same at every call).
int encode_rows_2d(specs_ctx* ctx, CUtensorMap* map, const void* base, uint64_t inner, uint64_t outer,
                   uint32_t box_inner, uint32_t box_outer, int elem_bytes) {
    for (const CachedMap& c : ctx->maps)
        if (c.base == base && c.inner == inner && c.outer == outer && c.box_inner == box_inner &&
            c.box_outer == box_outer && c.elem_bytes == elem_bytes) {
            *map = c.map;
            return SPECS_OK;
        }
    const cuuint64_t dims[2] = {inner, outer};
    const cuuint64_t strides[1] = {inner * (uint64_t)elem_bytes};   // bytes between consecutive rows
    const cuuint32_t box[2] = {box_inner, box_outer};
    const cuuint32_t elem_strides[2] = {1, 1};
    const CUresult r = ctx->encode_tiled(map, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                                                              : CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims,
                                         strides, box, elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return SPECS_ERR_CUDA;
    const CachedMap entry = {base, inner, outer, box_inner, box_outer, elem_bytes, *map};
    if (ctx->maps.size() < kMapCacheSize) {
        ctx->maps.push_back(entry);
    } else {
        ctx->maps[ctx->maps_next] = entry;
        ctx->maps_next = (ctx->maps_next + 1) % kMapCacheSize;
    }
    return SPECS_OK;
}

}  // namespace

int launch_quantize_rows(const void* x_bf16, int64_t n, int32_t d, uint8_t* codes, float* scale, cudaStream_t stream) {
    if (n == 0) return SPECS_OK;
    const int threads = 256;                                 // eight rows per block
    quantize_rows_kernel<<<(unsigned)((n + 7) / 8), threads, 0, stream>>>(static_cast<const __nv_bfloat16*>(x_bf16), n,
                                                                        d, codes, scale);
    return cuda_status(cudaGetLastError());
}

int launch_wait_expiry_probe(specs_ctx* ctx, unsigned long long limit_ns, cudaStream_t stream) {
    wait_expiry_probe_kernel<<<1, 64, 0, stream>>>(limit_ns, ctx->d_status);
    return cuda_status(cudaGetLastError());
}

int query_pair_units(int device, int num_sms) {
    // Per device, once: opt the kernels in to their dynamic shared memory (a per-device function
    // attribute) and ask how many CTA pairs the device keeps resident at once.
    static std::map<int, int> cached;                        // device -> resident pairs
    static std::mutex guard;
    std::lock_guard<std::mutex> lock(guard);
    const auto hit = cached.find(device);
    if (hit != cached.end()) return hit->second;
    int units = 0;
    bool ok1 = true, ok2 = true;
    for (int fp8 = 0; fp8 < 2; ++fp8)
        for (int second = 0; second < 2; ++second) {
            ok1 = ok1 && cudaFuncSetAttribute(score_kernel_for(false, fp8, second),
                                              cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)Shape<1>::kSmemBytes) == cudaSuccess;
            ok2 = ok2 && cudaFuncSetAttribute(score_kernel_for(true, fp8, second),
                                              cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)Shape<2>::kSmemBytes) == cudaSuccess;
        }
    if (ok2) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(num_sms & ~1), 1, 1);
        cfg.blockDim = dim3(kThreads, 1, 1);
        cfg.dynamicSmemBytes = Shape<2>::kSmemBytes;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        int clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&clusters, score_tiles_pair_kernel, &cfg) == cudaSuccess && clusters > 0)
            units = clusters < num_sms / 2 ? clusters : num_sms / 2;
    }
    cudaGetLastError();                                      // a failed query is not an error of the caller
    if (!ok1) return 0;                                      // try again on the next call
    cached[device] = units;
    return units;
}

namespace {

// One launch of the scoring kernel: the first pass over all rows, or the second over the marked ones.
int launch_score_pass(specs_ctx* ctx, const ScorePlan& plan_in, bool second, const void* hidden, const void* w_vocab,
                      const int32_t* token_ids, void* workspace, cudaStream_t stream, int32_t id_offset,
                      const float* hidden_scale, const float* w_scale) {
    static_assert(Shape<1>::kSmemBytes <= 227 * 1024 && Shape<2>::kSmemBytes <= 227 * 1024, "shared memory budget");
    static_assert(Shape<1>::kStages <= kMaxStages && Shape<2>::kStages <= kMaxStages, "barrier arrays");
    static_assert(sizeof(SharedLayout) <= kControlBytes, "control block");
    const bool pair = plan_in.cta_group == 2;
    if (pair && (plan_in.units > ctx->pair_units || (plan_in.grid & 1))) return SPECS_ERR_CUDA;
    if (second && !plan_in.adaptive) return SPECS_OK;        // only adaptive plans mark rows
    static std::atomic<uint32_t> launch_counter{0};
    ScorePlan plan = plan_in;
    plan.epoch = (launch_counter.fetch_add(1) % 0xfffeu) + 1u;  // never 0
    plan.lead_tiles = ctx->lead_tiles;
    {
        // Pace points per vocabulary tile: what the units of a wave keep live in L2 is the wave's hidden-state tiles
        // plus, per vocabulary chunk, the W bytes between the slowest and the fastest unit of the chunk (up to two
        // pace intervals).  One point per tile unless that exceeds about 50 MB (d = 5120: 31 + 31 MB; measured
        // 1.55 x the algorithmic HBM reads), then two or more.
        const double tile_w = (double)kBlockN * plan.d * plan.elem_bytes;
        const int gm = plan.full_waves > 0 ? plan.group_m : plan.rem_m;
        const int sp = plan.full_waves > 0 ? plan.split_full : plan.split_rem;
        const double hidden_live = (double)gm * kBlockM * plan.cta_group * plan.d * plan.elem_bytes;
        int points = 1;
        while (points < 4 && hidden_live + 2.0 * sp * tile_w / points > 50.0e6) ++points;
        plan.pace_points = points;
    }
    plan.id_offset = id_offset;
    query_pair_units(ctx->device, ctx->num_sms);             // shared-memory opt-in for this device
    const bool fp8 = plan.elem_bytes == 1;
    if (fp8 && (!hidden_scale || !w_scale)) return SPECS_ERR_NULL;
    const WsLayout lay = plan_layout(plan);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    const uint32_t box_k = (uint32_t)(kBlockK * 2 / plan.elem_bytes);       // 128 bytes of K
    CUtensorMap map_h, map_c, map_w;
    int st = encode_rows_2d(ctx, &map_h, hidden, (uint64_t)plan.d, (uint64_t)plan.rows, box_k, kBlockM,
                            plan.elem_bytes);
    if (st != SPECS_OK) return st;
    st = encode_rows_2d(ctx, &map_w, w_vocab, (uint64_t)plan.d, (uint64_t)plan.V, box_k,
                        pair ? Shape<2>::kBRows : Shape<1>::kBRows, plan.elem_bytes);
    if (st != SPECS_OK) return st;
    map_c = map_h;
    PassArgs pass = {nullptr, nullptr, nullptr, 0};
    if (plan.adaptive) {
        pass.ctl = reinterpret_cast<FixCtl*>(ws + lay.ctl);
        pass.list = reinterpret_cast<const int32_t*>(ws + lay.list);
        pass.scale_compact = reinterpret_cast<const float*>(ws + lay.compact_scale);
        pass.cap_rows = lay.cap_rows;
        if (second) {
            st = encode_rows_2d(ctx, &map_c, ws + lay.compact, (uint64_t)plan.d, (uint64_t)lay.cap_rows, box_k,
                                kBlockM, plan.elem_bytes);
            if (st != SPECS_OK) return st;
        }
    }
    float* slots = reinterpret_cast<float*>(second ? ws + lay.fix_slots : ws);

    TimedLaunch* tl = nullptr;
    if (ctx->timing) {
        if (ctx->timed_used == ctx->timed.size()) {
            TimedLaunch t;
            if (cudaEventCreate(&t.start) != cudaSuccess || cudaEventCreate(&t.stop) != cudaSuccess)
                return SPECS_ERR_CUDA;
            ctx->timed.push_back(t);
        }
        tl = &ctx->timed[ctx->timed_used++];
        tl->second_pass = second;
        cudaEventRecord(tl->start, stream);
    }
    // Programmatic stream serialisation: the launch is set up, and the CTAs do their prologue (barriers, tensor
    // memory), while the previous kernel of the stream still runs; griddepcontrol.wait in the kernel orders
    // everything that touches global memory after that kernel.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)plan.grid, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = pair ? Shape<2>::kSmemBytes : Shape<1>::kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t le = cudaLaunchKernelEx(&cfg, score_kernel_for(pair, fp8, second), map_h, map_c, map_w, plan,
                                              token_ids, slots, ctx->d_status, hidden_scale, w_scale, pass);
    if (le != cudaSuccess) return SPECS_ERR_CUDA;
    if (tl) cudaEventRecord(tl->stop, stream);
    return cuda_status(cudaGetLastError());
}

}  // namespace

int launch_score_tcgen05(specs_ctx* ctx, const ScorePlan& plan, const void* hidden, const void* w_vocab,
                         const int32_t* token_ids, void* workspace, cudaStream_t stream, int32_t id_offset,
                         const float* hidden_scale, const float* w_scale) {
    return launch_score_pass(ctx, plan, false, hidden, w_vocab, token_ids, workspace, stream, id_offset, hidden_scale,
                             w_scale);
}

int launch_score_second_pass(specs_ctx* ctx, const ScorePlan& plan, const void* hidden, const void* w_vocab,
                             const int32_t* token_ids, void* workspace, cudaStream_t stream, int32_t id_offset,
                             const float* hidden_scale, const float* w_scale) {
    return launch_score_pass(ctx, plan, true, hidden, w_vocab, token_ids, workspace, stream, id_offset, hidden_scale,
                             w_scale);
}

FixView fix_view(const ScorePlan& plan, const void* workspace) {
    FixView v = {nullptr, nullptr, nullptr, 0};
    if (!plan.adaptive || workspace == nullptr) return v;
    const WsLayout lay = plan_layout(plan);
    const uint8_t* ws = static_cast<const uint8_t*>(workspace);
    v.ctl = reinterpret_cast<const FixCtl*>(ws + lay.ctl);
    v.list = reinterpret_cast<const int32_t*>(ws + lay.list);
    v.slots = reinterpret_cast<const float*>(ws + lay.fix_slots);
    v.cap_rows = lay.cap_rows;
    return v;
}

}  // namespace specs
