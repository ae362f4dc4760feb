/*
 * specs.h -- C ABI of the B200 (sm_100a) block-scoring library for SPECS
 * (arxiv 2506.15733, "Faster Test-Time Scaling through Speculative Drafts and
 * Dynamic Switching").
 *
 * One beam step of the method scores n drafted candidate blocks per problem:
 * the target model's LM head gives log pi_target of every drafted token, the
 * per-block sums enter the score of Eq. (1) together with the generator's own
 * log-probabilities and the process-reward score, Algorithm 2 (SubSample)
 * samples one candidate with probability proportional to exp(S_i), and Step III
 * of Algorithm 1 decides whether the draft model may generate the next step.
 *
 * General rules for every call below
 *   - Pointers are DEVICE pointers unless their name starts with h_.  The
 *     caller owns every buffer; nothing passed in is retained after the work
 *     enqueued by the call has finished.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Calls validate their arguments on the host, enqueue work on the stream
 *     and return without synchronising, unless stated otherwise.
 *   - The return value is a specs_status.  On any value other than SPECS_OK
 *     nothing was launched and the outputs are untouched.
 *   - Conditions found on the device (a drafted id outside [0, V), a bounded
 *     wait inside a kernel that expired) never trap: they set bits in a device
 *     status word that specs_device_status() reads.
 *   - One context serves one stream at a time.
 */
#ifndef SPECS_H_
#define SPECS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct specs_ctx specs_ctx;

typedef enum specs_status {
    SPECS_OK = 0,
    SPECS_ERR_NULL = 1,            /* a required pointer is NULL */
    SPECS_ERR_SHAPE = 2,           /* rows < 0, d <= 0, d % 8 != 0, V <= 0, B < 0, P < 0, ... */
    SPECS_ERR_ALIGN = 3,           /* hidden / W_vocab / workspace not 16-byte aligned */
    SPECS_ERR_WORKSPACE = 4,       /* workspace smaller than specs_score_workspace_bytes() */
    SPECS_ERR_OFFSETS = 5,         /* h_ offsets not starting at 0 / decreasing / not ending at the total */
    SPECS_ERR_ARCH = 6,            /* device is not compute capability 10.x */
    SPECS_ERR_CUDA = 7,            /* a CUDA runtime or driver call failed */
    SPECS_ERR_DEVICE_TIMEOUT = 8,  /* device status: a bounded wait in a kernel expired */
    SPECS_ERR_TOKEN_RANGE = 9,     /* device status: some drafted id was outside [0, V) */
    SPECS_ERR_LIMIT = 10,          /* a size exceeds a documented maximum */
    SPECS_ERR_DEVICE_BOUNDS = 11   /* device status (checked build only): a kernel met an index outside its buffer */
} specs_status;

/* Bits of the device status word returned by specs_device_status(). */
#define SPECS_DEV_TIMEOUT      0x1u
#define SPECS_DEV_TOKEN_RANGE  0x2u
#define SPECS_DEV_ACCUM_RANGE  0x4u   /* informational: some rows were re-scored by the second pass, see
                                         specs_set_accum_chunk; does not change a return value */

#define SPECS_DEV_BOUNDS       0x8u   /* checked build only: an index check inside a kernel failed; the access
                                         was skipped (see specs_debug_build) */

/* 1 if the library was compiled with -DSPECS_DEBUG (the checked build), else 0.  The checked build
 * (libspecs_b200_debug.so; python -m paper_2506_15733_b200.build --debug) stands in for a memory
 * checker: every kernel tests the indices of its global-memory accesses against the extents the host
 * computed, skips an access that fails and raises SPECS_DEV_BOUNDS; it also contains the plain
 * CUDA-core scoring engine SPECS_ENGINE_SIMT, a second GPU implementation for bisecting the
 * tensor-core path.  Neither is in the default build. */
int specs_debug_build(void);

/* Scoring engines (see specs_set_engine). */
#define SPECS_ENGINE_TCGEN05      0   /* tensor-core path: TMA + tcgen05.mma + TMEM, fused epilogue (default);
                                        the planner picks the tile shape (one CTA or a CTA pair per tile) */
#define SPECS_ENGINE_SIMT         1   /* plain CUDA-core kernel; a bring-up and bisecting aid in the checked build only
                                        (specs_set_engine returns SPECS_ERR_SHAPE for it otherwise) */
#define SPECS_ENGINE_TCGEN05_1CTA 2   /* tensor-core path, forced to 128-row tiles run by single CTAs */
#define SPECS_ENGINE_TCGEN05_2CTA 3   /* tensor-core path, forced to 256-row tiles run by CTA pairs
                                        (tcgen05.mma.cta_group::2; each CTA stages half of the W tile) */

/* Human-readable name of a status value (static string, never NULL). */
const char* specs_status_string(int status);

/* Create / destroy a context on CUDA device `device`.  Creation allocates a few
 * bytes of device memory (the status word) and looks up the driver's tensor-map
 * encoder; it fails with SPECS_ERR_ARCH on anything but sm_100-class devices. */
int specs_create(specs_ctx** out, int device);
int specs_destroy(specs_ctx* ctx);

/* Select the scoring engine for later specs_score_blocks calls on this context
 * (SPECS_ERR_SHAPE for an unknown value; SPECS_ERR_CUDA if CTA pairs were asked
 * for and the device cannot launch them). */
int specs_set_engine(specs_ctx* ctx, int engine);

/* How the tensor-core kernel cuts the reduction over d into accumulation chunks.
 * The tensor core adds every K = 16 group of products into its fp32 accumulator
 * with truncation, which biases long reductions of large logits (about -5e-3 at
 * |logit| = 700, d = 5120).  The kernel therefore restarts the accumulator every
 * chunk and sums the chunks in registers with round-to-nearest, which divides the
 * bias by the number of chunks; every restart costs a read of the accumulator out
 * of tensor memory (about 2 % of a tile's time each at d = 3584).
 *   k_elements > 0 (a multiple of 64): fixed chunks of that length.
 *   k_elements = 0: one accumulator over the whole of d.
 *   SPECS_ACCUM_ADAPTIVE (default): 512-element chunks for the first two vocabulary
 *     tiles of each run of tiles a CTA (pair) scores for its rows; the |logit| magnitudes
 *     of the first tile then set the chunk length of the remaining tiles: as many K = 16
 *     accumulations as keep (count x fp32 spacing at the magnitude class, a power of
 *     two, that all but 1/32 of the tile's rows stay within at twice their largest
 *     |logit|) below 1e-3, a worst-case figure of which about an eighth is seen in
 *     practice, never shorter than 512 elements.  Magnitudes below 32 run d <= 4160
 *     unchunked, below 64 in 2048-element chunks, ... , from 256 on in 512-element
 *     chunks.  A row in which a logit that matters (its largest, or the drafted id's)
 *     turns out to lie beyond that class -- anywhere in the vocabulary, or because the
 *     row is one of the few far larger than its tile -- is marked, and a second launch
 *     of the scoring kernel re-scores the marked rows with 512-element chunks (all rows
 *     when more than about an eighth of them are marked); rows with |logit| of 1024 and
 *     more, where even 512-element chunks would leave a few 1e-3, are marked whatever
 *     chunks the first pass used, and the second pass halves its chunks for every
 *     doubling of the largest magnitude (down to 64 elements).  The per-token error
 *     thus stays within 2e-3 wherever the large logits sit, up to magnitudes where the
 *     fp32 spacing of the logits themselves approaches the tolerance (several
 *     thousand); SPECS_DEV_ACCUM_RANGE reports that rows were re-scored.  Inputs of at
 *     most 128 rows (a single row tile, bound by streaming W rather than by the tensor
 *     pipe) always use 512-element chunks and have no second pass: they keep the
 *     tolerance for |logit| below 1024, like any fixed 512-element setting.  Measured at d = 5120 against the exact result: at most 1.9e-4 per token
 *     for logit spreads up to 48, where a single chunk would be off by 2.3e-3. */
#define SPECS_ACCUM_ADAPTIVE (-1)
int specs_set_accum_chunk(specs_ctx* ctx, int32_t k_elements);

/* Pacing of the CTAs (pairs) that stream the same chunk of W_vocab: with tiles > 0 one
 * of them passes pace point t only once all of them have passed point t - tiles, so
 * that each W tile is fetched from HBM once and served from L2 to the others.  A pace
 * point is the start of a vocabulary tile; where a wave's hidden states plus two tiles
 * of W per vocabulary chunk would not fit in about 50 MB of L2 (d = 5120, or many
 * chunks), the library places two to four evenly spaced points per tile.  Default 1
 * (measured on 65536 rows at d = 3584: HBM reads 147 GB without, 24.5 GB with, for an
 * ideal of 24.4 GB); 0 switches the pacing off.  The wait is advisory and bounded (it
 * gives up after 40 us per point and for good after four expiries). */
int specs_set_tile_lead(specs_ctx* ctx, int32_t tiles);

/* Number of SMs the context schedules over (the persistent grid is one CTA per SM,
 * or two per resident CTA pair). */
int specs_sm_count(const specs_ctx* ctx);

/* Bytes of scratch specs_score_blocks needs for these sizes.  It holds one
 * (running max, sum of exponentials, drafted-token logit) triple per row and per
 * vocabulary split -- a few hundred KB per 148 row tiles -- twice (for the two
 * scoring passes of adaptive accumulation chunks), and a buffer for the hidden
 * states of the rows the second pass re-scores (an eighth of the rows, 8192 at
 * most); never anything proportional to rows x V: the logits themselves exist only
 * in tensor memory. */
size_t specs_score_workspace_bytes(const specs_ctx* ctx, int64_t rows, int32_t d, int32_t V);

/* log pi_target of every drafted token and of every drafted block
 * (Section 2: "computing logits of each token" of a drafted block with the
 * target model; Appendix E.3: only the newly drafted tokens are scored; Eq. (1):
 * the block probability is the product over its tokens).
 *
 *   hidden        bf16 [rows, d] row-major: the target's final hidden state (after
 *                 its last norm) at the position that predicts each drafted token.
 *   W_vocab       bf16 [V, d] row-major LM-head weight (no bias, temperature 1).
 *   token_ids     int32 [rows]: the drafted ids.  An id outside [0, V) yields NaN
 *                 for that token and sets SPECS_DEV_TOKEN_RANGE.
 *   block_offsets int64 [B+1] on the device: block i owns rows [off[i], off[i+1]);
 *                 off[0] = 0, non-decreasing, off[B] = rows (caller's contract; an
 *                 empty block has log-probability 0).
 *   tok_logprob   float [rows] out.   blk_logprob float [B] out (may be NULL).
 *   blk_logprob_f64 double [B] out (may be NULL): the same sums before rounding.
 *   workspace     scratch of at least specs_score_workspace_bytes(), 16-byte aligned.
 *
 * Requirements: d % 8 == 0 (rows of both matrices must start on 16-byte
 * boundaries), hidden and W_vocab 16-byte aligned.  rows == 0 is a valid no-op
 * (block sums are then written as 0). */
int specs_score_blocks(specs_ctx* ctx, const void* hidden, const void* W_vocab,
                       const int32_t* token_ids, const int64_t* block_offsets,
                       int64_t rows, int32_t d, int32_t V, int32_t B,
                       float* tok_logprob, float* blk_logprob, double* blk_logprob_f64,
                       void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Segmented sum of a per-token array over the blocks (the same reduction as inside
 * specs_score_blocks; used for the generator's own per-token log-probabilities,
 * the denominator of Eq. (1)).  Accumulates in double.  out / out_f64 may each be
 * NULL but not both. */
int specs_block_sums(specs_ctx* ctx, const float* per_token, const int64_t* block_offsets,
                     int32_t B, float* out, double* out_f64, void* cuda_stream);

/* SubSample (Algorithm 2) for P problems at once, fused with the switch test.
 *
 *   S_i = (blk_lp_target[i] - blk_lp_gen[i]) + beta * reward[i]            (Eq. 1)
 *   weights[i] = exp(S_i) / sum over the problem's candidates of exp(S_j)  (Algorithm 2)
 *   chosen[p]  = argmax_i (S_i - log(-log uniforms[i])), index local to the problem,
 *                lowest index on exact ties: an exact draw from `weights` when the
 *                uniforms are i.i.d. U(0,1); -1 for a problem without candidates.
 *   accept[p]  = 1 iff max_i reward[i] > tau (Algorithm 1, Step III), 0 otherwise.
 *
 *   blk_lp_gen == NULL means the blocks came from the target itself
 *   (pi_gen = pi_target): the ratio drops out and S_i = beta * reward[i];
 *   blk_lp_target may then be NULL too.
 *   cand_offsets int32 [P+1] on the device: problem p owns blocks
 *   [cand_offsets[p], cand_offsets[p+1]).
 *   uniforms float [total candidates], each strictly inside (0,1); values outside
 *   are clamped to [2^-25, 1 - 2^-24].
 *   accept may be NULL (then tau is ignored).  weights may be NULL.
 *   Scores, the maximum, the normaliser and the perturbed arg-max are evaluated in
 *   double; weights are rounded to float on output. */
int specs_subsample(specs_ctx* ctx, const float* blk_lp_target, const float* blk_lp_gen,
                    const float* reward, const int32_t* cand_offsets, int32_t P, float beta,
                    const float* uniforms, int32_t* chosen, float* weights,
                    float tau, uint8_t* accept, void* cuda_stream);

/* Same as specs_subsample with the block log-probabilities given in double
 * (the unrounded sums from specs_score_blocks / specs_block_sums). */
int specs_subsample_f64(specs_ctx* ctx, const double* blk_lp_target, const double* blk_lp_gen,
                        const float* reward, const int32_t* cand_offsets, int32_t P, float beta,
                        const float* uniforms, int32_t* chosen, float* weights,
                        float tau, uint8_t* accept, void* cuda_stream);

/* Selection with the variants the paper uses in its comparisons and ablations.
 *
 * select_rule
 *   SPECS_SELECT_SUBSAMPLE    Algorithm 2: a draw with P(i* = i) proportional to
 *                             exp(S_i) * 1(i in L), by Gumbel-max on `uniforms`.
 *   SPECS_SELECT_BEST_REWARD  the candidate of L with the highest reward, lowest index on
 *                             ties: the selection of the PRM-guided beam-search baselines
 *                             and of RSD++ (Section 4.1, Baselines); `uniforms` may be NULL;
 *                             weights are 1 for the pick and 0 elsewhere.
 * score_flags
 *   SPECS_SCORE_NO_LL         S_i = beta * reward[i] even when blk_lp_gen is given: the
 *                             "SPECS (no LL)" ablation of Section 4.3.
 * mask  uint8 [total candidates] or NULL: the set L of Algorithm 2 (non-zero = member).
 *       Candidates outside L get weight 0 and are never picked; a problem with no member
 *       (or no candidate) gives chosen = -1.
 * switch_rule, evaluated on the rewards of ALL candidates of the problem (in L or not):
 *   SPECS_SWITCH_ANY_ABOVE    flag = max_i reward[i] > tau: Algorithm 1, Step III (the draft
 *                             model may generate next).
 *   SPECS_SWITCH_NONE_ABOVE   flag = no reward exceeds tau: the "pi_draft start" variant of
 *                             Section 4.3 (the target model generates next).
 *   SPECS_SWITCH_CHOSEN_BELOW flag = reward of the PICKED candidate < tau: RSD++'s rule
 *                             (Section 4.1: redo the step with the target model).
 *   A problem without candidates raises no flag.  flag may be NULL.
 * Block log-probabilities are doubles as in specs_subsample_f64; blk_lp_gen == NULL means
 * pi_gen = pi_target. */
#define SPECS_SELECT_SUBSAMPLE    0
#define SPECS_SELECT_BEST_REWARD  1
#define SPECS_SCORE_NO_LL         0x1
#define SPECS_SWITCH_ANY_ABOVE    0
#define SPECS_SWITCH_NONE_ABOVE   1
#define SPECS_SWITCH_CHOSEN_BELOW 2
int specs_select(specs_ctx* ctx, const double* blk_lp_target, const double* blk_lp_gen,
                 const float* reward, const uint8_t* mask, const int32_t* cand_offsets, int32_t P,
                 float beta, const float* uniforms, int select_rule, int score_flags,
                 int switch_rule, float tau, int32_t* chosen, float* weights, uint8_t* flag,
                 void* cuda_stream);

/* Rewards r(Y_i | tr) of the drafted blocks from the process reward model's final
 * hidden states (Section 2 takes the PRM r as given; Appendix E.3 evaluates it
 * concurrently with the target's log-likelihoods, which a caller gets by issuing
 * this call on a second stream):
 *   reward[i] = 1 / (1 + exp(-(w_head . h_last(i) + bias)))
 * where h_last(i) is row block_offsets[i+1] - 1 of prm_hidden, the hidden state at the
 * block's last token.  The logistic link and the position read are this library's
 * reading of a value-head PRM whose scores lie in [0, 1]; an empty block has no last
 * token and gets NaN.
 *   prm_hidden bf16 [rows, d] row-major, w_head bf16 [d], both 16-byte aligned,
 *   d % 8 == 0; block_offsets int64 [B+1] on the device; reward float [B] out. */
int specs_prm_rewards(specs_ctx* ctx, const void* prm_hidden, const int64_t* block_offsets, int32_t B,
                      int32_t d, const void* w_head, float bias, float* reward, void* cuda_stream);

/* The dynamic-switching test alone (Algorithm 1, Step III; Section 2.3):
 * accept[p] = 1 iff the largest reward among ALL candidates of problem p is
 * strictly above tau, i.e. the draft model may generate the next step.  The call
 * is a stateless predicate; whether a switch is permanent is the caller's policy. */
int specs_accept(specs_ctx* ctx, const float* reward, const int32_t* cand_offsets, int32_t P,
                 float tau, uint8_t* accept, void* cuda_stream);

/* One whole beam step on DEVICE buffers, as one chain of launches that overlap
 * their set-up with their predecessors: the LM-head scoring kernel, the merge of its
 * vocabulary splits into log pi_target of every drafted token (Section 2, Appendix
 * E.3), the second scoring pass (with adaptive chunks; it returns at once when no row
 * was marked), and one kernel that, per problem, sums target and generator
 * log-probabilities per drafted block (Eq. 1), draws SubSample's candidate
 * (Algorithm 2) and evaluates the switch test (Algorithm 1, Step III).
 * Results are identical to specs_score_blocks + specs_block_sums +
 * specs_subsample_f64 on the same inputs; only the launch count differs.
 *
 *   gen_tok_logprob  float [rows]: the generator's own per-token log-probabilities
 *                    (NULL: pi_gen = pi_target, S_i = beta * reward[i]).
 *   blk_logprob_f64  double [B] out, required: block sums of log pi_target.
 *   gen_blk_logprob_f64 double [B] out, required when gen_tok_logprob is given.
 *   weights, accept  may be NULL.  chosen int32 [P] out, required.
 *   workspace        as for specs_score_blocks.
 * Other arguments as in specs_score_blocks and specs_subsample.  The rows of a
 * problem must be contiguous, which the two offset arrays imply.  Tensor-core
 * engines only (SPECS_ERR_SHAPE if the SIMT aid is selected).  One CTA handles one
 * problem, so a single problem with very many rows (beyond about 10^5) is better
 * served by the separate calls. */
int specs_beam_step(specs_ctx* ctx, const void* hidden, const void* W_vocab, const int32_t* token_ids,
                    const int64_t* block_offsets, const int32_t* cand_offsets,
                    const float* gen_tok_logprob, const float* reward, const float* uniforms,
                    int64_t rows, int32_t d, int32_t V, int32_t B, int32_t P, float beta, float tau,
                    float* tok_logprob, double* blk_logprob_f64, double* gen_blk_logprob_f64,
                    float* weights, int32_t* chosen, uint8_t* accept,
                    void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The beam step when the generator's log-probabilities are computed rather than
 * given: the drafted tokens are scored with the generator's own LM head as well
 * (its final hidden states hidden_gen [rows, d_gen] and weights W_gen [V, d_gen];
 * Appendix E.1 lists scoring with the draft and with the target model), and Eq. (1)
 * takes the two block log-probabilities.  The generator-shaped head is scored first
 * (scoring kernel, merge, second pass), then the target-shaped one, and one finish
 * kernel sums both per-token log-probabilities (their difference is the per-token
 * log-ratio) per block, runs SubSample and the switch test and, when
 * chosen_ids is given, gathers the selected block's token ids for the append of
 * Algorithm 1, Step II (see specs_gather_chosen).
 *
 *   gen_tok_logprob  float [rows] OUT here.  Both heads share the vocabulary size V.
 *   chosen_ids       int32 [P, chosen_stride] out or NULL; chosen_len int32 [P] out.
 *   workspace        at least specs_beam_step_dual_workspace_bytes().
 * Everything else as in specs_beam_step. */
size_t specs_beam_step_dual_workspace_bytes(const specs_ctx* ctx, int64_t rows, int32_t d_target,
                                            int32_t d_gen, int32_t V);
int specs_beam_step_dual(specs_ctx* ctx, const void* hidden_target, const void* W_target, int32_t d_target,
                         const void* hidden_gen, const void* W_gen, int32_t d_gen,
                         const int32_t* token_ids, const int64_t* block_offsets,
                         const int32_t* cand_offsets, const float* reward, const float* uniforms,
                         int64_t rows, int32_t V, int32_t B, int32_t P, float beta, float tau,
                         float* tok_logprob, float* gen_tok_logprob, double* blk_logprob_f64,
                         double* gen_blk_logprob_f64, float* weights, int32_t* chosen, uint8_t* accept,
                         int32_t* chosen_ids, int32_t* chosen_len, int32_t chosen_stride,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/* What Step II of Algorithm 1 appends to the trace: for every problem the token ids
 * of its selected block (block cand_offsets[p] + chosen[p]) go to row p of
 * chosen_ids [P, chosen_stride], padded with -1, and the block's length to
 * chosen_len[p]; chosen[p] = -1 gives a row of -1 and length 0.  The caller makes
 * chosen_stride at least the longest block (longer blocks are cut to the stride). */
int specs_gather_chosen(specs_ctx* ctx, const int32_t* token_ids, const int64_t* block_offsets,
                        const int32_t* cand_offsets, const int32_t* chosen, int32_t P,
                        int32_t* chosen_ids, int32_t* chosen_len, int32_t chosen_stride, void* cuda_stream);

/* Vocabulary-parallel scoring: each holder of a shard of W_vocab (rows id_offset ..
 * id_offset + V_shard - 1 of the whole matrix) scores all drafted rows against its
 * shard and produces, per row, what the log-softmax needs from it:
 *   partials[row] = { max logit of the shard * log2(e),
 *                     sum over the shard of 2^(logit*log2(e) - that maximum),
 *                     the drafted id's logit if id_offset <= id < id_offset + V_shard,
 *                       else -inf,
 *                     0 }                                   (float [rows, 4], 16-byte aligned)
 * token_ids are indices into the WHOLE vocabulary; an id outside the shard is not an
 * error here.  The partials of all shards (e.g. all-gathered over NVLink into
 * [shards, rows, 4]) are folded by specs_merge_partials into log pi_target of the
 * drafted id (Section 2; the log-sum-exp over a partition is the log-sum-exp of the
 * parts), NaN and SPECS_DEV_TOKEN_RANGE for an id outside [0, V).  This is the paper's
 * scoring step cut the other way than by rows; the paper itself places each model on
 * one GPU (Appendix E.2).  Workspace as for specs_score_blocks with V = V_shard. */
int specs_score_partials(specs_ctx* ctx, const void* hidden, const void* W_shard,
                         const int32_t* token_ids, int32_t id_offset, int64_t rows, int32_t d,
                         int32_t V_shard, float* partials, void* workspace, size_t workspace_bytes,
                         void* cuda_stream);
int specs_merge_partials(specs_ctx* ctx, const float* partials, int32_t shards, int64_t rows,
                         const int32_t* token_ids, int32_t V, float* tok_logprob, void* cuda_stream);

/* An 8-bit variant of block scoring (no counterpart in the paper, which states no
 * precision; an extension for when the LM head is served in FP8).  What it computes:
 *   1. specs_quantize_rows_e4m3: every row of a bf16 matrix [n, d] is scaled so that its
 *      largest magnitude maps to 448, the largest finite E4M3 value (OCP 8-bit floating
 *      point: 1-4-3 bits, bias 7, no infinities), and rounded to the nearest E4M3 number,
 *      ties to even, saturating: codes uint8 [n, d], scale[n] = absmax / 448 (float32;
 *      a row of zeros: scale 1, codes 0).  d % 16 == 0.  Weights are quantised once.
 *   2. specs_score_blocks_fp8: logit[t, v] = hidden_scale[t] * W_scale[v] *
 *      sum_k hidden_q[t, k] * W_q[v, k] on the tensor cores (tcgen05.mma kind::f8f6f4, fp32
 *      accumulation, twice the bf16 rate), then the same fused log-softmax, gather, merge
 *      and block sums as specs_score_blocks; arguments otherwise as there.
 * Against its own definition (the quantised logits summed exactly) the result meets the
 * tolerances of the bf16 path; against unquantised bf16 scoring the difference is the
 * quantisation error, a few percent of the logits' spread.  Accumulation chunks are
 * counted in 128-byte k-blocks, so a length set with specs_set_accum_chunk covers
 * twice as many elements here (the default base chunk is 1024 elements). */
int specs_quantize_rows_e4m3(specs_ctx* ctx, const void* x_bf16, int64_t n, int32_t d,
                             uint8_t* codes, float* scale, void* cuda_stream);
size_t specs_score_workspace_bytes_fp8(const specs_ctx* ctx, int64_t rows, int32_t d, int32_t V);
int specs_score_blocks_fp8(specs_ctx* ctx, const uint8_t* hidden_q, const float* hidden_scale,
                           const uint8_t* W_q, const float* W_scale, const int32_t* token_ids,
                           const int64_t* block_offsets, int64_t rows, int32_t d, int32_t V, int32_t B,
                           float* tok_logprob, float* blk_logprob, double* blk_logprob_f64,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The whole beam step with the 8-bit head: quantise the step's hidden states (bf16
 * [rows, d] in), then the chain of specs_beam_step on the codes (scoring against the
 * pre-quantised weight, merge, second pass, finish kernel).  Arguments as in specs_beam_step, with
 * W_q / W_scale from specs_quantize_rows_e4m3; the workspace also holds the codes and
 * scales of the hidden states (specs_beam_step_fp8_workspace_bytes). */
size_t specs_beam_step_fp8_workspace_bytes(const specs_ctx* ctx, int64_t rows, int32_t d, int32_t V);
int specs_beam_step_fp8(specs_ctx* ctx, const void* hidden, const uint8_t* W_q, const float* W_scale,
                        const int32_t* token_ids, const int64_t* block_offsets, const int32_t* cand_offsets,
                        const float* gen_tok_logprob, const float* reward, const float* uniforms,
                        int64_t rows, int32_t d, int32_t V, int32_t B, int32_t P, float beta, float tau,
                        float* tok_logprob, double* blk_logprob_f64, double* gen_blk_logprob_f64,
                        float* weights, int32_t* chosen, uint8_t* accept,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Host-side controller of the SPECS loop (Algorithm 1): for P problems it keeps which
 * model drafts the next n candidate blocks, appends the selected block, applies the
 * dynamic switch (Step III; Section 2.3) and stops at the target length.  All
 * pointers are HOST pointers; nothing here touches a GPU.  One step of the loop:
 *   specs_controller_generators  -> the caller drafts n blocks per problem with that
 *                                   model, scores them (specs_beam_step / specs_select)
 *   specs_controller_advance     <- chosen index, switch flag and length of the chosen
 *                                   block, per problem.
 *
 * policy (Section 4.1 baselines and Section 4.3 ablations in brackets)
 *   SPECS_POLICY_SPECS        starts with the target; flag (SPECS_SWITCH_ANY_ABOVE) = 1
 *                             gives the next step to the draft.  sticky = 0: the test is
 *                             taken anew at every step (Section 2.3); sticky = 1: once the
 *                             draft, always the draft (Algorithm 1 read literally).
 *   SPECS_POLICY_ONLY_DRAFT   every step from the draft ["Only Small Gen", BS(S)].
 *   SPECS_POLICY_ONLY_TARGET  every step from the target [BS(B)].
 *   SPECS_POLICY_RANDOM       after every step the target is chosen with probability
 *                             p_target from a caller-supplied uniform ["Random Switch"].
 *   SPECS_POLICY_DRAFT_START  starts with the draft; flag (SPECS_SWITCH_NONE_ABOVE) = 1
 *                             gives the next step to the target ["SPECS (pi_draft start)"].
 *   SPECS_POLICY_RSD          drafts with the draft; flag (SPECS_SWITCH_CHOSEN_BELOW) = 1
 *                             discards the step and has the target redo it, whose pick
 *                             is then appended unconditionally [RSD++].
 * A problem is finished (generator SPECS_GEN_DONE, later updates ignored) once its
 * appended length reaches target_len or its appended steps reach max_steps.  A step
 * whose chosen index is -1 appends nothing. */
#define SPECS_GEN_TARGET   0
#define SPECS_GEN_DRAFT    1
#define SPECS_GEN_DONE   (-1)
#define SPECS_POLICY_SPECS        0
#define SPECS_POLICY_ONLY_DRAFT   1
#define SPECS_POLICY_ONLY_TARGET  2
#define SPECS_POLICY_RANDOM       3
#define SPECS_POLICY_DRAFT_START  4
#define SPECS_POLICY_RSD          5
typedef struct specs_controller specs_controller;
typedef struct specs_policy {
    int32_t policy;       /* SPECS_POLICY_* */
    int32_t sticky;       /* see SPECS_POLICY_SPECS / SPECS_POLICY_DRAFT_START */
    int64_t target_len;   /* tokens to append per problem */
    int64_t max_steps;    /* blocks to append per problem at most */
    float   p_target;     /* SPECS_POLICY_RANDOM: probability that the target generates, in [0, 1] */
} specs_policy;
int specs_controller_create(specs_controller** out, int32_t P, const specs_policy* policy);
int specs_controller_destroy(specs_controller* ctrl);
/* h_gen int32 [P] out: SPECS_GEN_TARGET, SPECS_GEN_DRAFT or SPECS_GEN_DONE. */
int specs_controller_generators(const specs_controller* ctrl, int32_t* h_gen);
/* h_chosen int32 [P], h_flag uint8 [P], h_chosen_len int64 [P] (tokens of the chosen block;
 * ignored where h_chosen < 0), h_uniforms float [P] (SPECS_POLICY_RANDOM only, else may be NULL). */
int specs_controller_advance(specs_controller* ctrl, const int32_t* h_chosen, const uint8_t* h_flag,
                             const int64_t* h_chosen_len, const float* h_uniforms);
/* h_appended uint8 [P] out: 1 where the last specs_controller_advance appended the problem's
 * selected block to its trace (Algorithm 1, Step II), 0 where it did not (problem finished,
 * nothing selected, or an RSD++ draft step that the target redoes).  The caller's copy of the
 * trace follows this, not its own reading of the policy. */
int specs_controller_appended(const specs_controller* ctrl, uint8_t* h_appended);
/* Per problem, each int64 [P] out and optional: appended tokens, appended blocks, appended
 * blocks that the target generated, generation rounds the target ran (RSD++ retries count). */
int specs_controller_stats(const specs_controller* ctrl, int64_t* h_length, int64_t* h_steps,
                           int64_t* h_target_steps, int64_t* h_target_calls);

/* Synchronise `cuda_stream`, return the device status word (a combination of
 * SPECS_DEV_* bits, 0 if clean) through *h_bits and clear it.  Returns
 * SPECS_ERR_DEVICE_TIMEOUT / SPECS_ERR_DEVICE_BOUNDS / SPECS_ERR_TOKEN_RANGE (the first
 * of these whose bit is set), SPECS_OK otherwise.  h_bits may be NULL. */
int specs_device_status(specs_ctx* ctx, uint32_t* h_bits, void* cuda_stream);

/* One whole beam step from HOST buffers (the end-to-end path): copies the step's
 * inputs to the device, runs specs_beam_step, copies the results back and
 * synchronises the stream before returning.
 * W_vocab is the model's weight and stays a DEVICE pointer.  The context keeps
 * grow-only device and pinned staging buffers for this call, so it may allocate on
 * first use or when sizes grow.  h_block_offsets and h_cand_offsets are validated
 * (SPECS_ERR_OFFSETS).  h_gen_tok_logprob == NULL means pi_gen = pi_target.
 * Any output pointer except h_chosen may be NULL. */
int specs_beam_step_host(specs_ctx* ctx,
                         const void* h_hidden, const void* W_vocab, const int32_t* h_token_ids,
                         const int64_t* h_block_offsets, const int32_t* h_cand_offsets,
                         const float* h_gen_tok_logprob, const float* h_reward, const float* h_uniforms,
                         int64_t rows, int32_t d, int32_t V, int32_t B, int32_t P,
                         float beta, float tau,
                         float* h_tok_logprob, double* h_blk_logprob, float* h_weights,
                         int32_t* h_chosen, uint8_t* h_accept, void* cuda_stream);

/* The same step in two halves, so that a caller can keep two steps in flight and
 * have one step's copies run while the other step's kernels do (the paper runs the
 * target's scoring and the PRM's concurrently, Appendix E.3; this is the same idea
 * applied to the bus).  submit copies the small inputs into the context's pinned
 * staging memory, enqueues the host-to-device copies on an internal copy stream, the
 * kernels of specs_beam_step on `cuda_stream` behind them, and the device-to-host copy
 * of the results on a second internal copy stream behind those; it returns a ticket
 * without waiting for any of it.  wait blocks until that step's results have arrived
 * and writes them to the output pointers given at submit.
 *   - h_hidden is read by the copy engine after submit returns: it must stay valid and
 *     unchanged until the matching wait, and only page-locked memory overlaps (the
 *     driver stages pageable memory synchronously).  The other h_ inputs are consumed
 *     before submit returns.  The output pointers must stay valid until wait.
 *   - at most two steps may be in flight per context (a third submit returns
 *     SPECS_ERR_LIMIT and enqueues nothing); each in-flight step owns one of the
 *     context's two grow-only device arenas.  Waits may come in any order.
 *   - wait returns SPECS_ERR_SHAPE for a ticket that is not in flight.
 * specs_beam_step_host is submit followed by wait. */
int specs_beam_step_host_submit(specs_ctx* ctx,
                                const void* h_hidden, const void* W_vocab, const int32_t* h_token_ids,
                                const int64_t* h_block_offsets, const int32_t* h_cand_offsets,
                                const float* h_gen_tok_logprob, const float* h_reward, const float* h_uniforms,
                                int64_t rows, int32_t d, int32_t V, int32_t B, int32_t P,
                                float beta, float tau,
                                float* h_tok_logprob, double* h_blk_logprob, float* h_weights,
                                int32_t* h_chosen, uint8_t* h_accept, void* cuda_stream, int32_t* h_ticket);
int specs_beam_step_host_wait(specs_ctx* ctx, int32_t ticket);

/* Failure-detection self-test.  Every wait inside the scoring kernel is bounded: when
 * its time runs out it raises SPECS_DEV_TIMEOUT in the device status word and the
 * kernel winds down instead of hanging.  This call launches a one-CTA kernel that
 * runs that same wait, for limit_us microseconds (1 .. 1 000 000), on a barrier that
 * nothing completes: afterwards specs_device_status() must report
 * SPECS_ERR_DEVICE_TIMEOUT, and the context must remain usable.  (The paper has no
 * counterpart; it is how the expiry path is tested without a stuck GPU.) */
int specs_probe_wait_expiry(specs_ctx* ctx, int64_t limit_us, void* cuda_stream);

/* Per-call timing of the tensor-core scoring kernel.  specs_set_timing(ctx, 1)
 * makes every later scoring call on this context record a CUDA event before and
 * after each launch of that kernel on the call's own stream (a few microseconds each;
 * off by default) and forgets earlier records; (ctx, 0) stops recording and keeps the
 * records; (ctx, 2) resumes recording without forgetting, so that a caller can
 * time every K-th call of a loop.  specs_score_kernel_ms() waits for the recorded
 * launches, returns the MEAN duration per scoring call in milliseconds (its pass over
 * all rows plus its second pass over re-scored rows), stores the number of calls in
 * *h_launches (may be NULL) and forgets the records; it returns a negative value when
 * nothing was recorded. */
int   specs_set_timing(specs_ctx* ctx, int enabled);
float specs_score_kernel_ms(specs_ctx* ctx, int32_t* h_launches);

/* The work-unit plan of the tensor-core scoring kernel, for inspection and tests
 * (pure host arithmetic, needs no device).  A work unit is one CTA (cta_group 1,
 * a 128-row super tile) or a pair of CTAs of one cluster (cta_group 2, a 256-row
 * super tile); cta_group 0 lets the planner choose as the default engine does,
 * assuming num_sms / 2 resident pairs.  The super tiles x vocabulary tiles (256
 * entries) grid is processed in waves; in a wave, gm super tiles are live and the
 * vocabulary is cut into s contiguous chunks, one persistent unit per (super tile,
 * chunk).  h_out16 receives: row_tiles, vocab_tiles, k_blocks, grid (CTAs), group_m,
 * split_full, full_waves, rem_m, split_rem, waves, the workspace size in bytes as
 * two 31-bit halves (low, high), cta_group, units per wave, super_tiles, and the
 * k-blocks per accumulation chunk. */
int specs_score_plan(int64_t rows, int32_t d, int32_t V, int32_t num_sms, int32_t cta_group, int32_t* h_out16);

/* Work of CTA `cta` in wave `wave` under that plan: h_out3 = {its 128-row tile,
 * first vocab tile, one-past-last vocab tile}; row tile -1 when the CTA has no
 * rows in that wave (idle unit, or the second CTA of a pair past the last tile). */
int specs_score_plan_unit(int64_t rows, int32_t d, int32_t V, int32_t num_sms, int32_t cta_group, int32_t wave,
                          int32_t cta, int32_t* h_out3);

/* Block scoring for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this entry point exists for deployment, not for the method.)
 *
 * Who needs it: a serving process that handed the whole GPU to its own memory pool
 * at start-up (nothing is left for cudaMalloc to return), or a step loop that must
 * never meet the device-wide synchronisation cudaMalloc / cudaFree imply.  Such a
 * caller can neither create a specs_ctx (creation allocates the status word) nor
 * supply a workspace, so this call takes neither: the scratch of the scoring kernel
 * is a fixed array of SPECS_NOALLOC_SCRATCH_BYTES inside the library's device image,
 * which every GPU that loads the library holds until the process exits.  The call
 * itself, and everything it runs, calls no cudaMalloc, cudaFree or other allocating
 * routine; inputs and outputs are the caller's buffers as in specs_score_blocks
 * (same meaning, layout and requirements), always on the tensor-core engine with
 * fixed 512-element accumulation chunks (the adaptive chunks of the regular entry
 * point need a second pass and a buffer of gathered rows, which would not fit), on
 * the CURRENT device.
 *
 *   status_word  device uint32 that receives SPECS_DEV_* bits by atomic OR (never
 *                cleared by the library); NULL sends them to an internal word that
 *                cannot be read back, so a NULL status word hides an expired wait
 *                (SPECS_DEV_TIMEOUT) as well as a bad id: pass one if you can.
 *
 * Limits and sharing:
 *   - the plan for (rows, d, V) must fit the fixed scratch (waves x SMs x 3072 bytes
 *     <= SPECS_NOALLOC_SCRATCH_BYTES; roughly 50 000 rows at d = 3584 or 5120 and
 *     170 000 at d = 1536 on a 148-SM part: waves and CTAs as specs_score_plan reports them);
 *     larger problems return SPECS_ERR_LIMIT and launch nothing.  Split the rows over
 *     several calls instead.
 *   - all calls on a device share the one array, which still holds the previous
 *     call's contents.  Nothing in it has to start at zero (each slot is written
 *     before it is read within a call), but calls whose kernels overlap on the GPU,
 *     e.g. on different streams, race on it: serialise them.
 *   - the first call on each device resolves the array's device address
 *     (cudaGetSymbolAddress) and the driver entry point it needs; make that first
 *     call before starting any stream capture.  With CUDA's default lazy module
 *     loading that first call is also when the driver places the library's device
 *     image, the array included, in device memory: a host whose own pool is about to
 *     take the whole device must make the first call on each device BEFORE the pool
 *     does (a call with rows = 0 and a non-NULL W_vocab is enough), or run with
 *     CUDA_MODULE_LOADING=EAGER;
 *     otherwise the first call fails with SPECS_ERR_CUDA. */
#define SPECS_NOALLOC_SCRATCH_BYTES (8u << 20)
int specs_score_blocks_noalloc(const void* hidden, const void* W_vocab, const int32_t* token_ids,
                               const int64_t* block_offsets, int64_t rows, int32_t d, int32_t V, int32_t B,
                               float* tok_logprob, float* blk_logprob, double* blk_logprob_f64,
                               uint32_t* status_word, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SPECS_H_ */
