/*
 * disco.h - C ABI of the B200 (sm_100a) logit tails of DISCO speculative decoding
 * (Mamou et al., "Dynamic Speculation Lookahead Accelerates Speculative Decoding of
 * Large Language Models", arXiv 2405.04304).
 *
 * Two operations, each one enqueue of hand-written CUDA kernels on the caller's stream:
 *
 *   draft step   (Sec. 3, Eq. 2)  LM-head projection of one draft hidden state per sequence,
 *                soft-max statistics, greedy token, the features Concat(Top_k(y), Ent(y), i)
 *                with k = 10, the 2-layer halt classifier C_i = FFN(features) and the
 *                stopping rule  halt = (C_i < tau) or (n_drafted >= SL_max).
 *   verification (Sec. 2, Fig. 1; Sec. 3 "rejection sampling ... with zero temperature")
 *                LM-head projection of the SL+1 target hidden states, greedy token per
 *                position, longest accepted draft prefix, next ("bonus") token.
 *
 * Conventions
 *   - Every function returns DISCO_OK (0) or a negative DISCO_ERR_* code.  Nothing throws or
 *     aborts.  Argument errors are detected on the host before anything is enqueued.
 *   - Unless a parameter says "host", data pointers are DEVICE pointers owned by the caller,
 *     16-byte aligned, and must stay valid until the stream has run the call.
 *   - The LM heads and the classifier arrays are read-only inputs that the kernels start to read
 *     BEFORE the preceding kernel of the stream has finished (programmatic dependent launch; everything
 *     else is touched only after it has).  The work enqueued immediately before a call must therefore
 *     not write them.
 *   - bf16 matrices are row-major with the hidden dimension contiguous; hidden widths are
 *     multiples of 8.
 *   - The library owns only the opaque context: scratch for cross-block reductions, a device
 *     status word, and staging for the *_host entry points.  A context serves one stream at a
 *     time; calls on the same context must not overlap on the GPU.
 *   - No call synchronises the host except disco_create, disco_destroy,
 *     disco_last_device_status and the *_host entry points.
 *   - Kernels never trap or spin without bound: a condition they detect (inconsistent
 *     row offsets, a wait that ran out) is recorded in the device status word.
 */
#ifndef DISCO_H_
#define DISCO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DISCO_TOPK 10                 /* k of Top_k in Eq. 2 (footnote: k = 10 in all experiments) */
#define DISCO_NFEAT (DISCO_TOPK + 2)  /* top-k probabilities, entropy, position */
#define DISCO_MAX_CLF_HIDDEN 256

enum {
    DISCO_OK = 0,
    DISCO_ERR_INVALID_ARG = -1,       /* null / misaligned pointer, size out of range */
    DISCO_ERR_UNSUPPORTED_SHAPE = -2, /* shape outside what the kernels handle */
    DISCO_ERR_WORKSPACE = -3,         /* batch or row count beyond what the context was created for */
    DISCO_ERR_CUDA = -4,              /* a CUDA runtime call failed */
    DISCO_ERR_TIMEOUT = -5,           /* a bounded device-side wait ran out (device status word only); the
                                         context's counters are then undefined: destroy it */
    DISCO_ERR_STATIC_LIMIT = -6       /* size beyond the fixed scratch of disco_draft_step_static */
};

typedef struct disco_ctx disco_ctx;

/* Halt classifier of Eq. 2, read as the "shallow 2-layer FFN" of Sec. 4:
 *   C = sigmoid(w2 . relu(W1 x + b1) + b2),  x = the DISCO_NFEAT features.
 * The struct itself lives on the host; the four pointers are device fp32 arrays
 * (4-byte alignment is enough).  1 <= H <= DISCO_MAX_CLF_HIDDEN. */
typedef struct {
    const float* W1; /* [H, DISCO_NFEAT] row-major */
    const float* b1; /* [H] */
    const float* w2; /* [H] */
    const float* b2; /* [1] */
    int H;
} disco_clf;

/* Create a context on the current CUDA device for LM heads of V rows, draft hidden width
 * d_draft and target hidden width d_target, at most max_batch sequences per draft step and
 * at most max_rows (sum over sequences of SL+1) rows per verification.  k must be DISCO_TOPK;
 * clf_hidden is the largest classifier width that will be used.  Allocates device scratch
 * (host-synchronising).  *out is set only on success. */
int disco_create(disco_ctx** out, int V, int d_draft, int d_target, int max_batch, int max_rows,
                 int k, int clf_hidden);

/* Free everything the context owns.  The caller must have synchronised the stream(s) it used. */
int disco_destroy(disco_ctx* ctx);

/* Static, human-readable text for a return code. */
const char* disco_strerror(int code);

/* Host-synchronising: copy the device status word (DISCO_OK or the first DISCO_ERR_* a kernel
 * recorded since the last query) to *out and clear it.  Meant for tests and debugging. */
int disco_last_device_status(disco_ctx* ctx, int* out);

/* Number of kernels the library has launched through this context since creation. */
int disco_launch_count(disco_ctx* ctx, long long* out);

/* Kernel selection (tuning and tests): which = 0 automatic (default), 1 force the CUDA-core
 * streaming kernels, 2 force the tcgen05 kernels with the hidden rows on the TMEM lanes, 3 prefer the
 * tcgen05 kernel with the vocabulary on the TMEM lanes (draft step, up to 16 sequences). */
int disco_set_kernel_path(disco_ctx* ctx, int which);

/* For the test-suite: how the bounded device-side waits behave when what they wait for never comes.
 *   wait_budget_clocks  SM clock ticks after which a wait gives up and records DISCO_ERR_TIMEOUT in the device
 *                       status word (0 restores the default of about 0.05 s); applies to every context of the
 *                       process
 *   withhold_records    non-zero: the batched draft step (the tensor-core kernel for five sequences and more)
 *                       makes its finishing warps look for per-CTA records that no CTA publishes, so that
 *                       their wait runs out.  The kernel still returns by itself; its outputs are then
 *                       meaningless and the context must be destroyed (see DISCO_ERR_TIMEOUT).
 * Nothing traps, faults or waits without bound in either setting. */
int disco_test_hooks(disco_ctx* ctx, long long wait_budget_clocks, int withhold_records);

/*
 * One draft step for B sequences (Sec. 3, Eq. 2).  B = 1 is the single-sequence call.
 *   W_D        bf16 [V, d_draft]   draft LM head
 *   h_D        bf16 [B, d_draft]   last draft hidden state of each sequence
 *   pos        int32 [B]           feature i: position of the token being drafted, counted from
 *                                  the start of generation (App. D); used as (float) pos
 *   n_drafted  int32 [B]           draft tokens of this iteration including this one (>= 1)
 *   active     uint8 [B] or NULL   0 = skip the sequence: none of its outputs is written
 *   clf        host struct         classifier parameters (device arrays)
 *   tau        threshold; halt iff C < tau (C == tau continues) or n_drafted >= sl_max
 * Outputs
 *   token      int32 [B]           greedy draft token: lowest index attaining the largest logit
 *   conf       float [B]           C
 *   halt       uint8 [B]           1 = stop drafting and hand over to the target
 *   feats      float [B, DISCO_NFEAT] or NULL   the feature vector (top-10 probabilities
 *                                  descending, entropy in nats, (float) pos)
 *   probs      float [B, V] or NULL   the full soft-max vector; test/debug only (costs a second
 *                                  pass over [B, V] floats)
 * Logits are accumulated in fp32 from bf16 inputs and never written to memory (unless probs).
 */
int disco_draft_step(disco_ctx* ctx, const void* W_D, const void* h_D, int B,
                     const int32_t* pos, const int32_t* n_drafted, const uint8_t* active,
                     const disco_clf* clf, float tau, int sl_max,
                     int32_t* token, float* conf, uint8_t* halt, float* feats, float* probs,
                     void* stream);

/*
 * Draft step with the rule-based stopping test of App. F ("ppl SL-opt") in place of the classifier:
 * the confidence in the tokens drafted so far in this iteration is their perplexity,
 *     ppl_n = exp( -(1/n) * sum_{j <= n} ln y^D_j(t_j) ),
 * lower meaning more confident; drafting stops when ppl_n > ppl_max or n_drafted >= sl_max.
 * With greedy drafting t_j attains the largest logit, so -ln y^D_j(t_j) = ln Z_j (Z_j = sum exp(z - max z)).
 *   nll_sum    float [B], device, in/out: the sum of -ln y over the tokens drafted earlier in this
 *              iteration (0 before the first one); the call adds this token's term (active sequences only)
 *   n_drafted  int32 [B]  draft tokens of this iteration including this one (>= 1)
 * Outputs: token [B], ppl [B] (the perplexity including this token), halt [B].
 * Other arguments as in disco_draft_step.
 */
int disco_draft_step_ppl(disco_ctx* ctx, const void* W_D, const void* h_D, int B,
                         const int32_t* n_drafted, const uint8_t* active, float* nll_sum,
                         float ppl_max, int sl_max, int32_t* token, float* ppl, uint8_t* halt,
                         void* stream);

/*
 * Draft step with a sampled token (decoding at temperature 1, the mode of Table 6): everything as in
 * disco_draft_step, except that the token is drawn from y^D = softmax(W_D h) instead of being its
 * arg-max.  The draw is by inverse CDF with the caller's uniform:
 *     token = min { v : y^D_0 + .. + y^D_v > u * sum_w y^D_w }.
 * Features, classifier and stopping rule do not depend on the token and are unchanged.
 *   u        float [B], device   uniforms in [0, 1), one per sequence
 *   p_token  float [B] or NULL   y^D(token)
 *   probs    float [B, V], device, REQUIRED: receives y^D; the verification needs these rows (hand the
 *            rows of step i in as draft_probs[i] of disco_verify_sample_ragged)
 * Other arguments, layouts, ownership and errors as in disco_draft_step.
 */
int disco_draft_step_sample(disco_ctx* ctx, const void* W_D, const void* h_D, int B,
                            const int32_t* pos, const int32_t* n_drafted, const uint8_t* active,
                            const disco_clf* clf, float tau, int sl_max, const float* u,
                            int32_t* token, float* p_token, float* conf, uint8_t* halt, float* feats,
                            float* probs, void* stream);

/*
 * Verification with sampling (temperature 1; Table 6): the rejection-sampling scheme of Leviathan et al.
 * that Sec. 3 names, of which disco_verify_ragged is the zero-temperature case.  Rows and row_off as in
 * disco_verify_ragged.  With y^T_r = softmax(W_T H_T[r]) and y^D_i the distribution draft token t_i was
 * drawn from, token i of a sequence is accepted iff
 *     u_accept_i * y^D_i(t_i) < y^T_i(t_i)        (probability min(1, y^T_i(t_i) / y^D_i(t_i))),
 * n_accept is the number accepted before the first rejection, and next_token is drawn by inverse CDF with
 * u_sample[b] from norm(max(0, y^T_n - y^D_n)) after a rejection at position n, from y^T_SL if all were
 * accepted (a residual without mass falls back to y^T_n).
 *   draft_ids    int32 [R - B], device   packed as in disco_verify_ragged
 *   draft_probs  float [steps, B, V], device, steps >= max SL_b: draft_probs[i, b, :] = y^D of token i of
 *                sequence b (the probs output of draft step i); NULL allowed iff R == B.  The kernel cannot see
 *                `steps`: it reads draft_probs[i] for every i below the look-ahead that row_off gives a sequence
 *                (at most R - B), so a caller that cannot vouch for row_off sizes the array for R - B steps
 *   row_off      int32 [B + 1], device, or NULL for a uniform SL = R / B - 1
 *   u_accept     float [R - B], device   uniforms in [0, 1), packed like draft_ids
 *   u_sample     float [B], device       uniforms in [0, 1)
 * Outputs (device):
 *   n_accept [B], next_token [B]
 *   y_T         float [R, V], REQUIRED: receives the target distributions (also the call's work space)
 *   target_ids  int32 [R] or NULL: arg-max of every target row
 * Errors as in disco_verify_ragged; a draft id outside [0, V) sets the device status to
 * DISCO_ERR_INVALID_ARG and ends that sequence's acceptance there.
 */
int disco_verify_sample_ragged(disco_ctx* ctx, const void* W_T, const void* H_T,
                               const int32_t* draft_ids, const float* draft_probs,
                               const int32_t* row_off, int B, int R,
                               const float* u_accept, const float* u_sample,
                               int32_t* n_accept, int32_t* next_token, float* y_T, int32_t* target_ids,
                               void* stream);

/*
 * Bulk feature extraction for classifier training (App. D; Sec. 4 "SL classifier training"): N positions
 * at once, each with the draft model's and the target model's hidden state for the same prefix.
 *   y^D = softmax(W_D H_D[n]),  y^T = softmax(W_T H_T[n])
 *   feats_D[n] = Concat(Top_10(y^D), Ent(y^D), pos[n]);  feats_T[n] the same from y^T   (Eq. 2's features)
 *   label[n]   = 1 ("accepted") iff arg-max y^D == arg-max y^T, else 0
 *   tv[n]      = TV(y^D, y^T) = (1/2) sum_v |y^D_v - y^T_v|   (the distance named for the training loss)
 * Arguments (device pointers):
 *   W_D bf16 [V, d_draft], H_D bf16 [N, d_draft], W_T bf16 [V, d_target], H_T bf16 [N, d_target],
 *   pos int32 [N]; 1 <= N <= max_rows of disco_create
 * Outputs (device): feats_D, feats_T float [N, 12]; tv float [N]; label uint8 [N];
 *   token_D, token_T int32 [N] (the arg-max ids); y_D, y_T float [N, V]: the two distributions (also
 *   the call's work space).  All REQUIRED.
 * Errors as in disco_draft_step.
 */
int disco_extract_features(disco_ctx* ctx, const void* W_D, const void* H_D, const void* W_T, const void* H_T,
                           const int32_t* pos, int N, float* feats_D, float* feats_T, float* tv,
                           uint8_t* label, int32_t* token_D, int32_t* token_T, float* y_D, float* y_T,
                           void* stream);

/*
 * Verification with the same look-ahead SL for all B sequences (Sec. 2; Fig. 1).
 *   W_T        bf16 [V, d_target]          target LM head
 *   H_T        bf16 [B*(SL+1), d_target]   row b*(SL+1)+j is the target hidden state whose
 *                                          next-token prediction is compared with draft token
 *                                          j+1 of sequence b; row SL predicts the token after
 *                                          the last draft token
 *   draft_ids  int32 [B*SL]                (may be NULL when SL == 0)
 * Outputs
 *   n_accept   int32 [B]    length of the longest prefix with draft_ids[b,j] == target token j
 *   bonus      int32 [B]    target token at row n_accept (always emitted after the prefix)
 *   target_ids int32 [B*(SL+1)] or NULL   greedy target token of every row
 * SL = 0 is a plain target step: n_accept = 0, bonus = the target token.
 */
int disco_verify(disco_ctx* ctx, const void* W_T, const void* H_T, const int32_t* draft_ids,
                 int B, int SL, int32_t* n_accept, int32_t* bonus, int32_t* target_ids,
                 void* stream);

/*
 * Verification with a per-sequence look-ahead (the SL chosen by the halt classifier differs
 * between sequences).  Sequence b owns rows row_off[b] .. row_off[b+1]-1 of H_T (SL_b + 1 rows)
 * and the SL_b draft ids starting at draft_ids[row_off[b] - b].
 *   H_T        bf16 [R, d_target],  R = row_off[B] (passed by value; the host does not read row_off)
 *   draft_ids  int32 [R - B]
 *   row_off    int32 [B + 1], device, increasing by at least 1, row_off[0] = 0
 * If the kernel finds row_off inconsistent with R it records DISCO_ERR_INVALID_ARG in the
 * device status word and writes -1 to n_accept and bonus of the offending sequences.
 */
int disco_verify_ragged(disco_ctx* ctx, const void* W_T, const void* H_T, const int32_t* draft_ids,
                        const int32_t* row_off, int B, int R,
                        int32_t* n_accept, int32_t* bonus, int32_t* target_ids, void* stream);

/*
 * The draft phase of one speculative iteration with the look-ahead decided on the device (Sec. 3: the
 * classifier decides "immediately after generating any draft token" whether the next one is drafted; the
 * footnote on SL_max: fixed tensor shapes).  One enqueue runs up to sl_max draft steps; step i (1-based) is
 * disco_draft_step on the hidden states h_D[i-1] with pos = pos0 + i and n_drafted = i, for the sequences
 * that have not stopped yet, and the halt flag it produces is consumed on the device: no host round trip
 * between the steps.  A step that finds no sequence drafting any more returns at once.  (In this isolated
 * tail the hidden state of every step is an input; a decoder would produce h_D[i] from token i-1.  Step i
 * reads h_D[i-1] only after step i-1 has finished.)
 *   W_D            bf16 [V, d_draft]            draft LM head
 *   w_step_stride  bytes between the LM heads used by consecutive steps; 0 = the same head for every step
 *                  (the normal case).  Non-zero lets a benchmark rotate through copies of the head so that
 *                  no step finds it in L2; a multiple of 16
 *   h_D            bf16 [sl_max, B, d_draft]    step-major
 *   pos0           int32 [B]                    tokens generated before this iteration
 *   sl_forced      int32 [B] or NULL            non-NULL overrules the stopping rule: sequence b drafts
 *                  exactly min(sl_forced[b], sl_max) tokens (>= 1); the classifier still runs and reports
 *   tau <= 0 is the static policy (SL = sl_max for every sequence); tau > 1 gives SL = 1.
 * Outputs (device), step-major; entries of steps a sequence did not take are not written:
 *   token, conf, halt [sl_max, B];  feats [sl_max, B, DISCO_NFEAT] or NULL
 *   sl             int32 [B]                    tokens drafted by each sequence (1 .. sl_max)
 * B <= max_batch of disco_create.  Errors as in disco_draft_step.
 */
int disco_draft_loop(disco_ctx* ctx, const void* W_D, size_t w_step_stride, const void* h_D, int B,
                     const int32_t* pos0, const disco_clf* clf, float tau, int sl_max,
                     const int32_t* sl_forced, int32_t* token, float* conf, uint8_t* halt, float* feats,
                     int32_t* sl, void* stream);

/*
 * Verification in the fixed-shape layout, with the per-sequence look-ahead read from device memory (the sl
 * output of disco_draft_loop): the second half of a device-resident iteration (Sec. 2, Fig. 1; Sec. 3).
 *   H_T        bf16 [B, sl_max + 1, d_target]   row j of sequence b predicts the token after draft token j;
 *                                               rows beyond sl[b] are projected but do not count
 *   draft_ids  int32; draft token j of sequence b is draft_ids[b * ids_stride_b + j * ids_stride_j]
 *              ([B, sl_max] row-major: strides (sl_max, 1); the step-major token output of disco_draft_loop:
 *              strides (1, B)); may be NULL when sl_max == 0
 *   sl         int32 [B], device, 0 <= sl[b] <= sl_max (outside: DISCO_ERR_INVALID_ARG in the status word,
 *              -1 in that sequence's outputs)
 * Outputs (device): n_accept [B], bonus [B] as in disco_verify;
 *   target_ids int32 [B, sl_max + 1] or NULL: greedy target token of rows 0 .. sl[b] (others not written)
 *   row_off    int32 [B + 1] or NULL: exclusive prefix sums of sl[b] + 1, the offsets of the packed rows
 *   pos_next   int32 [B] or NULL: pos0[b] + n_accept[b] + 1, the token count after this iteration (its
 *              accepted tokens and the bonus token), i.e. the next iteration's pos0; may be pos0 itself
 *              (pos0 int32 [B], device, is read only for this and may be NULL when pos_next is)
 * B * (sl_max + 1) <= max_rows of disco_create.
 */
int disco_verify_sl(disco_ctx* ctx, const void* W_T, const void* H_T, const int32_t* draft_ids,
                    long long ids_stride_b, long long ids_stride_j, const int32_t* sl, int B, int sl_max,
                    int32_t* n_accept, int32_t* bonus, int32_t* target_ids, int32_t* row_off,
                    const int32_t* pos0, int32_t* pos_next, void* stream);

/*
 * One whole iteration as one call: disco_draft_loop, then disco_verify_sl on what it drafted.
 *   draft_ids  int32 [B, sl_max] or NULL.  NULL: the target checks the tokens the draft phase produced (the
 *              real loop).  Non-NULL: these ids are offered to the target instead (synthetic workloads plant
 *              the target's own tokens there, corrupted at a given rate, to set the acceptance rate).
 * Other arguments and outputs as in the two calls above.  Nothing is read back by the host.
 */
int disco_iteration(disco_ctx* ctx, const void* W_D, size_t w_step_stride, const void* h_D, const void* W_T,
                    const void* H_T, int B, const int32_t* pos0, const disco_clf* clf, float tau, int sl_max,
                    const int32_t* sl_forced, const int32_t* draft_ids,
                    int32_t* token, float* conf, uint8_t* halt, float* feats, int32_t* sl,
                    int32_t* n_accept, int32_t* bonus, int32_t* target_ids, int32_t* row_off,
                    int32_t* pos_next, void* stream);

/*
 * The same two operations for a caller whose per-step data lives in HOST memory (pinned memory
 * makes the copies asynchronous).  The LM heads and classifier parameters stay on the device;
 * the hidden states, integer inputs and every output are host pointers.  Each call copies the
 * hidden states to device staging owned by the context, passes the small inputs and outputs through
 * pinned host memory that the GPU maps (the kernels read and write it in place), runs the kernels
 * and synchronises the stream before returning.  feats / target_ids may be NULL.
 */
int disco_draft_step_host(disco_ctx* ctx, const void* W_D /*device*/, const void* h_D_host, int B,
                          const int32_t* pos_host, const int32_t* n_drafted_host,
                          const uint8_t* active_host /*or NULL*/, const disco_clf* clf /*device arrays*/,
                          float tau, int sl_max, int32_t* token_host, float* conf_host,
                          uint8_t* halt_host, float* feats_host, void* stream);

int disco_verify_ragged_host(disco_ctx* ctx, const void* W_T /*device*/, const void* H_T_host,
                             const int32_t* draft_ids_host, const int32_t* row_off_host, int B, int R,
                             int32_t* n_accept_host, int32_t* bonus_host, int32_t* target_ids_host,
                             void* stream);

/*
 * disco_iteration for a caller whose per-iteration data lives in HOST memory: the hidden states of all steps,
 * the target rows, pos0, sl_forced and draft_ids (either may be NULL) are host pointers, and so are the
 * outputs token, conf, halt [sl_max, B], sl, n_accept, bonus [B] and pos_next [B] (or NULL; may be pos0_host
 * itself).  One copy of each hidden-state block to device staging (the target rows travel on a stream the
 * context owns while the draft phase runs on the caller's; the verification waits for them), the small arrays
 * through pinned memory that the GPU maps, the whole iteration on the device, one synchronisation.  The LM
 * heads and the classifier stay on the device.  Entries of steps a sequence did not take keep the caller's
 * values.  Like every *_host entry point it returns with its work done, and it cannot be captured in a graph.
 */
int disco_iteration_host(disco_ctx* ctx, const void* W_D /*device*/, size_t w_step_stride, const void* h_D_host,
                         const void* W_T /*device*/, const void* H_T_host, int B, const int32_t* pos0_host,
                         const disco_clf* clf /*device arrays*/, float tau, int sl_max,
                         const int32_t* sl_forced_host, const int32_t* draft_ids_host,
                         int32_t* token_host, float* conf_host, uint8_t* halt_host, int32_t* sl_host,
                         int32_t* n_accept_host, int32_t* bonus_host, int32_t* pos_next_host, void* stream);

/*
 * Draft step without any allocation.  (The paper has no counterpart: this is a packaging variant of
 * disco_draft_step, not another operation.)
 *
 * Who needs it: hosts that must not allocate device memory - a serving process whose GPU memory is
 * owned and capped by another component that hands this library no allocator, or a decode loop that
 * cannot take the device-wide synchronisation a cudaMalloc may bring.  disco_create allocates its
 * scratch with cudaMalloc, so those hosts cannot have a context.  This entry point needs none: the
 * scratch for the cross-block reduction lives in a fixed array inside the library image
 * (about 256 KB of device memory on every GPU that loads the library, held until the process exits),
 * and the call itself uses no cudaMalloc, cudaFree or allocating library routine.
 *
 * Arguments and results are those of disco_draft_step (same layouts, device pointers owned by the
 * caller; there is no probs output), with the LM-head shape passed by value since there is no context.
 * Limits, checked before anything is enqueued: B <= DISCO_STATIC_MAX_BATCH and at most
 * DISCO_STATIC_MAX_GRID vocabulary slabs (V up to about two million rows); beyond them the call
 * returns DISCO_ERR_STATIC_LIMIT and does nothing.
 *
 * The first call on each device resolves the array's device address and raises the kernel's
 * shared-memory limit (with that device current; host threads that race to it take turns behind a
 * lock); make that first call before any stream capture.
 * All calls on a device share the one array: it keeps the previous call's contents (the call clears
 * the words that must start at zero), and two calls that overlap on the GPU - different streams, or a
 * context-free call racing another - corrupt each other's results.  Issue them on one stream, or
 * otherwise one after the other.  Kernel-detected conditions are not reported by this entry point.
 */
#define DISCO_STATIC_MAX_BATCH 4
#define DISCO_STATIC_MAX_GRID 1024
int disco_draft_step_static(int V, int d_draft, const void* W_D, const void* h_D, int B,
                            const int32_t* pos, const int32_t* n_drafted, const uint8_t* active,
                            const disco_clf* clf, float tau, int sl_max,
                            int32_t* token, float* conf, uint8_t* halt, float* feats, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* DISCO_H_ */
