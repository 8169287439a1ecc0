/*
 * svip.h -- C ABI of the SVIP speculative-decoding epilogue library (sm_100a).
 *
 * The library computes, on the GPU, the vocabulary-wide per-step work of
 * self-verification speculative decoding (SVIP, arXiv 2411.18462):
 *   draft side : temperature softmax, entropy, sample, entropy stop test
 *                (Algorithm 1 inner loop, Eq. 7)
 *   target side: softmax of the K+1 target rows, accept test min(1, p/q),
 *                first rejection, correction token from the normalised
 *                residual max(0, p - q) or bonus token
 *                (Algorithm 1 outer-loop body, Algorithms 2-5)
 * Model forwards are not part of it: callers hand over logits.
 *
 * Conventions for every call
 *   - Pointers marked DEVICE point to memory of the context's GPU, owned by
 *     the caller.  Logit rows must be aligned to their element size; any row
 *     start, any row stride and any V are accepted.  Pointers marked HOST are
 *     ordinary host memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Calls enqueue work on it and return; they never synchronise
 *     and never allocate (only svip_create and svip_graph_end allocate,
 *     only svip_read_status synchronises).
 *   - Return value: SVIP_OK (0) or a negative svip_status.  Argument errors
 *     are found on the host before anything is launched.  Data-dependent
 *     trouble (a row whose maximum is not finite, a draft length outside
 *     [1, K_max]) never traps: it sets bits in a device status word that
 *     svip_read_status returns.
 *   - Logits: SVIP_F32 = IEEE binary32, SVIP_BF16 = bfloat16.  Arithmetic is
 *     fp32.  -inf logits carry zero mass; NaN logits are treated as -inf.
 *   - Temperature T > 0 selects sampling; T == 0 selects the greedy variants
 *     (lowest-index argmax of the raw logits).
 *   - Uniform random numbers are inputs (fp32 in [0,1)); the library draws
 *     none itself.
 *   - Inverse-CDF sampling: the token is the first index whose cumulative
 *     weight, in index order, exceeds u * total.
 *   - A context is bound to one device and may be used by one host thread at
 *     a time; calls that share a context must not overlap on the GPU (they
 *     share its workspace).
 */
#ifndef SVIP_H
#define SVIP_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct svip_ctx svip_ctx;
typedef struct svip_graph svip_graph;

typedef enum { SVIP_F32 = 0, SVIP_BF16 = 1 } svip_dtype;

typedef enum {
    SVIP_OK = 0,
    SVIP_ERR_INVALID_ARG = -1, /* null pointer, size <= 0, T < 0, NaN threshold, misaligned pointer */
    SVIP_ERR_UNSUPPORTED = -2, /* unknown dtype, device that is not compute capability 10.x */
    SVIP_ERR_WORKSPACE = -3,   /* more rows than the context was created for */
    SVIP_ERR_CUDA = -4,        /* a CUDA runtime call failed; svip_last_cuda_error() has its code */
    SVIP_ERR_STATE = -5        /* graph capture begun twice, ended without begin, ... */
} svip_status;

/* bits of the device status word */
#define SVIP_STATUS_NONFINITE_ROW 1u /* some row's maximum was +inf, or every logit was -inf / NaN */
#define SVIP_STATUS_BAD_DRAFT_LEN 2u /* svip_pack_ragged saw K_i outside [1, K_max] (it was clamped) */
#define SVIP_STATUS_WAIT_TIMEOUT 4u  /* a block waited a second for its cluster's partial results and gave up; the
                                        outputs of that call are not valid */

#define SVIP_STATUS_BAD_TREE 8u      /* svip_verify_tree saw a parent index that is not below its node, or more
                                        rejected candidates at one node than it supports (the rest was ignored) */

#define SVIP_STATUS_DEBUG_OOB 16u    /* bounds-checked build only: a kernel asked for logits outside the buffers
                                        of its call (the load was not performed) */

/* draft-side layout selector for svip_verify: rows packed sequence after sequence */
#define SVIP_Q_PACKED (-1L)

/* Text for a status code (static storage). */
const char* svip_strerror(int status);

/* Library version, major*10000 + minor*100 + patch. */
int svip_version(void);

/* CUDA error code of the last call that returned SVIP_ERR_CUDA on this context (0 if none). */
int svip_last_cuda_error(const svip_ctx* ctx);

/*
 * Creates a context on `device` with a workspace for up to `max_rows` target
 * rows (and as many draft rows) per svip_verify call.  Allocates device
 * memory (about 32 bytes per row); makes `device` current while it runs and
 * restores the previous device.  *ctx is written only on success.
 */
int svip_create(svip_ctx** ctx, int device, int max_rows);

/* Frees the workspace.  The caller must have drained all streams that used the context. */
int svip_destroy(svip_ctx* ctx);

/*
 * Launch-shape override, for tests and tuning: `cluster_size` in 0..8
 * is the number of thread blocks (one cluster) that share one logits row;
 * 0 restores the automatic choice from (rows, V, dtype).  Every choice gives
 * the same integers, and entropies equal to within fp32 summation order.
 */
int svip_set_cluster_size(svip_ctx* ctx, int cluster_size);

/* Number of kernels this context has launched (or recorded into a graph) so far. */
long svip_launch_count(const svip_ctx* ctx);

/* Copies the device status word to *flags (HOST) and clears it.  Synchronises `stream`. */
int svip_read_status(svip_ctx* ctx, unsigned* flags, void* stream);

/*
 * One draft token for each of B sequences (Algorithm 1, inner loop: the
 * sampling line and the entropy test; Eq. 7).
 *
 *   logits      DEVICE, row b starts at element b*row_stride and has V logits
 *   T           temperature; T > 0: q = softmax(logits/T), token ~ q by inverse
 *               CDF at uniforms[b], entropy = H(q).  T == 0: token = argmax,
 *               entropy = H(softmax(logits)) (temperature 1).
 *   thresh      h of Eq. 7
 *   uniforms    DEVICE [B] fp32 in [0,1); may be NULL when T == 0
 *   token       DEVICE [B] int32 out
 *   entropy     DEVICE [B] fp32 out, nats, >= 0
 *   stop        DEVICE [B] uint8 out: 1 iff sqrt(entropy) > thresh (strict)
 *   row_stats   DEVICE [B][2] fp32 out or NULL: (m, Z) with m the largest logit
 *               and Z = sum_i exp((l_i - m)/T') where T' = T (or 1 when T == 0);
 *               svip_verify takes these as q_stats and then need not re-read
 *               the draft rows whose tokens it accepts
 */
int svip_draft_step(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V,
                    long row_stride, float T, float thresh, const float* uniforms,
                    int32_t* token, float* entropy, uint8_t* stop, float* row_stats,
                    void* stream);

/*
 * svip_draft_step with a per-row mask: rows whose active[b] is 0 are skipped
 * (their outputs are left untouched, their logits are not read).  `active` is
 * DEVICE [B] uint8, or NULL for "all rows", which is svip_draft_step.  This is
 * the draft step of a batch in which some sequences have already stopped
 * drafting (the inner loop of Algorithm 1, run for B sequences at once).
 */
int svip_draft_step_masked(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V,
                           long row_stride, float T, float thresh, const float* uniforms,
                           const uint8_t* active, int32_t* token, float* entropy, uint8_t* stop,
                           float* row_stats, void* stream);

/*
 * svip_draft_step_masked over a buffer that holds the logits of all draft
 * positions of a round, with the position taken from device memory: sequence b
 * reads the row that starts at element b*row_stride + pos[b]*pos_stride, takes
 * its uniform from uniforms[pos[b]*slot_stride + b] and writes token, entropy
 * and row_stats (two floats) at that same index pos[b]*slot_stride + b; stop[b]
 * is indexed by sequence alone.  With pos = the draft_len array of
 * svip_policy_advance, a position-major buffer [K_max][B][V] (pos_stride =
 * B*V, slot_stride = B) is filled slot by slot as Algorithm 1's inner loop
 * advances, each sequence at its own length, and svip_verify then reads the
 * rows, tokens and row_stats with q_seq_stride = 1, q_pos_stride = B.
 * `pos` is DEVICE [B] int32 (values >= 0; the caller keeps them below the
 * buffer's positions, e.g. through K_cap of svip_policy_advance); NULL means
 * position 0 for every sequence, i.e. svip_draft_step_masked.
 */
int svip_draft_step_at(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V,
                       long row_stride, long pos_stride, const int32_t* pos, long slot_stride,
                       float T, float thresh, const float* uniforms, const uint8_t* active,
                       int32_t* token, float* entropy, uint8_t* stop, float* row_stats, void* stream);

/*
 * Truncation threshold of every row for top-k and nucleus (top-p) sampling.
 * The paper runs its policy on top of samplers that truncate the distribution
 * but does not define the truncation; this library uses the published
 * definitions with ties kept by value:
 *   tau_k = the k-th largest logit of the row (top_k in 1..V-1; 0 or >= V: off)
 *   tau   = the largest logit value v for which the mass of {l >= v} reaches
 *           top_p times the mass of {l >= tau_k} (top_p in (0,1); >= 1: off,
 *           tau = tau_k), masses being those of softmax(l / T)
 * thr[r] receives tau of row r as a logit value (-inf when nothing is
 * dropped): the kept tokens are exactly those with logit >= thr[r], so tokens
 * tied with the last kept one stay.  tau_k is exact; the nucleus compares fp32
 * masses (summed as 2^-40 fixed point, so the result does not depend on the
 * order of summation) and may differ from an fp64 evaluation where the running
 * mass comes within about 1e-6 of top_p.  T > 0.  NaN logits count as -inf.
 * Cost: with a small top_k (at most a quarter of the threads that share a row,
 * i.e. 128 .. 1024) every row is read twice, with or without top_p; otherwise
 * once per radix pass: 2 (bf16) or 4 (fp32) passes for top-k, as many again
 * for the nucleus (+1 for the nucleus alone).
 *   logits  DEVICE, row r starts at element r*row_stride;  thr  DEVICE [n_rows] fp32 out
 *   stats   DEVICE [n_rows][2] fp32 out, or NULL: (m, Z) of the truncated
 *           distribution in the convention of svip_draft_step's row_stats (m the
 *           largest logit, Z the mass of the kept set relative to it), 8-byte
 *           aligned; svip_verify_filtered takes them as p_stats.  Free with a
 *           small top_k; one more pass over the row otherwise.
 */
int svip_row_threshold(svip_ctx* ctx, const void* logits, svip_dtype dtype, int n_rows, int V,
                       long row_stride, float T, int top_k, float top_p, float* thr, float* stats,
                       void* stream);

/*
 * The draft step and the verification round on truncated distributions: every
 * distribution is softmax(l / T) restricted to the tokens whose logit is >= the
 * row's threshold (from svip_row_threshold) and renormalised.  Sampling,
 * entropy and stop test (Algorithm 1, Eq. 7), acceptance (Algorithm 2) and the
 * residual (Algorithm 4) are those of svip_draft_step_masked / svip_verify
 * applied to these distributions; a draft token that the target's truncation
 * dropped has target probability zero and is rejected.  T > 0 only.
 *   thr     DEVICE [B] fp32: threshold of each draft row of this step
 *   q_thr   DEVICE fp32, indexed like draft_tokens / q_stats (by draft row)
 *   p_thr   DEVICE [n_target_rows] fp32
 *   p_stats DEVICE [n_target_rows][2] fp32 from svip_row_threshold, or NULL
 *           (then one more pass over the target rows computes them)
 * row_stats / q_stats hold (m, Z) of the truncated distribution.  Other
 * arguments as for svip_draft_step_masked and svip_verify.
 */
int svip_draft_step_filtered(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V,
                             long row_stride, float T, float thresh, const float* uniforms,
                             const uint8_t* active, const float* thr, int32_t* token, float* entropy,
                             uint8_t* stop, float* row_stats, void* stream);
/*
 * svip_row_threshold and svip_draft_step_filtered in one call and one kernel:
 * thr[b] receives the threshold of row b for (top_k, top_p), and token /
 * entropy / stop / row_stats the truncated draft step at it.  With a small
 * top_k (see svip_row_threshold) the kernel finishes the whole step from the
 * few candidates it holds in shared memory, two passes over the row in all;
 * rows it cannot finish that way (nucleus alone, large top_k, many ties at
 * the cut) are streamed once more at the threshold, by the same cluster.
 * Results are those of the two separate calls within the stated tolerances
 * (sums are formed in another order).
 */
int svip_draft_step_truncated(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V,
                              long row_stride, float T, float thresh, int top_k, float top_p,
                              const float* uniforms, const uint8_t* active, float* thr,
                              int32_t* token, float* entropy, uint8_t* stop, float* row_stats,
                              void* stream);
int svip_verify_filtered(svip_ctx* ctx, const int32_t* draft_tokens, const void* q_logits,
                         long q_row_stride, const float* q_stats, const float* q_thr,
                         long q_seq_stride, long q_pos_stride, const void* target_logits,
                         long t_row_stride, const float* p_thr, const float* p_stats,
                         svip_dtype dtype, const int32_t* cu_rows, int B, int K, int n_target_rows,
                         int V, float T, const float* uniforms, int32_t* n_accepted,
                         int32_t* next_token, void* stream);

/*
 * Draft-length policies, kept on the device so that the drafting loop needs no
 * host round trip per token.
 *   SVIP_POLICY_ENTROPY    the paper's rule: a sequence stops drafting when the
 *                          draft step raised its stop flag (Eq. 7; Algorithm 1)
 *   SVIP_POLICY_CONSTANT   baseline 1 of Section 3: exactly gamma[i] tokens
 *   SVIP_POLICY_HEURISTIC  baseline 2 of Section 3: like CONSTANT, and after
 *                          every verification gamma[i] grows by 2 if all draft
 *                          tokens of the round were accepted, else shrinks by 1
 * Every policy also stops at K_cap tokens (the paper caps the length at 40);
 * gamma stays within [1, K_cap].
 *
 * svip_policy_advance, after each draft step: for every sequence with
 * active[i] != 0, draft_len[i] += 1, then active[i] = 0 if the policy says
 * stop.  *n_active (DEVICE int32, may be NULL) receives the number of
 * sequences still drafting.  `stop` is read by ENTROPY only, `gamma` by the
 * other two (either may be NULL when unused).  B <= any size; one thread block.
 *
 * svip_policy_update, after svip_verify: HEURISTIC adapts gamma[i] from
 * n_accepted[i] == draft_len[i]; every policy then resets draft_len[i] = 0
 * and active[i] = 1 for the next round.
 * All arrays DEVICE: stop, active uint8 [B]; gamma, draft_len, n_accepted int32 [B].
 */
typedef enum { SVIP_POLICY_ENTROPY = 0, SVIP_POLICY_CONSTANT = 1, SVIP_POLICY_HEURISTIC = 2 } svip_policy;
int svip_policy_advance(svip_ctx* ctx, int policy, const uint8_t* stop, const int32_t* gamma,
                        int32_t* draft_len, uint8_t* active, int B, int K_cap, int32_t* n_active,
                        void* stream);
int svip_policy_update(svip_ctx* ctx, int policy, const int32_t* n_accepted, int32_t* draft_len,
                       int32_t* gamma, uint8_t* active, int B, int K_cap, void* stream);

/*
 * Ragged packing of per-sequence draft lengths (the per-sequence gamma that
 * Algorithm 1 sets when the stop test fires; batching sequences of different
 * gamma is an addition of this library -- the paper's algorithms handle one
 * sequence).
 *
 *   draft_len   DEVICE [B] int32, K_i in [1, K_max] (else clamped + status bit)
 *   cu_rows     DEVICE [B+1] int32 out: exclusive prefix of (K_i + 1); target row
 *               of (sequence i, position j) is cu_rows[i] + j, draft row of the
 *               packed layout is cu_rows[i] - i + j
 *   row_seq     DEVICE [B*(K_max+1)] int32 out or NULL: sequence of each target row
 *   row_pos     DEVICE [B*(K_max+1)] int32 out or NULL: position of each target row
 *               (entries past the last target row are left untouched)
 * 1 <= B <= 65536, 1 <= K_max, B*(K_max+1) < 2^31.
 */
int svip_pack_ragged(svip_ctx* ctx, const int32_t* draft_len, int B, int K_max,
                     int32_t* cu_rows, int32_t* row_seq, int32_t* row_pos, void* stream);

/*
 * One verification round for B sequences (Algorithm 1, outer-loop body).
 *
 * For sequence i with K_i draft tokens, T > 0: for j = 0..K_i-1 in order,
 * accept while uniforms[cu_rows[i]+j] < p_j(x_j)/q_j(x_j) (Algorithm 2); at
 * the first failure n_accepted[i] = j and next_token[i] is drawn from
 * max(0, p_j - q_j)/sum (Algorithm 4, with the sign that keeps the target
 * distribution) by inverse CDF at uniforms[cu_rows[i]+K_i]; if nothing fails,
 * n_accepted[i] = K_i and next_token[i] ~ p_{K_i} with that same uniform.
 * T == 0: accept while argmax p_j == x_j (Algorithm 3); next_token is the
 * argmax of target row n_accepted (Algorithm 5); uniforms unused (may be NULL).
 * p_j = softmax(target row j / T), q_j = softmax(draft row j / T).
 *
 *   draft_tokens   DEVICE int32, indexed by draft row
 *   q_logits       DEVICE draft logits, draft row r starts at element r*q_row_stride
 *                  (may be NULL when T == 0)
 *   q_stats        DEVICE [draft rows][2] fp32 as written by svip_draft_step with
 *                  the same T, or NULL (then recomputed from q_logits)
 *   q_seq_stride,  draft row of (i, j) = i*q_seq_stride + j*q_pos_stride; or, with
 *   q_pos_stride   q_seq_stride == SVIP_Q_PACKED, cu_rows[i] - i + j (which is
 *                  i*K + j when cu_rows == NULL)
 *   target_logits  DEVICE, target row r starts at element r*t_row_stride
 *   cu_rows        DEVICE [B+1] from svip_pack_ragged, or NULL: every sequence
 *                  has the fixed draft length K
 *   K              the fixed draft length (cu_rows == NULL), else K_max
 *   n_target_rows  total target rows, sum (K_i + 1); the host knows it from the
 *                  target forward.  Must be B*(K+1) when cu_rows == NULL.
 *   uniforms       DEVICE [n_target_rows] fp32 in [0,1), indexed like target rows
 *   n_accepted     DEVICE [B] int32 out, in [0, K_i]
 *   next_token     DEVICE [B] int32 out
 * Needs n_target_rows <= max_rows of svip_create (else SVIP_ERR_WORKSPACE).
 * Probabilities are fp32: where p and q of the rejected position agree to
 * within about 1e-6 in total (a rejection there has that probability), the
 * residual is at rounding level and next_token is only approximately
 * distributed as Algorithm 4 asks.
 */
int svip_verify(svip_ctx* ctx, const int32_t* draft_tokens, const void* q_logits,
                long q_row_stride, const float* q_stats, long q_seq_stride, long q_pos_stride,
                const void* target_logits, long t_row_stride, svip_dtype dtype,
                const int32_t* cu_rows, int B, int K, int n_target_rows, int V, float T,
                const float* uniforms, int32_t* n_accepted, int32_t* next_token, void* stream);

/*
 * svip_verify with the same arguments, results and error behaviour, reading
 * less: the accept tests of a sequence end at its first rejection (Algorithm 1,
 * verify loop), so the target rows after it are never needed.  One group of
 * thread blocks per sequence reads the sequence's target rows in order and
 * stops at the first rejection (or after the bonus row); rows after it are not
 * read.  The rows of one sequence are read one after another, so this pays off
 * where the batch is large enough to fill the GPU with sequences (B of a few
 * dozen and more) and rejections come early; for a few sequences with long
 * accepted runs svip_verify, which reads all rows at once, is faster.
 * Same arithmetic as svip_verify; the rows are cut over another number of
 * thread blocks, so the fp32 normalisers can differ from svip_verify's in
 * their last bits (a result can differ only where a draw lies within fp32
 * rounding of a boundary).  q_stats == NULL costs one more pass over all draft
 * rows first.
 */
int svip_verify_early_exit(svip_ctx* ctx, const int32_t* draft_tokens, const void* q_logits,
                           long q_row_stride, const float* q_stats, long q_seq_stride,
                           long q_pos_stride, const void* target_logits, long t_row_stride,
                           svip_dtype dtype, const int32_t* cu_rows, int B, int K,
                           int n_target_rows, int V, float T, const float* uniforms,
                           int32_t* n_accepted, int32_t* next_token, void* stream);

/*
 * Vocabulary-parallel draft step: the V logits of every row are sharded over G
 * ranks (a tensor-parallel LM head), rank g holding the V_shard columns that
 * start at vocab_offset.  The paper's draft step (Algorithm 1 inner loop, Eq. 7)
 * is unchanged; this is how it is computed when no rank holds a whole row.
 *
 *   1. every rank:  svip_vp_partial  -> partial[B][4] fp32 = (largest logit m,
 *      Z = sum exp((l-m)/T), A = sum exp((l-m)/T)*(l-m)/T in log2 units, global
 *      index of the first maximum as int bits)        (one pass over the shard)
 *   2. the ranks all-gather their partials (16 bytes per row and rank) into
 *      partials[G][B][4], rank-major -- the caller's job (NCCL, any transport)
 *   3. every rank:  svip_vp_combine  -> entropy[B], stop[B] (identical on all
 *      ranks), owner[B] = rank whose shard holds the sampled token (-1 when
 *      greedy), token[B] = the global argmax when T == 0 and -1 otherwise,
 *      local_target[B] and active[B] = (owner == rank) for step 4
 *   4. the owner of a row:  svip_vp_locate  -> token[b] for rows with
 *      active[b] != 0 (others untouched): a second pass over the owner's shard
 *      of that row only, i.e. 1/G of the logits are read twice.  The ranks then
 *      share the tokens (max-reduce of token[], which is -1 where not owned).
 * T == 0 needs steps 1-3 only.  Results equal svip_draft_step on the whole
 * rows within the same tolerances (the shards are reduced in rank order).
 * All pointers DEVICE; partial / partials must be 16-byte aligned.
 */
int svip_vp_partial(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V_shard,
                    long row_stride, float T, int vocab_offset, float* partial, void* stream);
int svip_vp_combine(svip_ctx* ctx, const float* partials, int G, int rank, int B, float T, float thresh,
                    const float* uniforms, float* entropy, uint8_t* stop, int32_t* token,
                    int32_t* owner, float* local_target, uint8_t* active, void* stream);
int svip_vp_locate(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V_shard,
                   long row_stride, float T, const float* local_target, const uint8_t* active,
                   int vocab_offset, int32_t* token, void* stream);

/*
 * The quantities of the paper's analysis for n_pairs (target row, draft row)
 * pairs (Section 2.2: Eq. 1-6; appendix B), with p = softmax(target/T),
 * q = softmax(draft/T), T > 0, all in nats:
 *   out[r][0] beta  = sum_x min(p, q), the expected acceptance probability (Eq. 1)
 *   out[r][1] H_q, the entropy of the draft distribution
 *   out[r][2] H_qp, the cross entropy -sum q ln p
 *   out[r][3] KL(q || p) = H_qp - H_q
 *   out[r][4] gamma = H_qp / H_q
 *   out[r][5] 1 - sqrt(KL / 2), the Pinsker ("oracle") bound (Eq. 3-4)
 *   out[r][6] 1 - sqrt(1 - exp(-KL)), the Bretagnolle-Huber bound (appendix B)
 *   out[r][7] 1 - sqrt(c_bound * H_q), the approximation bound (Eq. 6)
 * Every entry of [5..7] is a lower bound on beta ([7] only when gamma <= 2*c_bound + 1).
 * Pair r reads target row r (element r*t_row_stride) and draft row r (element
 * r*q_row_stride).  `out` is DEVICE [n_pairs][8] fp32.  Where the target masks
 * a token (-inf) that the draft gives mass, KL, H_qp and gamma are +inf.
 * Entropies are fp32 sums, good to about 1e-7 nats.  gamma = H_qp / H_q =
 * 1 + KL / H_q: where H_q comes out as 0 (a draft row that is one-hot to that
 * resolution) gamma is +inf if KL > 0 and 1 if KL is 0 too; no NaN is written.
 * One kernel: both rows are streamed once for the normalisers, the entropy and
 * KL, then once more for beta, which needs the normalisers.
 *
 * svip_pair_stats_given is the same for callers that already hold the rows'
 * normalisers: q_stats / p_stats are DEVICE [n_pairs, 2] (max logit, Z) of the
 * draft / target row of every pair, as svip_draft_step writes its row_stats and
 * svip_row_threshold its stats (with top_k = 0, top_p = 1 for the whole row),
 * at the same T.  Everything then comes out of one pass over the two rows.
 * Both NULL: the call is svip_pair_stats.
 */
int svip_pair_stats(svip_ctx* ctx, const void* q_logits, long q_row_stride, const void* target_logits,
                    long t_row_stride, svip_dtype dtype, int n_pairs, int V, float T, float c_bound,
                    float* out, void* stream);
int svip_pair_stats_given(svip_ctx* ctx, const void* q_logits, long q_row_stride, const float* q_stats,
                          const void* target_logits, long t_row_stride, const float* p_stats, svip_dtype dtype,
                          int n_pairs, int V, float T, float c_bound, float* out, void* stream);

/*
 * Verification of a TREE of draft candidates: several candidates per position,
 * as when the length policy runs on top of a tree drafter (the EAGLE-2 setting
 * of Section 3.3).  The paper states no accept rule for that setting; this is
 * the published multi-candidate generalisation of Algorithms 2 and 4
 * (recursive rejection sampling), under which every emitted token follows the
 * target distribution if the candidates of a node were drawn independently
 * from the node's draft distribution.  At a node with target distribution p,
 * draft distribution q and candidates x_1..x_m (its children, in index order):
 *     p_1 = p;  x_i is accepted if r_i < min(1, p_i(x_i) / q(x_i)),
 *     else p_{i+1} = max(0, p_i - q) / sum max(0, p_i - q);
 * an accepted candidate becomes the current node; when none is accepted, or
 * the node has no child, the next token is drawn from p_{m+1} (from p at a
 * leaf) with the sequence's last draw, and the walk ends.  With one candidate
 * per node the call computes what svip_verify computes.  T == 0: a child is
 * accepted iff its token is the lowest-index argmax of the node's target row,
 * else that argmax is the next token (Algorithms 3 and 5 at every node).
 *
 *   B sequences with N candidate nodes each (N >= 1).
 *   tokens, parent   DEVICE int32 [B, N]: candidate token of node i and its
 *                    parent, -1 for a child of the root, else an index < i.
 *   q_logits, target_logits   DEVICE [B * (N + 1), V] rows (strides in
 *                    elements): row b*(N+1) belongs to the root of sequence b
 *                    (the distributions after the accepted prefix), row
 *                    b*(N+1)+1+i to its node i.  Draft rows of leaves are not
 *                    read by the walk.
 *   q_stats          DEVICE [B * (N + 1), 2] (max logit, Z) of the draft rows
 *                    as svip_draft_step writes them, or NULL (one more pass
 *                    over the draft rows then computes them).  Unused if T == 0.
 *   uniforms         DEVICE [B, N + 1], in [0,1): the accept draw of node i,
 *                    then the draw for the final token.  Unused if T == 0.
 *   n_accepted       DEVICE int32 [B]: length of the accepted path.
 *   path             DEVICE int32 [B, N]: the accepted nodes from the root
 *                    down, then -1.
 *   next_token       DEVICE int32 [B].
 * Needs B * (N + 1) <= max_rows of svip_create.  At most 15 candidates of one
 * node can be rejected; further ones are ignored and SVIP_STATUS_BAD_TREE is
 * set, as for a parent index that is not below its node.  Each rejection costs
 * one pass over the node's two rows (they are read from L2 after the first
 * pass), so the call is bound by the length of that chain, not by bandwidth.
 */
int svip_verify_tree(svip_ctx* ctx, const int32_t* tokens, const int32_t* parent, const void* q_logits,
                     long q_row_stride, const float* q_stats, const void* target_logits, long t_row_stride,
                     svip_dtype dtype, int B, int N, int V, float T, const float* uniforms,
                     int32_t* n_accepted, int32_t* path, int32_t* next_token, void* stream);

/* ---------------------------------------------------------------------------
 * Instrumentation and self-test.  Not part of the method (the paper has no
 * counterpart); benchmarks and tests use these, a serving loop does not.
 * ------------------------------------------------------------------------- */

/*
 * Timing of the row-statistics kernel (the one pass over all target rows inside
 * svip_verify, its dominant kernel) with CUDA events recorded on the caller's
 * stream around that launch.  Benchmarks use it to report the kernel's
 * bandwidth without a profiler.
 *   svip_profile_enable(ctx, 1) creates the events (not inside a graph
 *   capture) and turns recording on; (ctx, 0) turns it off.  While on, every
 *   svip_verify call records one event pair (at most 4096 pairs are kept
 *   between reads; later calls are not recorded).
 *   svip_profile_read synchronises on the recorded events, writes the summed
 *   kernel time in milliseconds and the number of launches it covers (HOST
 *   pointers), and starts a new interval.
 */
int svip_profile_enable(svip_ctx* ctx, int on);
int svip_profile_read(svip_ctx* ctx, double* total_ms, long* launches);

/*
 * Exercises the time-out of the one wait the kernels contain: the blocks of a
 * cluster wait for one another's partial results on an mbarrier, for at most a
 * second; if the time runs out they set SVIP_STATUS_WAIT_TIMEOUT and carry on,
 * so that a lost peer ends in an error status and not in a hang.  This call
 * launches one block that waits, with the same routine, for `wait_ns`
 * nanoseconds (1 .. 10^8) on an mbarrier that nothing completes.  Afterwards
 * svip_read_status reports SVIP_STATUS_WAIT_TIMEOUT and the context works as
 * before.
 */
int svip_selftest_wait_timeout(svip_ctx* ctx, long wait_ns, void* stream);

/*
 * CUDA-graph replay for latency-bound use (small B).  Between begin and end
 * every svip_* call on `stream` is recorded instead of run; svip_graph_end
 * returns an executable graph that svip_graph_launch replays.  All pointers
 * passed while recording must stay valid and are re-read at every replay
 * (refill the logits / uniforms buffers in place between replays).
 * The paper has no counterpart; this serves the B = 1 step latency.
 */
int svip_graph_begin(svip_ctx* ctx, void* stream);
int svip_graph_end(svip_ctx* ctx, void* stream, svip_graph** graph);
int svip_graph_launch(svip_graph* graph, void* stream);
int svip_graph_destroy(svip_graph* graph);

/*
 * The drafting loop of Algorithm 1 ("draft a token, stop when the entropy test
 * fires") as a loop inside the recorded graph, so that one replay drafts a
 * whole round without the host reading a stop flag per token.
 *
 * svip_graph_loop_begin, between svip_graph_begin and svip_graph_end on the
 * same `stream`: everything recorded on `stream` so far runs before the loop,
 * everything recorded on it afterwards runs after the loop.  *body_stream
 * receives a stream owned by the context; every call issued on it (this
 * library's, or the caller's own kernels, e.g. the draft model's forward) until
 * svip_graph_loop_end becomes the loop body.  At replay the body runs once,
 * then again while *n_active > 0 (DEVICE int32, read after the body: the
 * counter that svip_policy_advance writes), and in no case more than
 * `max_iters` times.  If the body holds an svip_policy_advance with this
 * `n_active`, that kernel takes the decision itself; otherwise
 * svip_graph_loop_end appends a one-thread kernel that does.
 * One loop at a time (no nesting); svip_graph_end on a graph whose loop body
 * was not closed, or could not be recorded, returns SVIP_ERR_STATE and hands
 * out no graph.  Calls inside the body must come from the thread that opened
 * it.  The paper has no counterpart beyond the loop of Algorithm 1 itself.
 */
int svip_graph_loop_begin(svip_ctx* ctx, void* stream, const int32_t* n_active, int max_iters,
                          void** body_stream);
int svip_graph_loop_end(svip_ctx* ctx);

/*
 * svip_verify for callers that must not allocate device memory.
 *
 * The paper has no counterpart; this entry point exists for integration.  Some
 * hosts of this library cannot call cudaMalloc where they run the verify
 * round: code executing inside a region where the serving framework has
 * frozen its memory pool (for example while it records or replays a fixed
 * memory plan), plugins that are handed a stream but no allocator, and
 * processes whose device memory is fully pre-partitioned at start-up.  They
 * cannot create an svip_ctx either, because svip_create allocates the
 * workspace.  This call takes no context: its workspace (the per-row
 * normalisers, per-row argmax and the status word of one verify round) is a
 * fixed array that lives in the library's own device image.
 *
 * Same arguments, semantics and results as svip_verify, with these differences
 *   - `device` is the GPU whose memory the pointers refer to; it must be the
 *     calling thread's current device.
 *   - n_target_rows must be <= SVIP_NOALLOC_MAX_ROWS, otherwise the call
 *     returns SVIP_ERR_WORKSPACE and launches nothing.
 *   - `status` (DEVICE, may be NULL) receives the status bits of this call;
 *     the call clears it first.  With NULL the bits are dropped.
 *   - The call never calls cudaMalloc, cudaFree or any allocating routine.
 *     The first call on each device looks up the array's device address and
 *     raises the kernels' shared-memory limit; make that first call outside
 *     any stream capture.
 *   - The array costs about 160 KB of device memory on every GPU that loads
 *     the library, for the life of the process.
 *   - All calls on one device share the array and it keeps the previous
 *     call's contents: calls that overlap on the GPU (different streams, or
 *     the same stream from several threads) race.  Run them one after another
 *     on one stream, or order them with events.
 */
#define SVIP_NOALLOC_MAX_ROWS 8192
int svip_verify_noalloc(int device, const int32_t* draft_tokens, const void* q_logits,
                        long q_row_stride, const float* q_stats, long q_seq_stride,
                        long q_pos_stride, const void* target_logits, long t_row_stride,
                        svip_dtype dtype, const int32_t* cu_rows, int B, int K, int n_target_rows,
                        int V, float T, const float* uniforms, int32_t* n_accepted,
                        int32_t* next_token, unsigned* status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SVIP_H */
