/* disc.h - C ABI of the B200 (sm_100a) DISC + PPV constrained-decoding hot path.
 *
 * The library implements the per-step work of the paper "Efficient and Asymptotically Unbiased
 * Constrained Decoding for Large Language Models" (DISC, Algorithm 1; PPV, Algorithm 2):
 *
 *   disc_build_set   Algorithm 2, line 1 ("Prepare") and Section 3.2 "Array Preparation": sort the
 *                    members of S lexicographically by token id and keep the array on the GPU.
 *   disc_mask        Algorithm 2, lines 3-7 with M = |V|: the mask of the valid set A_{a,S}
 *                    (Section 2.1) of a prefix a.
 *   disc_verify      Algorithm 2, lines 4-6 as stated: M candidate tokens per prefix verified by
 *                    binary search in the sorted array (top-M mode).
 *   disc_topm        Algorithm 2, line 3: the M most probable tokens of every row.
 *   disc_step_topm   Algorithm 1, lines 5-8 with the mask of Algorithm 2 as the paper runs it: the
 *                    top-M tokens are verified against the sorted array and the token is drawn
 *                    among the verified ones.
 *   disc_step        Algorithm 1, lines 5-8 for a batch of partial sequences: mask, sample from
 *                    P.mask/|P.mask|_1, append, multiply the importance score by |P.mask|_1.
 *   disc_project_step  the same step with line 5's P = L(a, T) folded in: the model's last projection
 *                    (hidden vectors times the vocabulary matrix) runs on the tensor cores and
 *                    only the pieces of the logits the step looks at ever reach memory.
 *   disc_resample    Algorithm 1, line 22: among K finished candidates pick one with probability
 *                    x_k / sum_j x_j.
 *   disc_accept      Algorithm 1, line 16: accept a candidate when x > eps ~ U[0,1].
 *   disc_accept_resample  Algorithm 1, lines 11-22: K ordered accept tests, then the K-way draw
 *                    over K fresh candidates.
 *
 * Conventions
 *   - Every function returns 0 (DISC_OK) or a negative DISC_ERR_* code.  Return codes cover
 *     argument validation and CUDA launch/allocation errors only; problems of a single row are
 *     reported in that row's status byte and never fail the call.
 *   - "host" pointers are ordinary CPU memory, "device" pointers are memory of the current CUDA
 *     device, owned by the caller.  `stream` is a cudaStream_t (NULL = the default stream).
 *     A handle belongs to the device that was current when it was built; calls that take a
 *     handle return DISC_ERR_ARG when another device is current.
 *   - Except for disc_build_set / disc_free_set / disc_set_info / disc_set_rows, calls only enqueue
 *     kernels on `stream`: they allocate nothing, do not synchronise the host, and finish in
 *     stream order.
 *   - The importance score x of Algorithm 1 is kept as its logarithm `logw` in fp32 (x starts at 1,
 *     logw at 0; each step adds log |P.mask|_1).
 *   - The set must be prefix-free (all members of one length, or every member closed by an
 *     end-of-sequence token that is an ordinary token): "a in S" (Algorithm 1, line 4) is then
 *     "a's node has no child".
 *   - Mask layout: W = ceil(V/32) uint32 words per row; token v is bit (v & 31) of word (v >> 5);
 *     bits at positions >= V are zero.
 *   - Random numbers: Philox4x32-10, key = (seed low 32 bits, seed high 32 bits).  The uniform of
 *     output word r is u = ((r >> 9) + 0.5) * 2^-23 (u and 1-u exact in fp32).  Counters:
 *       group noise  (((G>>10)<<8) | (G&255), step, row, 0), word (G>>8)&3   per token group G
 *       in-group     (G, step, row, 3), word 0
 *       resample     (query, 0, 0, 1), word 0
 *       accept       (query, k, 0, 2), word 0
 *     where `row` / `query` is row_base / query_base plus the index inside the call.  Each is one
 *     32-bit counter word: row_base + n and query_base + B must not exceed 2^32
 *     (DISC_ERR_UNSUPPORTED otherwise).
 *   - Sampling draws exactly from P.mask/|P.mask|_1 in two stages.  Tokens are taken in groups of
 *     8 consecutive ids (G = v >> 3).  Stage 1 is Gumbel-max over groups: the group maximising
 *     log(sum of e^{z_v/T} over its allowed tokens) - log(-log u_G) wins (the lowest G on an exact
 *     tie); it is therefore chosen with probability proportional to its allowed mass.  Stage 2
 *     picks, inside the winner, the smallest allowed token whose inclusive cumulative weight
 *     exceeds u' * mass (tokens in ascending id).
 */
#ifndef DISC_H_
#define DISC_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DISC_OK 0
#define DISC_ERR_ARG (-1)         /* null, negative, out-of-range or misaligned argument          */
#define DISC_ERR_EMPTY (-2)       /* empty set or empty member                                    */
#define DISC_ERR_TOKEN (-3)       /* token id outside [0, vocab_size)                             */
#define DISC_ERR_PREFIX (-4)      /* a member is a proper prefix of another member                */
#define DISC_ERR_OOM (-5)         /* device or host allocation failed                             */
#define DISC_ERR_CUDA (-6)        /* a CUDA call failed; see disc_last_cuda_error()               */
#define DISC_ERR_UNSUPPORTED (-7) /* size or dtype outside what the kernels support               */

/* per-row status bits */
#define DISC_ROW_DEAD 1     /* prefix / node is not a prefix of any member                        */
#define DISC_ROW_NOMASS 2   /* allowed probability mass is zero or not finite                     */
#define DISC_ROW_NONFINITE 4 /* NaN or +Inf among the row's logits (or NaN among the weights)     */
#define DISC_ROW_DONE 8     /* row was already complete: nothing read, state untouched            */
#define DISC_ROW_FAULT 16   /* reserved for kernels that wait inside the device; no present kernel sets it
                               (disc_project_step reports a wait that ran out through
                               disc_project_error instead)                                        */

typedef struct disc_set disc_set_t; /* opaque; owns its device memory */

typedef enum { DISC_F32 = 0, DISC_BF16 = 1 } disc_dtype_t;

#define DISC_MAX_DEPTH 64

typedef struct {
    int64_t n_members;       /* N: members after de-duplication                                  */
    int64_t n_entries;       /* E: int32 entries of the sorted table                             */
    int64_t n_nodes;         /* distinct non-empty prefixes of members (index nodes)             */
    int32_t vocab_size;      /* V                                                                */
    int32_t mask_words;      /* W = ceil(V/32)                                                   */
    int32_t l_max;           /* longest member                                                   */
    int32_t n_heavy;         /* nodes with more than 1024 children (their masks are prebuilt)    */
    int64_t device_bytes;    /* device memory held by the handle                                 */
    double build_seconds;    /* wall time of disc_build_set                                      */
    int64_t level_nodes[DISC_MAX_DEPTH]; /* distinct prefixes of length d+1, d = 0..l_max-1      */
} disc_set_info_t;

/* Build the device-resident constraint array (Algorithm 2, line 1; Section 3.2 "Array
 * Preparation").
 *   tokens       host, int32[row_offsets[n_rows]]: the members back to back, in any order
 *   row_offsets  host, int64[n_rows+1]: member r is tokens[row_offsets[r] .. row_offsets[r+1])
 *   vocab_size   V; every token must lie in [0, V)
 *   flags        must be 0
 *   stream       stream the build kernels run on; the call synchronises it before returning
 *   out          receives the handle (NULL on error)
 * The inputs are copied.  Members are sorted lexicographically by token id (a shorter sequence
 * before its extensions), duplicates are collapsed.  Besides the sorted table the handle holds an
 * index with one node per distinct non-empty prefix, level by level, from which the valid set of
 * any prefix is read as a contiguous list.
 * Errors: DISC_ERR_ARG, DISC_ERR_EMPTY (no member / an empty member), DISC_ERR_TOKEN,
 * DISC_ERR_PREFIX, DISC_ERR_UNSUPPORTED (n_rows >= 2^31, entries >= 2^32, member longer than
 * DISC_MAX_DEPTH, V > 4,000,000), DISC_ERR_OOM, DISC_ERR_CUDA. */
int disc_build_set(const int32_t* tokens, const int64_t* row_offsets, int64_t n_rows,
                   int32_t vocab_size, uint32_t flags, void* stream, disc_set_t** out);

/* The same build for sets in which a member may be a proper prefix of another member (Section 2.1
 * lets the model stop at a member by emitting an end-of-keyword token there).  Every member is
 * closed by eok_token (on a host copy; the caller's arrays are not changed), which makes the set
 * prefix-free, and disc_build_set follows.  Afterwards the valid set of a prefix that is itself a
 * member contains eok_token next to the tokens that extend it, and a candidate is complete once
 * it has produced eok_token; sequences returned by disc_step / disc_resample end with it.
 *   eok_token   in [0, vocab_size); must not occur inside any member (DISC_ERR_TOKEN otherwise)
 * The longest member may have DISC_MAX_DEPTH - 1 tokens.  Other arguments and errors as for
 * disc_build_set (DISC_ERR_PREFIX cannot occur). */
int disc_build_set_eok(const int32_t* tokens, const int64_t* row_offsets, int64_t n_rows,
                       int32_t vocab_size, int32_t eok_token, void* stream, disc_set_t** out);

/* Release the handle and its device memory.  NULL is allowed. */
void disc_free_set(disc_set_t* s);

/* Sizes of the built set.  `info` is host memory. */
int disc_set_info(const disc_set_t* s, disc_set_info_t* info);

/* Copy the sorted, de-duplicated table back (the array X of Algorithm 2, without padding).
 *   tokens_out       host, int32[n_entries]
 *   row_offsets_out  host, int64[n_members+1]
 * Synchronises the device. */
int disc_set_rows(const disc_set_t* s, int32_t* tokens_out, int64_t* row_offsets_out);

/* Start n candidates at the empty sequence (Algorithm 1, line 3: a = [], x = 1).
 * All arrays are device memory with n entries: node = root, [lo, hi) = [0, N), depth = 0,
 * logw = 0, done = 0. */
int disc_state_init(const disc_set_t* s, int64_t n, int32_t* node, int32_t* lo, int32_t* hi,
                    int32_t* depth, float* logw, uint8_t* done, void* stream);

/* Valid-set masks of n prefixes (Algorithm 2, lines 3-7 in the M = |V| limit; Section 2.1).
 *   prefix      device, int32[n][prefix_ld]; row i holds prefix_len[i] tokens
 *   prefix_len  device, int32[n], 0 <= prefix_len[i] <= prefix_ld
 *   mask_out    device, uint32[n][W] (nullable): bit v set iff prefix+[v] is a prefix of a member
 *   lo_out, hi_out  device, int32[n] (nullable): the members having the prefix are rows [lo, hi)
 *               of the sorted table
 *   node_out    device, int32[n] (nullable): index node of the prefix (the cursor disc_step uses)
 *   status_out  device, uint8[n]: 0, or DISC_ROW_DEAD when the prefix is a prefix of no member
 *               (then the mask is zero and lo = hi = node = -1)
 * A complete member has an empty mask and a range of one row.
 * With mask_out given, the call keeps a row counter in the set handle: two such calls on the
 * same handle must not run on the device at the same time (calls issued to one stream never do;
 * calls on different streams need an event between them, or a handle each).  n must be below
 * 2^31 - 2^20 (DISC_ERR_UNSUPPORTED otherwise). */
int disc_mask(const disc_set_t* s, const int32_t* prefix, int32_t prefix_ld,
              const int32_t* prefix_len, int64_t n, uint32_t* mask_out, int32_t* lo_out,
              int32_t* hi_out, int32_t* node_out, uint8_t* status_out, void* stream);

/* disc_mask with the writer's row counter in a fixed word block inside the loaded module (a
 * file-scope device array of 256 bytes per device) instead of device memory obtained from the
 * allocator.  The paper has no counterpart of this entry point; it exists for callers that cannot
 * let a library allocate device memory on their behalf: a serving process that sizes its own pool
 * to all of the memory left at start-up has no room to give later, and an allocation made behind
 * its back can fail or push it over its budget.  This call performs no allocation and frees
 * nothing, on the device or through the CUDA allocator.
 * Arguments, outputs and errors are those of disc_mask.  In addition:
 *   - n must not exceed DISC_MASK_STATIC_MAX_ROWS; a larger n is refused with DISC_ERR_UNSUPPORTED
 *     before anything is launched;
 *   - the first call on a device looks up the address of the word block (with that device
 *     current) and keeps it; make that first call outside any stream capture;
 *   - the block is shared by every call on that device, whatever the handle or stream: two calls
 *     must not run on the device at the same time (calls on one stream never do).  Nothing has to be
 *     cleared between calls: the first kernel of each call resets the counter, and what an earlier
 *     call left there is never read. */
#define DISC_MASK_STATIC_MAX_ROWS 1073741824 /* 2^30 prefixes per call */
int disc_mask_static(const disc_set_t* s, const int32_t* prefix, int32_t prefix_ld,
                     const int32_t* prefix_len, int64_t n, uint32_t* mask_out, int32_t* lo_out,
                     int32_t* hi_out, int32_t* node_out, uint8_t* status_out, void* stream);

/* Algorithm 2 as stated (lines 4-6; Section 3.2 "Parallel Verification"): for each of n partial
 * sequences a and each of its M candidate tokens t_m, find by binary search in the sorted member
 * array X the smallest row that is not lexicographically smaller than V_m = a + [t_m]; t_m is
 * valid iff V_m is a prefix of that row.  Only the sorted table is read, not the prefix index.
 *   prefix, prefix_ld, prefix_len   as for disc_mask (0 <= prefix_len[i] <= prefix_ld, at most
 *               DISC_MAX_DEPTH; a prefix outside that gets the empty range [0, 0))
 *   cand        device, int32[n][M]: the candidates (for instance the top-M tokens of P); ids
 *               outside [0, V) are invalid
 *   valid_out   device, uint8[n][M]: mask_V of Algorithm 2, line 5
 *   row_out     device, int32[n][M] (nullable): the row index the search lands on (N when every
 *               row is smaller)
 *   mask_out    device, uint32[n][W] (nullable): line 6, bit t_m set iff t_m is valid, all other
 *               bits zero; with every token among the candidates this is disc_mask's mask
 *   lo_out, hi_out  device, int32[n] (required): the rows having a as a prefix are [lo, hi) (empty
 *               range with lo = hi = insertion point when there is none)
 * M = 0 computes the ranges only.  Errors: DISC_ERR_ARG; DISC_ERR_UNSUPPORTED when n*M >= 2^38. */
int disc_verify(const disc_set_t* s, const int32_t* prefix, int32_t prefix_ld, const int32_t* prefix_len,
                int64_t n, const int32_t* cand, int32_t M, uint8_t* valid_out, int32_t* row_out,
                uint32_t* mask_out, int32_t* lo_out, int32_t* hi_out, void* stream);

/* One decoding step for n candidates (Algorithm 1, lines 5-8; score closed form in Appendix A).
 *   logits   device, n rows of V values of type `dtype`, row i at element offset i*ld.  The fast
 *            path needs the base 16-byte aligned and ld*sizeof(value) a multiple of 16; other
 *            layouts take a slower scalar path.  Pinned (page-locked, device-accessible) host
 *            memory is accepted as well: the kernel then reads it in place over PCIe, and rows
 *            that are already complete are not read at all.
 *   inv_temperature  1/T (Algorithm 1's T), finite and > 0
 *   seed, step, row_base  random-number coordinates (see top of file); `step` must differ between
 *            the steps of one decode
 *   node, lo, hi, depth, logw, done   device, in/out state, n entries each
 *   token_out   device, int32[n]: sampled token, -1 for rows that did nothing
 *   seq_tokens  device, int32[n][seq_ld] (nullable): the token is also stored at
 *            seq_tokens[i][depth[i]] (depth before the step) when depth[i] < seq_ld
 *   logq_out    device, float[n] (nullable): log-probability of the token under the masked,
 *            renormalised distribution
 *   logp_out    device, float[n] (nullable): its log-probability under the unmasked distribution
 *   mask_out    device, uint32[n][W] (nullable): the valid-set mask used by each live row
 *   status_out  device, uint8[n]
 * Per live row: z_v = logit_v / T; lse_all = log sum_v e^{z_v}; lse_ok = the same over the valid
 * set; logw += lse_ok - lse_all; token drawn from the valid set (two-stage rule at the top of this
 * file); the state moves to the extended prefix; done is set when the extended prefix is a member.
 * Rows with done != 0 are skipped (status DISC_ROW_DONE, token -1, no logits read).  A row whose
 * valid mass is zero keeps going with the lowest valid token (status DISC_ROW_NOMASS,
 * logw = -inf); NaN/+Inf logits give status DISC_ROW_NONFINITE, a NaN/Inf logw and some valid
 * token (which one is unspecified). */
int disc_step(const disc_set_t* s, const void* logits, disc_dtype_t dtype, int64_t ld, int64_t n,
              float inv_temperature, uint64_t seed, uint32_t step, int64_t row_base,
              int32_t* node, int32_t* lo, int32_t* hi, int32_t* depth, float* logw, uint8_t* done,
              int32_t* token_out, int32_t* seq_tokens, int32_t seq_ld, float* logq_out,
              float* logp_out, uint32_t* mask_out, uint8_t* status_out, void* stream);

/* Algorithm 2, line 3: the M tokens of largest logit of each of n rows (the M most probable ones).
 * Equal logits (-0 and +0 are equal) are ordered by token id, the lower id first; NaN logits come
 * last.  The selection is exact for every input.
 *   logits, dtype, ld   as for disc_step (device memory; rows of vocab_size values)
 *   done        device, uint8[n] (nullable): rows with done != 0 are skipped (candidates -1)
 *   cand_out    device, int32[n][M]: the selected token ids in ascending order, -1 padded when
 *               M > vocab_size
 *   lse_out     device, float[n][2] (nullable): the pair (m, s) with
 *               sum_v 2^(logit_v * log2(e) * inv_temperature) = 2^m * s, a by-product of the passes
 *               over the row (inv_temperature is used for this output only)
 * Errors: DISC_ERR_ARG, DISC_ERR_UNSUPPORTED (dtype; n >= 2^31). */
int disc_topm(const void* logits, disc_dtype_t dtype, int64_t ld, int64_t n, int32_t vocab_size, int32_t M,
              float inv_temperature, const uint8_t* done, int32_t* cand_out, float* lse_out, void* stream);

/* One decoding step in the paper's top-M mode (Algorithm 1, lines 5-8, with mask = PPV_S(P, a) computed
 * as Algorithm 2 states it: line 3 selects the M most probable tokens, lines 4-5 verify each
 * a + [t_m] by binary search in the sorted array, line 6 is the mask of the verified ones).  The
 * token is drawn among the verified candidates by disc_step's two-stage rule, the importance
 * log-weight grows by the log of their probability mass.  With M = |V| the result is disc_step's.
 * A row none of whose candidates is valid has reached a dead end: it would fail Algorithm 1's test
 * "a in S" (line 15), so it ends here with status DISC_ROW_DEAD, token -1, done = 1 and
 * logw = -inf (the K-way draw then never picks it).
 *   M           1 <= M <= 1024
 *   seq_tokens  device, int32[n][seq_ld], required, seq_ld >= l_max: the tokens produced so far
 *               (the prefix a of every row, which the verification searches for); the new token
 *               is appended as in disc_step
 *   cand_out    device, int32[n][M]: receives the candidates (ascending id)
 *   scratch     device, disc_step_topm_scratch_bytes(n, M) bytes, 8-byte aligned, caller-owned
 *   other arguments as for disc_step (mask_out receives the mask of the verified candidates)
 * Four kernels are enqueued on `stream` (selection, prefix ranges and candidate verification, step). */
int64_t disc_step_topm_scratch_bytes(int64_t n, int32_t M);
int disc_step_topm(const disc_set_t* s, const void* logits, disc_dtype_t dtype, int64_t ld, int64_t n, int32_t M,
                   float inv_temperature, uint64_t seed, uint32_t step, int64_t row_base, int32_t* node, int32_t* lo,
                   int32_t* hi, int32_t* depth, float* logw, uint8_t* done, int32_t* token_out, int32_t* seq_tokens,
                   int32_t seq_ld, float* logq_out, float* logp_out, uint32_t* mask_out, uint8_t* status_out,
                   int32_t* cand_out, void* scratch, int64_t scratch_bytes, void* stream);

/* One decoding step with the language model's last projection fused in (Algorithm 1, lines 5-8,
 * where line 5's next-token distribution is softmax(h W / T) of the model's final hidden vectors).
 *   logit[i][v] = bf16( sum_k hidden[i][k] * wt[v][k] )       (fp32 accumulation, rounded once to
 * bf16: the value a separate projection would have stored), then exactly disc_step on those logits.
 * The projection runs on the tensor cores; per row it keeps the sums the log-sum-exp over the
 * whole vocabulary needs, and writes logits only for the 256-wide vocabulary tiles that hold a
 * valid next token of the row (all tiles for a row at the empty prefix or at a node with more than
 * 1024 children), so that for the typical row deep in the prefix tree 512 bytes instead of 2V reach
 * memory.
 *   hidden      device, bf16[n][hidden_ld], d values used per row
 *   wt          device, bf16[V][wt_ld], d values used per row: the vocabulary projection, one
 *               vocabulary entry per row
 *   d           model width; a multiple of 8.  hidden, wt, logits_buf and scratch must be 16-byte
 *               aligned and the row pitches multiples of 16 bytes (DISC_ERR_ARG /
 *               DISC_ERR_UNSUPPORTED otherwise)
 *   inv_temperature, seed, step, row_base, state arrays, token_out, seq_tokens, seq_ld, logq_out,
 *   logp_out, status_out      as for disc_step
 *   logits_buf  device, bf16[n][logits_ld], logits_ld >= V: receives the logits pieces; with
 *               store_all != 0 every logit is written (the complete matrix a separate projection
 *               would have produced: for tests and diagnostics), otherwise what is not written
 *               keeps its old contents
 *   scratch     device, disc_project_scratch_bytes(s, n) bytes, caller-owned; its first word is an
 *               error flag the call clears and the kernel sets when one of its bounded waits ran
 *               out (read it with disc_project_error)
 * Rows with NaN or +-Inf logits get DISC_ROW_NONFINITE / DISC_ROW_NOMASS as in disc_step; their
 * log-weights are not finite but need not equal disc_step's bit for bit.
 * Three kernels are enqueued on `stream` (tile flags, projection, step); nothing is allocated. */
int64_t disc_project_scratch_bytes(const disc_set_t* s, int64_t n);
int disc_project_step(const disc_set_t* s, const void* hidden, int64_t hidden_ld, const void* wt, int64_t wt_ld,
                      int32_t d, int64_t n, float inv_temperature, uint64_t seed, uint32_t step, int64_t row_base,
                      int32_t* node, int32_t* lo, int32_t* hi, int32_t* depth, float* logw, uint8_t* done,
                      int32_t* token_out, int32_t* seq_tokens, int32_t seq_ld, float* logq_out, float* logp_out,
                      uint8_t* status_out, void* logits_buf, int64_t logits_ld, int32_t store_all, void* scratch,
                      int64_t scratch_bytes, void* stream);

/* Synchronises `stream` and returns DISC_ERR_CUDA when the projection kernel of an earlier
 * disc_project_step with this scratch buffer gave up on one of its waits (its results are then
 * invalid), DISC_OK otherwise. */
int disc_project_error(const void* scratch, void* stream);

/* K-way importance draw (Algorithm 1, line 22; Appendix A).
 *   logw        device, float[B][K]: log importance scores of the K candidates of each query
 *   idx_out     device, int32[B]: chosen candidate, P(k) = x_k / sum_j x_j
 *   logz_out    device, float[B] (nullable): log((1/K) sum_k x_k), an estimate of log P_L(S)
 *   seq_tokens  device, int32[B][K][seq_ld] (nullable) and tokens_out device int32[B][seq_ld]
 *               (nullable): when both are given the chosen candidate's tokens are copied out
 *   status_out  device, uint8[B]: DISC_ROW_NOMASS when no candidate has a finite positive weight
 *               (the pick is then uniform), DISC_ROW_NONFINITE when a weight is NaN (it counts as 0)
 * The pick is the smallest k whose inclusive prefix sum of weights exceeds u * total. */
int disc_resample(const float* logw, int32_t B, int32_t K, uint64_t seed, int64_t query_base,
                  int32_t* idx_out, float* logz_out, const int32_t* seq_tokens, int32_t seq_ld,
                  int32_t* tokens_out, uint8_t* status_out, void* stream);

/* Accept test over K finished candidates per query, in order (Algorithm 1, lines 12-21):
 *   first_out   device, int32[B]: smallest k with logw[b][k] > log(eps_{b,k}), eps uniform in
 *               (0,1); -1 when all K candidates are rejected (the caller then falls back to
 *               disc_resample on K fresh candidates). */
int disc_accept(const float* logw, int32_t B, int32_t K, uint64_t seed, int64_t query_base,
                int32_t* first_out, void* stream);

/* Algorithm 1, lines 11-22 for B queries with 2K finished candidates each: candidates 0..K-1 are
 * put to the accept test in order (line 16, as disc_accept); the first accepted one is returned;
 * when all K are rejected, one of the fresh candidates K..2K-1 is drawn with probability
 * x_k / sum_j x_j (line 22, as disc_resample over those K).  The output then follows
 * (1 - p_b^K) P_S + p_b^K Q_K (Appendix A), p_b = 1 - P_L(S).
 *   logw        device, float[B][2K]
 *   choice_out  device, int32[B]: the candidate returned, in [0, 2K)
 *   first_out   device, int32[B] (nullable): the accepted candidate, or -1 after K rejections
 *   logz_out    device, float[B] (nullable): log((1/K) sum x) over the fresh candidates
 *   seq_tokens  device, int32[B][2K][seq_ld] (nullable) with tokens_out int32[B][seq_ld] (nullable):
 *               the returned candidate's tokens are copied out
 *   status_out  device, uint8[B]: status of the K-way draw over the fresh candidates (see
 *               disc_resample); it matters only where first_out is -1
 * Random numbers: those of disc_accept and disc_resample for the same seed and query. */
int disc_accept_resample(const float* logw, int32_t B, int32_t K, uint64_t seed, int64_t query_base,
                         int32_t* choice_out, int32_t* first_out, float* logz_out,
                         const int32_t* seq_tokens, int32_t seq_ld, int32_t* tokens_out,
                         uint8_t* status_out, void* stream);

/* Diagnostic: the n group-noise uniforms of token groups g0 .. g0+n-1 for (seed, step, row), fp32.
 *   out  device, float[n] */
int disc_sampling_uniforms(uint64_t seed, uint32_t step, uint32_t row, int32_t g0, int32_t n,
                           float* out, void* stream);

/* Text for a DISC_ERR_* code. */
const char* disc_error_string(int code);

/* cudaError_t (as int) of the most recent failed CUDA call made by this library on this thread. */
int disc_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* DISC_H_ */
