/*
 * sam.h - C ABI of the B200 (sm_100a) suffix-automaton draft + greedy-verify library.
 *
 * The operations are those of the AgentSAM speculative decoding loop (Section 5.4.2
 * "Algorithm design", Section 5.4.3 "System design", Algorithm 3):
 *   build the automaton over the context memory once (setup),
 *   per decoding step: follow automaton transitions over the newly verified tokens and
 *   emit a continuation of bounded length (draft), let the target model score the proposal
 *   (its logits are an INPUT here), take the row-wise greedy choice, commit the longest
 *   matching prefix plus the model's own token at the first mismatch (verify), and feed the
 *   committed tokens straight back into the automaton walk (step).
 *
 * General rules
 *   - Every function returns an int status: SAM_OK (0) or a negative SAM_ERR_* code.
 *     Nothing throws, aborts or traps; device code never faults on out-of-vocabulary tokens.
 *   - "host" pointers are ordinary CPU memory; "device" pointers are CUDA device memory of
 *     the current device, allocated and owned by the caller (e.g. torch tensors).
 *   - Hot-path calls (sam_draft, sam_verify, sam_step) only enqueue kernels on the given
 *     stream (a cudaStream_t passed as void*, NULL = default stream).  They never allocate,
 *     never synchronise and never copy to the host; outputs are valid once the stream reaches
 *     the end of the enqueued work.
 *   - Token ids are int32.  The per-stream state is the pair (state, matched_len), owned by
 *     the caller; a new stream starts at (0, 0).
 *   - There is no CPU fallback: without a usable CUDA device the hot-path calls fail with
 *     SAM_ERR_CUDA.
 *   - Calls may come from several host threads at once, on different streams, as long as they share
 *     neither scratch nor output buffers (one handle may serve them all: hot-path calls only read it).
 *     The diagnostic switches (sam_profile_*, sam_set_argmax_variant) are process-wide and not for
 *     concurrent use.
 *   - sam_step / sam_step_ex may be recorded in a CUDA graph by stream capture and replayed (tested:
 *     the replayed step gives the oracle's trace).  Make one ordinary call on the device first (it
 *     does the library's first-use set-up); the recorded launches keep the pointers, sizes and
 *     options of the recorded call, and replays share its scratch, so they must not overlap.
 */
#ifndef SAM_B200_H
#define SAM_B200_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SAM_OK                 0
#define SAM_ERR_INVALID_ARG   (-1)  /* null pointer, size out of range, misaligned pointer */
#define SAM_ERR_NOMEM         (-2)  /* host allocation failed during sam_build */
#define SAM_ERR_NOT_UPLOADED  (-3)  /* hot-path call before a successful sam_upload */
#define SAM_ERR_CUDA          (-4)  /* a CUDA runtime call or kernel launch failed; see sam_last_cuda_error */
#define SAM_ERR_TOO_SMALL     (-5)  /* caller buffer (device blob, workspace) smaller than required */

#define SAM_ERR_TOO_LARGE     (-6)  /* size beyond a built-in limit of the called entry point */

#define SAM_K_MAX             32    /* largest draft length K accepted by the hot path */
#define SAM_MAX_SEPARATORS    16    /* largest number of separator ids */

typedef struct sam_index sam_index; /* opaque; owns the host-side automaton; device memory belongs to the caller */

/* ---------------------------------------------------------------- setup (host, blocking) */

/* Builds the suffix automaton of corpus[0..n) by the online, token-by-token construction
 * (Section 5.4.3: incremental, linear in the context length).  States are numbered in
 * creation order: root 0, then for each position the new state followed by its clone when a
 * split happens; a clone copies transitions, suffix link and first end position.
 * Separators are ordinary symbols for construction and for the walk; they only stop draft
 * emission and are never emitted.
 *   corpus      host, n int32 tokens, 1 <= n <= 2^29, every id in [0, 2^24) (the dense root table and the
 *               hashed rows of the device layout are sized for 24-bit ids; other ids are refused here,
 *               while the hot path itself takes any int32 and treats unknown ids as having no transition)
 *   separators  host, n_sep ids (0 <= n_sep <= SAM_MAX_SEPARATORS); may be NULL when n_sep = 0
 *   out         receives the handle; release it with sam_free
 * Errors: SAM_ERR_INVALID_ARG (also: a token id outside [0, 2^24)), SAM_ERR_NOMEM, SAM_ERR_TOO_LARGE (the
 * transitions of states with three or more successors do not fit 2^31 - 1 edge slots). */
int sam_build(const int32_t* corpus, int64_t n, const int32_t* separators, int32_t n_sep,
              sam_index** out);

/* Sizes of the built automaton and the byte size of the device blob sam_upload needs.
 * Any output pointer may be NULL. */
int sam_sizes(const sam_index* idx, int64_t* n_states, int64_t* n_edges, int64_t* device_bytes);

/* Copies the automaton as flat host arrays (for inspection and parity checks):
 *   len, link, firstpos  [n_states] int32  (root: 0, -1, -1; firstpos = smallest end position)
 *   row_ptr              [n_states + 1] int64, CSR offsets into the edge arrays
 *   edge_tok, edge_dst   [n_edges] int32, each row strictly ascending by token id
 * All six are host buffers owned by the caller; any may be NULL to skip it. */
int sam_export(const sam_index* idx, int32_t* len, int32_t* link, int32_t* firstpos,
               int64_t* row_ptr, int32_t* edge_tok, int32_t* edge_dst);

/* Packs the automaton and the corpus into the device layout and copies it into device_buf
 * (device, 256-byte aligned, at least device_bytes from sam_sizes) with cudaMemcpyAsync on the
 * stream, then synchronises that stream once (setup, not the hot path).  The handle remembers
 * device_buf; the caller keeps it alive and unmodified while hot-path calls use the handle.
 * Errors: SAM_ERR_INVALID_ARG, SAM_ERR_TOO_SMALL, SAM_ERR_CUDA, SAM_ERR_NOMEM. */
int sam_upload(sam_index* idx, void* device_buf, int64_t bytes, void* cuda_stream);

/* Releases the host-side automaton.  Device memory is the caller's. NULL is allowed. */
void sam_free(sam_index* idx);

/* ---------------------------------------------------------------- verification scratch */

/* Bytes of device scratch sam_verify / sam_step need for B streams and draft length K
 * (one 64-bit partial result per logits row, the walk-ahead states of every draft position, one
 * completion counter per stream and per row, a row list with its bookkeeping words and a status word).
 * Returns a negative SAM_ERR_* on bad sizes. */
int64_t sam_workspace_bytes(int32_t B, int32_t K);

/* Zero-fills the scratch (device, 8-byte aligned) on the stream.  Required once before the
 * first sam_verify / sam_step that uses it; every successful call leaves it ready for the next one
 * (not all zero: a row list for the next step and a count of launches may stay in it).
 * Call it again after a hot-path call returned an error.  Calls that share one workspace
 * must not overlap on the device. */
int sam_workspace_init(void* workspace, int64_t bytes, void* cuda_stream);

/* Reads the status word the verification kernels keep inside the scratch: 0 = fine,
 * 1 = a kernel gave up on one of its internal (bounded) waits, 2 = a kernel was handed more
 * finished streams than its internal queue holds (the host sizes the launch so that this does not
 * happen), 3 = SAM_STEP_ROW_LIST_READY was given but the scratch holds no row list for this batch shape.  After a non-zero status the outputs of that call are not valid - re-initialise the
 * scratch and retry.  Copies one int to the host and synchronises the stream: a diagnostic, not a
 * hot-path call.  B and K locate the word (same values as in the calls that used the scratch). */
int sam_workspace_status(const void* workspace, int32_t B, int32_t K, int32_t* status_out, void* cuda_stream);

/* ---------------------------------------------------------------- hot path (device, async) */

/* Draft (Section 5.4.2; Algorithm 3 "FollowTransitions" and "Emit speculative tokens").
 * For every stream b: consume new_tokens[b, 0..n_new[b]) from (state[b], matched_len[b]):
 * a transition on the token extends the match by one; on a miss the suffix link is followed
 * and the match shortened to that state's length, and a miss at the root resets the match to 0.
 * Then, if matched_len[b] >= min_match, emit the tokens that follow the FIRST occurrence of
 * the matched suffix in the corpus: up to K tokens, stopping before a separator or the corpus
 * end; otherwise emit nothing.
 *   B            streams, >= 0 (0 is a no-op)
 *   state, matched_len   device [B] int32, in/out
 *   new_tokens   device [B, ld] int32 row-major; n_new device [B] int32 with 0 <= n_new[b] <= ld
 *                (values above ld are clamped to ld, negative to 0); n_new[b] = 0 re-emits the draft
 *   K            1..SAM_K_MAX;  min_match >= 1
 *   drafts       device [B, K] int32, unused slots = -1;  n_draft device [B] int32
 * Errors: SAM_ERR_INVALID_ARG, SAM_ERR_NOT_UPLOADED, SAM_ERR_CUDA. */
int sam_draft(const sam_index* idx, int32_t B, int32_t* state, int32_t* matched_len,
              const int32_t* new_tokens, int32_t ld, const int32_t* n_new,
              int32_t K, int32_t min_match, int32_t* drafts, int32_t* n_draft,
              void* cuda_stream);

/* Greedy verification (Algorithm 3 "Validate with main LLM; commit matched prefix; fallback").
 * logits row (b, j), j = 0..K, holds the target model's scores after the committed tokens and
 * drafts[b, 0..j).  For all B*(K+1) rows: argmax over V bf16 values, the lowest index winning
 * ties (-0 equals +0; a NaN never beats a number; a row whose element 0 is NaN yields 0).
 * Then a = number of leading j < n_draft[b] with drafts[b,j] == argmax[b,j];
 * accepted[b] = drafts[b,0..a) followed by argmax[b,a]; n_accepted[b] = a + 1.
 *   logits_bf16       device, bf16, element (row r, column v) at logits_bf16[r*row_stride_elems + v],
 *                     r = b*(K+1)+j; 2-byte aligned; read-only; fastest when rows are 16-byte aligned
 *   row_stride_elems  >= V
 *   drafts, n_draft   device [B,K], [B] (n_draft clamped to 0..K)
 *   argmax_out        device [B, K+1] int32 (all rows, also those beyond n_draft)
 *   accepted          device [B, K+1] int32, unused slots = -1;  n_accepted device [B] int32
 *   workspace         device scratch of sam_workspace_bytes(B, K), zeroed by sam_workspace_init
 * Errors: SAM_ERR_INVALID_ARG, SAM_ERR_TOO_SMALL, SAM_ERR_CUDA. */
int sam_verify(const void* logits_bf16, int64_t row_stride_elems, int32_t B, int32_t K, int32_t V,
               const int32_t* drafts, const int32_t* n_draft,
               int32_t* argmax_out, int32_t* accepted, int32_t* n_accepted,
               void* workspace, int64_t workspace_bytes, void* cuda_stream);

/* Fused steady-state step (Algorithm 3, one iteration of the speculative decoding loop):
 * sam_verify, then the accepted tokens of each stream are walked from (state, matched_len)
 * exactly as sam_draft would with new_tokens = accepted, n_new = n_accepted, and the next
 * draft is emitted - all on the device, with no host round trip in between.
 * next_drafts / next_n_draft may alias drafts / n_draft.
 * Errors: as sam_verify and sam_draft. */
int sam_step(const sam_index* idx,
             const void* logits_bf16, int64_t row_stride_elems, int32_t B, int32_t K, int32_t V,
             const int32_t* drafts, const int32_t* n_draft,
             int32_t* argmax_out, int32_t* accepted, int32_t* n_accepted,
             int32_t* state, int32_t* matched_len, int32_t min_match,
             int32_t* next_drafts, int32_t* next_n_draft,
             void* workspace, int64_t workspace_bytes, void* cuda_stream);

/* Step options and running statistics.
 *   SAM_STEP_NO_SPECULATION   (Section 5.4.3 "Adaptive switch"; Algorithm 3 step 4) speculation is off
 *       for this call: every stream verifies an empty proposal (plain decoding: row 0 gives the one
 *       committed token), the automaton still follows that token so that drafting can resume at once,
 *       and no new draft is emitted (next_n_draft = 0, next_drafts = -1).
 *   SAM_STEP_SKIP_UNUSED_ROWS only rows 0..n_draft[b] of stream b are read (row n_draft[b] supplies the
 *       model's own token after a full accept); argmax_out of the rows beyond is -1.  A small kernel
 *       lists the used rows first, then the argmax kernel streams only those - the bytes read per call
 *       drop from B*(K+1) rows to sum(n_draft)+B rows.
 *   SAM_STEP_ROW_LIST_READY   (sam_step_ex only, together with SAM_STEP_SKIP_UNUSED_ROWS) the caller states
 *       that the previous call through this workspace was a sam_step_ex with SAM_STEP_SKIP_UNUSED_ROWS for
 *       the same B and K, and that drafts / n_draft are what that call wrote to next_drafts / next_n_draft,
 *       unmodified.  Every such call leaves the list of the rows its successor needs in the workspace (its
 *       accept kernel writes it as a by-product), so the listing kernel is not launched: two launches per
 *       step instead of three.  If the workspace holds no list for this B and K (first call, workspace
 *       re-initialised, another shape in between) nothing is reduced, the outputs of the call are not
 *       valid and the status word reads 3 (sam_workspace_status); a list that is stale in any other way
 *       gives the results of the rows it names - wrong for this call, but every access stays inside the
 *       caller's buffers.
 *   counters  device, int64[SAM_N_COUNTERS], 8-byte aligned, or NULL.  Every call ADDS, per stream:
 *       [0] verification passes (1), [1] committed tokens, [2] proposed draft tokens, [3] accepted draft
 *       tokens, [4] non-empty proposals, [5] logits rows read.  Section 6.5: OTE = [1]/[0],
 *       SHR = [3]/[2] (or [3]/(K*[4]) when every proposal counts as K tokens).  The caller zeroes and
 *       reads them (a device-to-host copy of 48 bytes whenever it wants the figures).
 * Everything else is as in sam_verify / sam_step, which are these calls with flags = 0, counters = NULL. */
#define SAM_STEP_NO_SPECULATION   1u
#define SAM_STEP_SKIP_UNUSED_ROWS 2u
#define SAM_STEP_ROW_LIST_READY   4u
#define SAM_N_COUNTERS            6
int sam_verify_ex(const void* logits_bf16, int64_t row_stride_elems, int32_t B, int32_t K, int32_t V,
                  const int32_t* drafts, const int32_t* n_draft,
                  int32_t* argmax_out, int32_t* accepted, int32_t* n_accepted,
                  uint32_t flags, int64_t* counters,
                  void* workspace, int64_t workspace_bytes, void* cuda_stream);
int sam_step_ex(const sam_index* idx,
                const void* logits_bf16, int64_t row_stride_elems, int32_t B, int32_t K, int32_t V,
                const int32_t* drafts, const int32_t* n_draft,
                int32_t* argmax_out, int32_t* accepted, int32_t* n_accepted,
                int32_t* state, int32_t* matched_len, int32_t min_match,
                int32_t* next_drafts, int32_t* next_n_draft,
                uint32_t flags, int64_t* counters,
                void* workspace, int64_t workspace_bytes, void* cuda_stream);

/* Verification in two halves, for a vocabulary that is split over several GPUs (the target model's
 * output layer under tensor parallelism; the paper runs its models with TP 2-8 but does not discuss
 * verification there - this is the natural composition).
 *
 * sam_argmax_partial reduces rows x V logits that are columns v_offset .. v_offset+V-1 of the full
 * vocabulary and leaves one 64-bit word per row in keys: 0 when the shard holds nothing greater than
 * -inf, otherwise a packed (value, index) whose signed 64-bit order is "greater value first, then
 * smaller GLOBAL index".  The elementwise maximum of the shards' words - one MAX all-reduce of
 * rows x 8 bytes over NCCL, or any other route - is therefore the word of the full row, ties and all.
 *   keys   device, int64[rows + 1], 8-byte aligned; zeroed by this call; keys[rows] is a status word
 *          (0 = fine, see sam_workspace_status) and should be left out of the reduction
 *   A row whose GLOBAL element 0 is NaN yields index 0 (only the shard with v_offset = 0 can tell).
 * sam_step_from_keys takes the reduced words (device, int64[B*(K+1)]; they are re-zeroed), decodes them
 * into argmax_out and then does what sam_step does after its argmax: accept, follow the committed
 * tokens from (state, matched_len), emit the next draft.
 * Errors: SAM_ERR_INVALID_ARG, SAM_ERR_NOT_UPLOADED, SAM_ERR_CUDA. */
int sam_argmax_partial(const void* logits_bf16, int64_t row_stride_elems, int64_t rows, int32_t V, int32_t v_offset,
                       int64_t* keys, void* cuda_stream);
int sam_step_from_keys(const sam_index* idx, int64_t* keys, int32_t B, int32_t K,
                       const int32_t* drafts, const int32_t* n_draft,
                       int32_t* argmax_out, int32_t* accepted, int32_t* n_accepted,
                       int32_t* state, int32_t* matched_len, int32_t min_match,
                       int32_t* next_drafts, int32_t* next_n_draft, void* cuda_stream);

/* The adaptive switch itself (Section 5.4.3; Algorithm 3 step 4): 1 = keep speculating, 0 = fall back
 * to plain decoding because the context length or the batch size exceeds its threshold.  The
 * thresholds are deployment-specific ("empirically determined" in the paper); a host-side helper,
 * no device work. */
int sam_adaptive_switch(int64_t context_len, int64_t batch_size, int64_t max_context_len, int64_t max_batch_size);

/* The same decision taken from the running statistics instead of fixed thresholds (Section 5.4.3: speculation is
 * disabled "when its overhead outweighs the gains"; Section 6.5: OTE).  The paper leaves the rule to the
 * deployment; the one here prices a verification pass over r of the K+1 rows at 1 + (cost_ratio - 1)(r - 1)/K
 * one-row passes - cost_ratio, the measured cost of a full (K+1)-row pass relative to a one-row pass, comes from
 * the caller - and keeps speculating when the passes behind the counters committed more tokens than they cost
 * (plain decoding commits one token per one-row pass):
 *     accepted draft tokens * K  >  (cost_ratio - 1) * (rows read - passes)      in double precision;
 * with all K+1 rows read in every pass this is OTE > cost_ratio.
 *   counters    HOST, int64[SAM_N_COUNTERS]: a copy of the device counters of sam_step_ex / sam_verify_ex over
 *               the window to judge (the caller zeroes them, or subtracts two readings); only passes [0],
 *               accepted draft tokens [3] and rows read [5] are used.  Take them from passes that did speculate:
 *               passes with SAM_STEP_NO_SPECULATION show OTE = 1 by construction, so a caller that has switched
 *               speculation off should try it again from time to time.
 *   K           the draft length those passes used, 1..SAM_K_MAX;  cost_ratio > 0
 * Returns 1 (speculate), 0 (do not), or SAM_ERR_INVALID_ARG.  A window without passes returns 1.  Host only. */
int sam_speculation_pays(const int64_t* counters, int32_t K, double cost_ratio);

/* Allocation-free form of sam_verify (a packaging variant; the paper has no counterpart).
 * Some callers cannot obtain device scratch at all: a plugin running inside a serving engine
 * that has already handed every free byte of device memory to its own pools (a late cudaMalloc
 * there fails, or stalls the whole device while it runs), or a caller that only holds raw
 * pointers from another runtime and has no allocator to ask.  For them the per-row scratch of
 * the verification kernels lives inside the library image itself, in a fixed device array of
 * SAM_STATIC_MAX_ROWS 64-bit words (128 KiB) that every GPU which loads the library holds until
 * the process exits.  Arguments, results and semantics are exactly those of sam_verify, minus
 * the workspace; inputs and outputs are still the caller's device buffers.
 *   - B * (K + 1) must not exceed SAM_STATIC_MAX_ROWS, otherwise SAM_ERR_TOO_LARGE is returned
 *     and nothing is launched.
 *   - The call itself allocates nothing (no cudaMalloc / cudaFree, no allocating library
 *     routine): it zero-fills the rows it is about to use with a stream-ordered memset and
 *     enqueues the two kernels.
 *   - The first call on each device looks up the device address of the array (with that device
 *     current) and keeps it; make that first call outside any stream capture.
 *   - All calls on a device share the one array, which keeps whatever the previous call left
 *     in it: two calls that overlap on the GPU (different streams, no ordering between them)
 *     race on it and return garbage.  Order them, or use sam_verify with separate workspaces.
 *   - The array also holds the status word of the verification kernels (see sam_workspace_status);
 *     every call clears it together with its rows, and sam_static_status reads it: 0 = the last
 *     call on this device completed normally, otherwise a kernel gave up on a bounded wait and that
 *     call's outputs are not valid (simply call again).  sam_static_status copies one int to the
 *     host and synchronises the stream - a diagnostic that allocates nothing either.
 * Errors: SAM_ERR_INVALID_ARG, SAM_ERR_TOO_LARGE, SAM_ERR_CUDA. */
#define SAM_STATIC_MAX_ROWS   16384
int sam_verify_static(const void* logits_bf16, int64_t row_stride_elems, int32_t B, int32_t K, int32_t V,
                      const int32_t* drafts, const int32_t* n_draft,
                      int32_t* argmax_out, int32_t* accepted, int32_t* n_accepted,
                      void* cuda_stream);
int sam_static_status(int32_t* status_out, void* cuda_stream);

/* Host-buffer form of sam_step, for callers whose logits and bookkeeping live in host memory
 * (Algorithm 3, one loop iteration, end to end).  Copies logits [B*(K+1) rows, row_stride_elems
 * apart, V used], drafts, n_draft, state and matched_len from the host into `staging`, runs
 * sam_step there, copies argmax_out, accepted, n_accepted, state, matched_len, next_drafts and
 * next_n_draft back and synchronises the stream before returning.  Every pointer except
 * `staging` is HOST memory (pinned memory makes the copies asynchronous and faster); `staging`
 * is device memory of at least sam_step_host_staging_bytes(...), 256-byte aligned, contents
 * undefined between calls (it embeds the verification scratch, which the call zeroes itself).
 * Errors: as sam_step. */
int64_t sam_step_host_staging_bytes(int64_t row_stride_elems, int32_t B, int32_t K, int32_t V);
int sam_step_host(const sam_index* idx,
                  const void* logits_bf16, int64_t row_stride_elems, int32_t B, int32_t K, int32_t V,
                  const int32_t* drafts, const int32_t* n_draft,
                  int32_t* argmax_out, int32_t* accepted, int32_t* n_accepted,
                  int32_t* state, int32_t* matched_len, int32_t min_match,
                  int32_t* next_drafts, int32_t* next_n_draft,
                  void* staging, int64_t staging_bytes, void* cuda_stream);

/* sam_step_host with step options (SAM_STEP_*; SAM_STEP_ROW_LIST_READY is not accepted here).  With
 * SAM_STEP_SKIP_UNUSED_ROWS only rows 0..n_draft[b] of every stream are copied to the device (one copy per
 * run of rows that touch or nearly touch) - the host-to-device traffic, which dominates this call, shrinks
 * with the proposals. */
int sam_step_host_ex(const sam_index* idx,
                     const void* logits_bf16, int64_t row_stride_elems, int32_t B, int32_t K, int32_t V,
                     const int32_t* drafts, const int32_t* n_draft,
                     int32_t* argmax_out, int32_t* accepted, int32_t* n_accepted,
                     int32_t* state, int32_t* matched_len, int32_t min_match,
                     int32_t* next_drafts, int32_t* next_n_draft, uint32_t flags,
                     void* staging, int64_t staging_bytes, void* cuda_stream);

/* ---------------------------------------------------------------- growing index */

/* An index that keeps absorbing text after it was built (Section 5.4.2: verified tokens are
 * inserted into the automaton so that it follows the growing context; Section 5.4.3 "Asynchronous
 * SAM construction": building is handed to a child thread that serves a waiting queue, and
 * drafting carries on with what is available until the new part is ready).
 *
 * sam_build_growing builds the automaton of corpus[0..n) (n may be 0) like sam_build, keeps the
 * builder alive in a thread of its own, and sizes the device blob (sam_sizes) for up to max_tokens
 * tokens: room for 2*max_tokens+2 state records, 8*max_tokens wide edges, a dense root table for token ids
 * 0..max_token_id, the text, an 8 MiB staging area for large updates and eight 1 MiB slots for small ones.  sam_upload, sam_draft,
 * sam_verify, sam_step, sam_export, sam_sizes and sam_free work as for any other index.
 *   max_tokens    1 .. 2^29, >= n;  max_token_id  largest token id that will ever be indexed
 *                 (separators included), < 2^24
 * Errors: SAM_ERR_INVALID_ARG, SAM_ERR_NOMEM. */
int sam_build_growing(const int32_t* corpus, int64_t n, const int32_t* separators, int32_t n_sep,
                      int64_t max_tokens, int32_t max_token_id, sam_index** out);

/* Appends tokens[0..n) (host) to the indexed text.  sam_extend_async copies them into the builder
 * thread's queue and returns at once; sam_extend also waits until the builder thread has indexed
 * everything queued so far.  Separators are appended like any other token (a new session is
 * "SEP, tokens...").  Nothing changes on the device until sam_sync.
 * Errors: SAM_ERR_INVALID_ARG (not a growing index, token id outside 0..max_token_id),
 * SAM_ERR_TOO_LARGE (more than max_tokens in total), SAM_ERR_NOMEM. */
int sam_extend_async(sam_index* idx, const int32_t* tokens, int64_t n);
int sam_extend(sam_index* idx, const int32_t* tokens, int64_t n);

/* Progress of a growing index, in tokens: handed in so far, indexed on the host so far, visible to
 * the device kernels so far.  Any pointer may be NULL. */
int sam_pending(sam_index* idx, int64_t* tokens_queued, int64_t* tokens_built, int64_t* tokens_on_device);

/* Brings the device copy up to date with everything the builder thread has finished: the records
 * of changed states, rewritten wide rows, changed root entries and the appended text are scattered
 * into the live arrays by a small kernel on the stream (a whole new image is copied instead after
 * the wide-edge area had to be laid out afresh).  Does not wait for the builder thread and does not
 * synchronise the stream; hot-path calls enqueued afterwards on the same stream see the grown
 * automaton.  Call it from the thread that makes the hot-path calls.
 * Where the bytes travel: an update of up to 1 MiB (what accumulates between two decoding steps) has
 * normally been copied into one of the blob's slots already, by the builder thread, through page-locked
 * memory on a stream the library owns (both created by sam_upload of a growing index, released by
 * sam_free), while earlier steps were running; sam_sync then only makes the caller's stream wait for
 * that copy's event and launches the scatter kernel.  The copy touches nothing a kernel reads; every
 * write into live records, rows, root table and text happens in the scatter kernel, in stream order
 * between the step before and the step after.  An update that was not sent ahead (no free slot, or
 * larger than a slot) is copied on the caller's stream instead, as before.
 * After it, run sam_renormalize on every batch of stream states that will be used again - or use
 * sam_sync_renormalize, which does both.
 * Errors: SAM_ERR_INVALID_ARG, SAM_ERR_NOT_UPLOADED, SAM_ERR_TOO_LARGE (the automaton no longer
 * fits the blob), SAM_ERR_CUDA. */
int sam_sync(sam_index* idx, void* cuda_stream, int64_t* tokens_on_device);

/* sam_sync followed by sam_renormalize(idx, B, state, matched_len) in as few launches as possible: when
 * the last pending update is a small one, the block of its scatter kernel that finishes last repairs the
 * stream states, so ONE kernel stands between the previous decoding step and the next; when nothing is
 * pending nothing is launched (states only need repair after growth).  Same results as the two calls.
 * Errors: as sam_sync and sam_renormalize. */
int sam_sync_renormalize(sam_index* idx, int32_t B, int32_t* state, const int32_t* matched_len, void* cuda_stream,
                         int64_t* tokens_on_device);

/* What sam_sync has applied to the device so far: updates that scattered only what changed, updates
 * that copied a whole new image, and the host-to-device bytes of both.  Any pointer may be NULL. */
int sam_update_stats(const sam_index* idx, int64_t* incremental, int64_t* full_images, int64_t* bytes_copied);

/* Forces the rare path of sam_sync: with every > 0, each every-th update the builder thread packs lays the
 * wide rows out afresh and reaches the device as a whole image - what otherwise happens only when the
 * wide-edge area fills up.  0 (the default) never forces it.  For tests and for measuring that path; takes
 * effect with the next update the builder thread packs.  No counterpart in the paper.
 * Errors: SAM_ERR_INVALID_ARG (not a growing index, every < 0). */
int sam_growing_set_relayout_every(sam_index* idx, int64_t every);

/* When the text grows, a state can be split, and a stream's (state, matched_len) may then name the
 * half that no longer holds its string.  This moves every state[b] (device, [B], in place) up its
 * suffix links to the state with len(link(s)) < matched_len[b] <= len(s); matched_len is unchanged.
 * (The paper does not discuss this; it follows from what the states of a suffix automaton are.)
 * Errors: SAM_ERR_INVALID_ARG, SAM_ERR_NOT_UPLOADED, SAM_ERR_CUDA. */
int sam_renormalize(const sam_index* idx, int32_t B, int32_t* state, const int32_t* matched_len, void* cuda_stream);

/* ---------------------------------------------------------------- composite drafting */

/* Drafting from several automata at once (Section 5.4.2; Algorithm 3 step 1: the automaton of the
 * current session is combined with those of the top-K retrieved contexts, "the similarity scores
 * determine the weights of each SAM").  The paper does not define the combination; the rule here:
 * every stream has M slots, each naming one member index and carrying a weight; each slot keeps its
 * own (state, matched_len) and follows the new tokens in its own automaton; the draft is emitted by
 * the slot with the largest weight * matched_len (float32 product) among the slots whose match
 * reaches min_match, the lowest slot winning ties; if no slot qualifies there is no draft.
 * Retrieval and similarity scoring are the caller's business: slots and weights are inputs.
 *
 * sam_set_create copies the device views of n_members uploaded indexes into a caller-owned device
 * table (device_buf, at least sam_set_bytes(n_members), 16-byte aligned); the member handles must
 * outlive the set.  After a member has grown (sam_sync), sam_set_refresh copies the views again.
 *
 * sam_multi_draft: as sam_draft, with per-slot state:
 *   slots        device [B, M] int32, member number or -1 for an empty slot;  1 <= M <= 8
 *   weights      device [B, M] float32
 *   state, matched_len   device [B, M] int32, in/out (a new slot starts at (0, 0))
 *   new_tokens, ld, n_new, K, min_match, drafts, n_draft   as in sam_draft (shared by all slots)
 *   chosen       device [B] int32: the slot that drafted, or -1
 * Verification needs nothing new: sam_verify on the emitted drafts, then sam_multi_draft with
 * new_tokens = accepted, n_new = n_accepted.
 * Errors: SAM_ERR_INVALID_ARG, SAM_ERR_TOO_SMALL, SAM_ERR_NOT_UPLOADED, SAM_ERR_NOMEM, SAM_ERR_CUDA. */
typedef struct sam_set sam_set;
int64_t sam_set_bytes(int32_t n_members);
int sam_set_create(const sam_index* const* members, int32_t n_members, void* device_buf, int64_t bytes,
                   void* cuda_stream, sam_set** out);
int sam_set_refresh(sam_set* set, void* cuda_stream);
void sam_set_free(sam_set* set);
/* sam_renormalize for composite state: after member number `member` has grown (sam_sync, sam_set_refresh),
 * every slot that names it is moved to the state that now holds its string; other slots are untouched.
 * slots, state, matched_len: device [B, M]. */
int sam_set_renormalize(const sam_set* set, int32_t member, int32_t B, int32_t M, const int32_t* slots,
                        int32_t* state, const int32_t* matched_len, void* cuda_stream);
int sam_multi_draft(const sam_set* set, int32_t B, int32_t M, const int32_t* slots, const float* weights,
                    int32_t* state, int32_t* matched_len, const int32_t* new_tokens, int32_t ld, const int32_t* n_new,
                    int32_t K, int32_t min_match, int32_t* drafts, int32_t* n_draft, int32_t* chosen,
                    void* cuda_stream);

/* One decoding step with composite drafting, fused like sam_step: vocabulary argmax over all B*(K+1) rows
 * (with every slot's walk-ahead over the drafts riding along), accept, then every slot follows the
 * committed tokens in its own automaton and the slots compete for the next draft - the result is what
 * sam_verify followed by sam_multi_draft(new_tokens = accepted, n_new = n_accepted) gives.
 *   workspace   device scratch of sam_multi_workspace_bytes(B, K, M), zeroed once by sam_workspace_init
 *   other arguments as in sam_verify and sam_multi_draft; next_drafts / next_n_draft may alias drafts / n_draft
 * Errors: SAM_ERR_INVALID_ARG, SAM_ERR_TOO_SMALL, SAM_ERR_CUDA. */
int64_t sam_multi_workspace_bytes(int32_t B, int32_t K, int32_t M);
int sam_multi_step(const sam_set* set,
                   const void* logits_bf16, int64_t row_stride_elems, int32_t B, int32_t K, int32_t V,
                   const int32_t* drafts, const int32_t* n_draft,
                   int32_t* argmax_out, int32_t* accepted, int32_t* n_accepted,
                   int32_t M, const int32_t* slots, const float* weights, int32_t* state, int32_t* matched_len,
                   int32_t min_match, int32_t* next_drafts, int32_t* next_n_draft, int32_t* chosen,
                   void* workspace, int64_t workspace_bytes, void* cuda_stream);

/* ---------------------------------------------------------------- diagnostics */

/* Per-kernel device timing of sam_verify / sam_step (measurement aid; the paper has no
 * counterpart).  sam_profile_enable(n) creates CUDA events for the next n calls (n = 0 turns
 * profiling off and frees them); while enabled, each call records events before the argmax
 * kernel, between the two kernels and after the accept kernel on the caller's stream.
 * sam_profile_read(i, ...) returns the two durations of the i-th profiled call in
 * milliseconds; the stream must have been synchronised by the caller first.
 * Process-wide state, not thread-safe; enable/disable is not a hot-path call. */
int sam_profile_enable(int32_t max_calls);
/* Selects the kernels of sam_verify / sam_step for later calls (process-wide; for measurements
 * and tests):
 *   0 = automatic (default): the bulk-copy pipelined argmax kernel when the logits base and row
 *       stride are 16-byte aligned and the call is large (more than 768 MiB of logits, or K > 16);
 *       the direct-load kernel otherwise; each followed by the accept kernel as a dependent launch;
 *   1 = always the direct-load kernel;
 *   2 = the bulk-copy kernel whenever the rows are aligned, with the accept step of every stream
 *       inside it: every CTA takes the rows its streams' proposals use (0 .. n_draft) first, a stream's
 *       accept step runs as soon as those rows are complete, and the rows behind the proposals are
 *       reported by the kernel when they are (one launch per call; measured slower than two launches
 *       on B200, so not the default; rows too short for 48 KB tiles fall back to two launches);
 *   3 = the bulk-copy kernel whenever the rows are aligned, followed by the accept kernel. */
int sam_set_argmax_variant(int32_t variant);
int32_t sam_profile_count(void);
int sam_profile_read(int32_t call, float* argmax_ms, float* accept_ms);

/* Number of kernels this library has enqueued in this process so far (all entry points, all
 * threads); a measurement aid with no counterpart in the paper. */
int64_t sam_launch_count(void);

/* Static description of a status code. */
const char* sam_strerror(int status);

/* cudaError_t value of the most recent failed CUDA call made by this library on the calling
 * thread (0 if none). */
int sam_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SAM_B200_H */
