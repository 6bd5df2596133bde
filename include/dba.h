/*
 * dba.h -- C ABI of the Dynamic Beam Allocation step library (CUDA, sm_100a).
 *
 * The library runs, for a batch of B independent sentences with beam size k and vocabulary V, the
 * per-timestep step of lexically constrained beam search with dynamic beam allocation
 * (Post & Vilar 2018: Algorithm 2 "KBEST-DBA", Sections 3.1-3.3) with the log-softmax of Section 2 in
 * front of it.  All arithmetic of the step runs in CUDA kernels; there is no CPU fallback.
 *
 * Conventions
 *   - Every function returns a dba_status; nothing throws or aborts.  Argument errors are detected on
 *     the host before anything is launched.
 *   - "dev" pointers are device memory, "host" pointers are host memory.  The library allocates no
 *     device memory: the caller provides one workspace (dba_workspace_bytes) that must outlive the
 *     handle, and owns every input and output buffer.  The library owns only the handle.
 *   - dba_step only enqueues work on the stream given to dba_init and does not synchronise.
 *   - Row r = b*k + h of any [B*k, ...] array belongs to beam slot h of sentence b.
 *   - Token ids are int32 in [0, V).  pad_id / bos_id / eos_id are the special symbols.
 *   - Logits must be finite or -inf.  With NaN or +inf in a row the selection is unspecified.
 *   - Limits: k <= 64, at most 64 constraint tokens per sentence, k*V < 2^31, V >= 1.  One thread block keeps
 *     a sentence's k*(P+2) candidates (P = phrases of the sentence that has most) and its rows' partial
 *     lists in shared memory: every constraint set fits for k <= 40; at k = 64 sets of up to 36 phrases fit
 *     for rows of up to 352 KB and sets of up to 12 phrases for rows of up to 1 MiB.  dba_init returns
 *     DBA_ERR_UNSUPPORTED when the configuration does not fit.
 *   - Threads: calls on one handle must not overlap, nor may two dba_init calls (the kernels' shared-memory
 *     limits are raised there, once per process and device); different handles may otherwise be used from
 *     different host threads.  A handle belongs to the device that was current in dba_init; make it current
 *     again for every call on the handle.
 *   - Speed: the streaming row scan needs 16-byte aligned rows (base pointer and row stride) whose length in
 *     bytes is a multiple of 16 and at most 1 MiB; other shapes are served by a plain multi-pass kernel, exact
 *     but many times slower.  Rows in which more than 256 entries of a 44 KB stretch tie at the value of its
 *     (k+2)-th largest entry cost an extra pass over that stretch (dba_counters reports how often).
 *
 * Slot kinds: a slot is EMPTY when its score is -inf, FINISHED when it is live and its last token is
 * eos_id, OPEN otherwise.  After dba_init (and dba_reset) slot 0 of every sentence is open with score 0
 * and last token bos_id; slots 1..k-1 are empty.
 */
#ifndef DBA_H
#define DBA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dba_handle dba_handle;

typedef enum {
    DBA_OK = 0,
    DBA_ERR_INVALID_ARG = 1,   /* null pointer, bad size, malformed constraint table, bad token id      */
    DBA_ERR_UNSUPPORTED = 2,   /* over a documented limit (k > 64, > 64 constraint tokens, k*V >= 2^31,
                                  candidates beyond shared memory)                                      */
    DBA_ERR_STATE = 3,         /* step after max_steps, host-staging call without the staging flag     */
    DBA_ERR_CUDA = 4,          /* a CUDA runtime call failed                                            */
    DBA_ERR_TIMEOUT = 5,       /* a bounded device-side wait gave up (reported by dba_finalize)        */
    DBA_ERR_WORKSPACE = 6      /* workspace too small or misaligned                                     */
} dba_status;

typedef enum { DBA_F32 = 0, DBA_BF16 = 1 } dba_dtype;

enum {
    DBA_FLAG_ADJUST_OFF   = 1u,  /* Section 5 (grid-beam-search simulation): no bank adjustment        */
    DBA_FLAG_LENGTH_NORM  = 2u,  /* Section 4: dba_finalize ranks completed hypotheses by score/length  */
    DBA_FLAG_HOST_STAGING = 4u,  /* reserve workspace for dba_step_host                                 */
    DBA_FLAG_PRUNE_NORMALISED = 8u, /* Section 4, read the other way: the threshold pruning compares completed
                                    hypotheses by score/length (see prune_threshold)                    */
    DBA_FLAG_FUSED_PROJECTION = 16u /* reserve workspace for dba_step_fused (needs k <= 30)              */
};

/* Bits of dba_step_out.stop (Section 4's stopping rule; Section 6.4's early stopping). */
enum {
    DBA_STOP_ALL_COMPLETED  = 1,  /* the beam is not empty and every hypothesis on it has generated eos_id */
    DBA_STOP_SOME_COMPLETED = 2   /* some hypothesis on the beam has generated eos_id                       */
};

/*
 * Problem statement (Section 3): a fixed beam size k and, per sentence, a set of word constraints (one
 * token) and phrasal constraints (two or more contiguous tokens, met in order).  C_b, the number of
 * constraints of sentence b, counts every token of every word and phrase.
 * The constraint arrays are HOST memory, read during dba_init only; the caller keeps ownership.
 */
typedef struct {
    int32_t B, k, V, max_steps;
    int32_t pad_id, bos_id, eos_id;
    int32_t logit_dtype;               /* dba_dtype */
    uint32_t flags;
    const int32_t* sent_phrase_off;    /* [B+1]  phrases of sentence b are [off[b], off[b+1])             */
    const int32_t* phrase_tok_off;     /* [P+1]  tokens of phrase p are   [off[p], off[p+1]), non-empty   */
    const int32_t* tok;                /* [sum]  token ids in [0, V), none of pad/bos/eos                 */
    float prune_threshold;             /* Section 4: > 0 removes, after every step, the hypotheses (completed or
                                          not) whose score is more than this below the best completed
                                          hypothesis on the beam (the paper uses 20); <= 0: no pruning.
                                          Scores are cumulative log-probabilities on both sides; with
                                          DBA_FLAG_PRUNE_NORMALISED a completed hypothesis enters the comparison
                                          (as the reference and as the one tested) with score / length, as
                                          Section 4 normalises completed hypotheses before it prunes; the beam
                                          stays ordered by cumulative score either way                       */
} dba_config;

/*
 * Outputs of one step: the new beam, in decreasing score order (ties: lower back-pointer*V + token
 * first), empty slots last.  Each array is [B*k]; any pointer may be NULL (that output is skipped).
 * dba_step takes DEVICE pointers here, dba_step_host takes HOST pointers.
 *   backptr   beam slot (0..k-1) of the previous beam this hypothesis extends (Algorithm 2: i of (i,j))
 *   token     the token generated (Algorithm 2: j of (i,j)); pad_id for empty slots
 *   score     cumulative log-probability (fp32); -inf for empty slots
 *   bank      number of constraint tokens met (Section 3.2); -1 for empty slots
 *   met_mask  bit j set = constraint token position j (phrases flattened in order) is marked met
 *   active    position of the last met token of a begun, unfinished phrase, else -1
 *   row_lse   log-sum-exp of the INPUT rows of this step (fp32; 0 for rows that were not open)
 *   stop      [B], not [B*k]: DBA_STOP_* bits of each sentence's new beam.  The library keeps stepping a
 *             sentence whatever they say (completed hypotheses repeat eos_id at an unchanged score); the
 *             caller owns the loop: "all completed" is the paper's stopping rule, "some completed" its
 *             early-stopping variant.
 */
typedef struct {
    int32_t*  backptr;
    int32_t*  token;
    float*    score;
    int32_t*  bank;
    uint64_t* met_mask;
    int32_t*  active;
    float*    row_lse;
    int32_t*  stop;
} dba_step_out;

/* Bytes of device workspace a handle for this configuration needs (256-byte aligned base). */
dba_status dba_workspace_bytes(const dba_config* cfg, size_t* bytes);

/*
 * Validates cfg, flattens the constraint tables, copies them to the workspace and sets the initial
 * beam (Algorithm 1, DECODER-INIT).  `cuda_stream` is a cudaStream_t (NULL = default stream); all later
 * work of the handle is enqueued on it.  Synchronises the stream once before returning.
 */
dba_status dba_init(const dba_config* cfg, void* workspace_dev, size_t workspace_bytes,
                    void* cuda_stream, dba_handle** out);

/* Back to the initial beam and step 0, same constraints (enqueued; does not synchronise). */
dba_status dba_reset(dba_handle* h);

/*
 * One timestep (Algorithm 2).  logits_dev: [B*k, V] of the configured dtype, element (r, w) at
 * logits_dev[r*row_stride_elems + w]; row r must hold the model output for the hypothesis currently in
 * beam slot r (the caller re-orders its decoder state by the previous step's backptr).
 * Rows of empty and finished slots are not read.
 *   Section 2 / 3.1  score(h, w) = fl32(fl32(x[h,w] - lse_h) + score_h); a finished slot only continues
 *                    with eos_id at an unchanged score.
 *   Section 3.3      score(h, eos_id) = -inf while slot h has unmet constraint tokens.
 *   Section 3.1      candidates = the k best cells of the k x V matrix, every token that advances an
 *                    open slot through its constraints, and every live slot's best token; each carries
 *                    its updated constraint marks (a broken phrase is unwound).
 *   Section 3.2      the k slots are divided over the C_b+1 banks (floor(k/(C_b+1)) each, the rest to
 *                    the top bank; unfillable slots move to the nearest banks that can use them) and
 *                    each bank keeps its best candidates.
 *   Section 4        with prune_threshold > 0, hypotheses of the new beam scoring below (best completed
 *                    score - prune_threshold) are removed: their slots are empty.
 * row_lse_in_dev (optional, [B*k] fp32): when non-NULL, the row normalisers are taken from it instead
 * of being computed from the logits (e.g. all zeros when the rows are log-probabilities already); the
 * computed values are still what out->row_lse reports.
 * Returns DBA_ERR_STATE after max_steps steps.
 */
dba_status dba_step(dba_handle* h, const void* logits_dev, int64_t row_stride_elems,
                    const float* row_lse_in_dev, const dba_step_out* out_dev);

/*
 * The same step fused into its producer (Section 2: the k x |V_T| matrix is DECODER-STEP's output, the decoder's
 * final hidden states times the output embedding): the caller passes the hidden states of the R = B*k hypotheses and
 * the embedding, the logits are computed on the tensor cores and consumed as they appear (see dba_project_scan for
 * shapes, alignment and accuracy), and the rest of the step is dba_step's.  Needs DBA_FLAG_FUSED_PROJECTION.
 *   hidden_dev [B*k, D] bf16, row r = hypothesis in beam slot r;  embed_dev [V, D] bf16.
 * Every row is projected, open or not.  One corner differs from dba_step: when a row's scores are equal over a run
 * that reaches past the k+2 entries kept of the row, dba_step looks the row up again to find the lowest word ids
 * of the run; here there is no row to look up, the kept entries stand, and counters[1] of dba_counters counts it.
 */
dba_status dba_step_fused(dba_handle* h, const void* hidden_dev, int64_t hidden_stride_elems, const void* embed_dev,
                          int64_t embed_stride_elems, int32_t D, const dba_step_out* out_dev);

/*
 * The same step with HOST buffers: copies the logits to a staging area in the workspace, runs the
 * step, copies the requested outputs back and synchronises the stream.  Needs DBA_FLAG_HOST_STAGING.
 * Pinned host memory makes the copies asynchronous with respect to the host until the final wait.
 */
dba_status dba_step_host(dba_handle* h, const void* logits_host, int64_t row_stride_elems,
                         const dba_step_out* out_host);

/*
 * Section 3.3: per sentence the completed hypothesis (last token eos_id) with the highest score
 * (score / length with DBA_FLAG_LENGTH_NORM, length counting the end token), lowest slot on ties; if
 * none is completed, the best live slot of the highest occupied bank, flagged not completed.
 * tokens_host [B, max_steps]: generated tokens up to and including the first eos_id (bos excluded),
 * padded with pad_id;  len_host [B];  score_host [B];  flags_host [B], bit 0 = completed.
 * Any pointer may be NULL.  Synchronises the stream.  Returns DBA_ERR_TIMEOUT / DBA_ERR_CUDA if a
 * kernel of an earlier step recorded a problem in the device status word.
 */
dba_status dba_finalize(dba_handle* h, int32_t* tokens_host, int32_t* len_host, float* score_host,
                        int32_t* flags_host);

/*
 * Optional per-kernel timing for benchmarks.  While enabled, dba_step brackets each of its two kernels
 * (row scan; candidates with the allocation at their end) with CUDA events on the handle's stream; dba_step_fused
 * brackets the projection with its merge, and the rest (constraint-token logits, candidates).
 * dba_timing_read waits for the stream, adds up the elapsed milliseconds of every step recorded since the last
 * read into ms_total[0..1] (ms_total[2] is 0: the allocation has no kernel of its own), stores the number of
 * steps in *steps and clears the record.  At most 4096 steps are
 * kept between reads (further steps are not recorded).  Off by default.
 */
dba_status dba_timing_enable(dba_handle* h, int32_t on);
dba_status dba_timing_read(dba_handle* h, double ms_total[3], int64_t* steps);

/*
 * Diagnostic counters of the handle's device status block (never an error).  Synchronises the stream.
 *   counters[0]  row segments whose k+2 best entries the row scan had to find by a second, slow pass over global
 *                memory, because more entries tied at its selection bound than its lists hold (long runs of
 *                equal logits).  Results are exact either way; a large count explains a slow step.
 *   counters[1]  dba_step_fused only: rows whose run of equal scores reached past the kept entries (see there).
 *   counters[2..3]  reserved, 0.
 */
dba_status dba_counters(dba_handle* h, uint32_t counters[4]);

/* Number of kernels this handle has launched so far (for accounting in benchmarks). */
uint64_t dba_launch_count(const dba_handle* h);

/*
 * Testing aid (no step of the method): shortens the bounded device-side waits of the streaming row scan and
 * can make one of them run out, so that the DBA_ERR_TIMEOUT path can be exercised without any fault.
 *   wait_clocks  > 0: GPU clocks a wait may last before the kernel gives up (default: about a second)
 *   drop_item    >= 0: every thread block announces the copy of this item (a stretch of up to 44 KB of a row) of
 *                its sequence but does not issue it, so the wait for it runs out after wait_clocks; the kernel
 *                then records the failure and returns (nothing faults or hangs).  < 0: every copy is issued.
 * The fused projection (dba_step_fused, dba_project_scan) takes the same two: there the item is a 64-deep slice
 * of the operands in the sequence of the first thread block of every pair, which announces its copies of that
 * slice without issuing them; both blocks of the pair then give up at their next wait and leave together.
 * h == NULL sets the two for the stand-alone scans of this process (dba_row_scan, dba_row_scan_static,
 * dba_project_scan).
 */
dba_status dba_test_hook(dba_handle* h, int64_t wait_clocks, int32_t drop_item);

/* Frees the handle (not the workspace). NULL is allowed. */
void dba_destroy(dba_handle* h);

const char* dba_status_string(dba_status s);

/*
 * The first kernel of the step on its own (Section 2's row normaliser plus the ARGMAX_K of
 * Algorithm 1 restricted to single rows): for each of R rows of V logits, the log-sum-exp and the
 * n_top largest entries in order (value descending, lower index first among equals).
 *   row_lse_dev [R] fp32;  top_val_dev [R, n_top] fp32 (widened);  top_idx_dev [R, n_top] int32.
 * If V < n_top the tail is filled with (-inf, -1).  scratch_dev must hold dba_row_scan_scratch_bytes.
 * Enqueues on `cuda_stream`, does not synchronise.  n_top <= 66.
 * Failure of a device-side wait (a copy that never arrived; see DBA_ERR_TIMEOUT) cannot be returned by a call
 * that does not synchronise: in that case EVERY row's result is replaced by row_lse = NaN and a list of
 * (-inf, -1), which no successful scan produces (a row without finite entries has row_lse = -inf).
 */
dba_status dba_row_scan_scratch_bytes(int32_t R, int32_t V, int32_t n_top, int32_t logit_dtype, size_t* bytes);
dba_status dba_row_scan(const void* logits_dev, int32_t logit_dtype, int32_t R, int32_t V,
                        int64_t row_stride_elems, int32_t n_top, void* scratch_dev, size_t scratch_bytes,
                        float* row_lse_dev, float* top_val_dev, int32_t* top_idx_dev, void* cuda_stream);

/*
 * The row scan fused into the step before it (Section 2: the k x |V_T| matrix is the output of DECODER-STEP, whose
 * last stage multiplies the decoder's final hidden states by the output embedding).  logits[r, w] =
 * sum_j hidden[r, j] * embed[w, j] are computed on the tensor cores (bf16 operands, fp32 accumulation) and consumed
 * as they are produced: the R x V matrix is never written to memory.  Results as for dba_row_scan, for the logits so
 * defined (they agree with a double-precision evaluation of the inner products to within the rounding of an fp32
 * accumulation over D terms; where two logits are closer than that, their order in the list may differ from the
 * exactly evaluated one).
 *   hidden_dev [R, D] bf16, rows hidden_stride_elems apart;  embed_dev [V, D] bf16, rows embed_stride_elems apart;
 *   both 16-byte aligned with strides that are multiples of 8 elements; D a multiple of 8.  n_top <= 32.
 *   Other shapes: DBA_ERR_UNSUPPORTED.  scratch_dev must hold dba_project_scan_scratch_bytes (for the current device).
 * Enqueues on `cuda_stream`, does not synchronise.  A failed device-side wait, or a row of which 48 or more
 * logits within one stretch of the vocabulary (the part one thread works through: every other 256-word tile of
 * a run of up to 256 tiles) agree with its n_top-th largest value in sign, exponent and the leading 7 bits of
 * the mantissa, is reported as for dba_row_scan: every row's result is replaced by row_lse = NaN and a list of
 * (-inf, -1).
 */
dba_status dba_project_scan_scratch_bytes(int32_t R, int32_t V, int32_t n_top, size_t* bytes);
dba_status dba_project_scan(const void* hidden_dev, int64_t hidden_stride_elems, const void* embed_dev,
                            int64_t embed_stride_elems, int32_t R, int32_t V, int32_t D, int32_t n_top,
                            void* scratch_dev, size_t scratch_bytes, float* row_lse_dev, float* top_val_dev,
                            int32_t* top_idx_dev, void* cuda_stream);

/*
 * dba_row_scan for callers that cannot allocate device memory (the paper has no counterpart: this is a
 * packaging variant of the entry point above, not a step of the method).  Use it where cudaMalloc is not
 * an option: a serving process whose memory pool is fixed at start-up, a plug-in that receives buffers but
 * owns no allocator, a latency path that must not risk the device-wide synchronisation an allocation can
 * cause.  The scratch that dba_row_scan takes from the caller lives here in a fixed array inside the
 * library image: 4 MiB (dba_row_scan_static_max_bytes) on every GPU that loads the library, for as long as
 * the process runs.  Inputs, outputs and results are those of dba_row_scan.
 *   - A problem whose scratch need (dba_row_scan_scratch_bytes) exceeds the fixed size is refused with
 *     DBA_ERR_UNSUPPORTED and nothing is launched.
 *   - No device memory is allocated or freed, here or in anything this function calls.
 *   - The first call on each device looks up the array's device address (with that device current); make
 *     that first call outside any stream capture.
 *   - All calls on one device share the one array.  Each call overwrites what it later reads, so calls
 *     that follow one another on a stream are independent; calls that can overlap on the GPU (different
 *     streams, no ordering between them) race on it and give undefined results.
 */
dba_status dba_row_scan_static(const void* logits_dev, int32_t logit_dtype, int32_t R, int32_t V,
                               int64_t row_stride_elems, int32_t n_top, float* row_lse_dev,
                               float* top_val_dev, int32_t* top_idx_dev, void* cuda_stream);
size_t dba_row_scan_static_max_bytes(void);

#ifdef __cplusplus
}
#endif
#endif /* DBA_H */
