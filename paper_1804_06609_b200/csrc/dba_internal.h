// Internal declarations shared by the translation units of libdba (not part of the public ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "dba.h"

namespace dba {

constexpr int kMaxK = 64;          // beam size limit
constexpr int kMaxC = 64;          // constraint tokens per sentence (one bit each in a 64-bit mask)
constexpr int kMaxTop = kMaxK + 2; // entries kept per row: k, one for a masked end token, one sentinel
constexpr int kMaxSeg = 8;         // row segments scanned by different CTAs: as far as short rows are split up
constexpr int kMaxSegLong = 24;    // segments of a row too long for kMaxSeg full-length segments (up to 1 MiB)

// device status word bits (sticky; read by dba_finalize)
constexpr uint32_t kStatusTimeout = 1u;    // a bounded wait on an mbarrier gave up
constexpr uint32_t kStatusOverflow = 2u;   // an internal list ran out of room (results of that step invalid)
// further words of the status block: counters (diagnostics, never an error)
constexpr int kStatusWordRescans = 1;      // stretches of rows the scan kernel had to rank from global memory again
constexpr int kStatusWordUnresolved = 2;   // fused step: rows whose equal scores ran past the row's list and could not be looked up
constexpr int kStatusWordTicket = 4;       // stand-alone row scan: the counter its CTAs draw their items from (cleared with the block)

// Per-sentence constraint table, phrases flattened to token positions 0..C-1 (Section 3 of the paper:
// the constraint count is the total number of tokens over all words and phrases).
struct SentCons {
    int32_t C;
    int32_t n_phrases;
    uint64_t first_mask;   // bit j: position j opens its word/phrase
    uint64_t last_mask;    // bit j: position j closes its word/phrase
    int32_t ctok[kMaxC];
    uint8_t pstart[kMaxC]; // first position of the phrase position j belongs to
    uint8_t prev_same[kMaxC]; // nearest earlier phrase-opening position with the same token (255: none)
};

// One beam (all sentences): arrays of R = B*k entries.
struct Beam {
    float* score;
    int32_t* token;
    uint64_t* mask;
    int32_t* active;
    int32_t* len;
    int32_t* bank;
    int32_t* backptr;
};

struct Dims {
    int32_t B, k, V, R;
    int32_t K1;        // entries kept per row by the scan kernel (k + 2)
    int32_t S;         // segments per row
    int32_t seg_len;   // elements per segment (multiple of the scan kernel's chunk)
    int32_t max_cand;  // candidate capacity per sentence
    int32_t pad_id, bos_id, eos_id;
    int32_t dtype;
    uint32_t flags;
    float prune;       // Section 4's pruning threshold (<= 0: off)
};

// Results of the row scan, per row.
struct RowTop {
    float* lse;        // [R] log-sum-exp of the row (-inf if it holds no finite value)
    float* val;        // [R*K1] the K1 largest entries, descending (ties: lower index first); (-inf, -1) padded
    int32_t* idx;      // [R*K1] column within the row
};

// Results of the streaming scan, one entry per (row, segment).  (m == nullptr where a kernel is told that the rows'
// finished results are in a RowTop instead.)
struct ScanScratch {
    float* m;          // [R*S] reference maximum of the segment (-inf if it holds no finite value)
    float* s;          // [R*S] sum of exp(x - m)
    float* val;        // [R*S*K1] values, descending (ties: lower index first); (-inf, -1) padded
    int32_t* idx;      // [R*S*K1] column within the row
};

// Partial results of the fused projection, per (row, piece): the piece's sum of exponentials against its whole-number
// reference, and its candidates for the row's K1 largest logits (unordered; cap = project_list_cap()).
struct ProjPieces {
    int32_t* ref;      // [R*P]
    float* sum;        // [R*P]
    int32_t* n;        // [R*P] candidates the piece holds
    float* val;        // [R*P*cap]
    int32_t* col;      // [R*P*cap]
    uint32_t* row_tau; // [R] the bound the row's pieces share while the kernel runs (an ordered integer; zeroed per launch)
};

// Testing aids of the streaming scan and of the fused projection (see dba_test_hook in dba.h).
struct ScanDebug {
    long long wait_clocks = 0;   // > 0: how many clocks a wait on an mbarrier may last
    int drop_item = -1;          // >= 0: every CTA (projection: the first of every pair) announces the copy of this item
                                 //       of its sequence but never issues it
};

// How the candidate kernel is launched for one handle: fixed at dba_init from the handle's own device.
struct CandLaunch {
    int threads = 0;
    size_t smem = 0;
};

// Launch with programmatic stream serialisation: the kernel may begin before the previous kernel of the
// stream has finished (see grid_dependency_wait in dba_device.cuh).
template <typename... Params, typename... Args>
inline cudaError_t launch_after(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);
}

// --- launchers (each enqueues on `st` and returns the CUDA error of the launch) ----------------------
// `open_score` / `open_token` (may be null): rows whose slot is empty (score -inf) or finished
// (token == eos) are skipped.
// `open_list` / `open_count` (may be null): the same set of rows as a compact list in device memory.
// `zero_count` (may be null): a counter the kernel sets to zero (the count of the list the step's last kernel
// builds for the next step: the two counts alternate).
cudaError_t launch_row_scan(const void* logits, int64_t stride, const Dims& d, const float* open_score,
                            const int32_t* open_token, const int32_t* open_list, const int32_t* open_count,
                            int32_t* zero_count, const RowTop& out, const ScanScratch& part, uint32_t* status,
                            int sm_count, const ScanDebug& dbg, cudaStream_t st, int* launches, bool* partial);
// (*partial: the streaming kernel ran and left per-segment results in `part`; otherwise the rows' finished results are in `out`)
// stand-alone merge of per-segment results into finished rows
cudaError_t launch_row_merge(const Dims& d, const ScanScratch& part, int n_top, float* row_lse, float* top_val,
                             int32_t* top_idx, cudaStream_t st, int* launches);
// streaming (TMA) version: usable when rows start on 16-byte boundaries and segments are whole chunks
bool row_scan_tma_usable(const void* logits, int64_t stride, const Dims& d);
cudaError_t configure_row_scan_tma();
cudaError_t launch_row_scan_tma(const void* logits, int64_t stride, const Dims& d, const int32_t* open_list,
                                const int32_t* open_count, int32_t* zero_count, const ScanScratch& part,
                                uint32_t* status, int sm_count, const ScanDebug& dbg, cudaStream_t st);
// Chooses S and seg_len for a row of V elements when R rows are scanned (fills d.S, d.seg_len, d.K1).
void plan_segments(Dims& d, int sm_count);
// The most segments plan_segments can choose for such rows: what the per-segment arrays are sized for.
int max_segments(int V, int dtype);
// Output projection fused with the row scan (hidden [R, D] and embed [V, D], bf16, row-major): tensor-core GEMM whose
// epilogue keeps per row the normaliser and the candidates, then an exact merge into the row scan's result format.
int project_pieces(int R, int V, int sm_count);       // pieces a row may have: the stride of ProjPieces
int project_list_cap();
bool project_scan_usable(const void* hidden, int64_t hidden_stride, const void* embed, int64_t embed_stride, int D, int K1);
cudaError_t configure_project_scan(int* max_pairs);      // *max_pairs: pairs of CTAs the device runs at once
cudaError_t launch_project_scan(const void* hidden, int64_t hidden_stride, const void* embed, int64_t embed_stride,
                                int R, int V, int D, int K1, const ProjPieces& pieces, int piece_stride,
                                const RowTop& top, uint32_t* status, int max_pairs, const ScanDebug& dbg, cudaStream_t st, int* launches);
// logits of every sentence's constraint tokens for its rows: out[r * 64 + j] = <hidden[r], embed[token j of the
// sentence of row r]> (fp32), for the fused step, which has no logit matrix to look them up in
cudaError_t launch_constraint_logits(const void* hidden, int64_t hidden_stride, const void* embed, int64_t embed_stride,
                                     int D, const Dims& d, const SentCons* cons, float* out, cudaStream_t st, int* launches);
// after a stand-alone scan: replaces the results by (NaN, -inf, -1) if the scan recorded a failed wait
cudaError_t launch_scan_check(const uint32_t* status, int R, int n_top, const RowTop& top, cudaStream_t st);
// candidates, allocation and the new beam (one kernel); appends the new beam's open rows to open_list / open_count
cudaError_t launch_candidates(const void* logits, int64_t stride, const Dims& d, const SentCons* cons,
                              const Beam& cur, const Beam& next, const RowTop& top, const ScanScratch& part,
                              const float* lse_in, const float* s2_given, const dba_step_out& out, int32_t* hist_bp, int32_t* hist_tok, uint32_t* status,
                              int32_t* open_list, int32_t* open_count, const CandLaunch& cl, cudaStream_t st,
                              int* launches);
cudaError_t launch_reset(const Dims& d, const Beam& beam, int32_t* open_list, int32_t* open_count,
                         const RowTop& top, cudaStream_t st, int* launches);
cudaError_t launch_finalize(const Dims& d, const Beam& beam, const int32_t* hist_bp, const int32_t* hist_tok,
                            int32_t steps, int32_t max_steps, int32_t* tokens, int32_t* len, float* score,
                            int32_t* flags, cudaStream_t st, int* launches);

// Chooses the block size and opts the candidate kernel in to the dynamic shared memory it needs on the current
// device.  *fits = false (and nothing configured) when even the smallest block is over the device's limit.
cudaError_t configure_candidates(const Dims& d, CandLaunch* cl, bool* fits);

}  // namespace dba
