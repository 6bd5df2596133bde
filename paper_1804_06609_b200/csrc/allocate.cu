// The small kernels that reset the beam (Algorithm 1, DECODER-INIT) and pick / trace back the final
// hypothesis (Section 3.3).
#include "dba_device.cuh"
#include "dba_internal.h"

namespace dba {

namespace {

// Algorithm 1, DECODER-INIT: slot 0 holds the start symbol at score 0, the other slots are empty.
__global__ void reset_kernel(Dims d, Beam beam, int32_t* __restrict__ open_list, int32_t* __restrict__ open_count,
                             RowTop top) {
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= d.R) return;
    // the row lists start out empty and well-formed, so that a scan that fails (a wait that ran out) leaves the
    // candidate kernel nothing it could misread
    top.lse[r] = 0.f;
    for (int e = 0; e < d.K1; ++e) { top.val[(int64_t)r * d.K1 + e] = neg_inf(); top.idx[(int64_t)r * d.K1 + e] = -1; }
    const bool first = (r % d.k) == 0;
    beam.score[r] = first ? 0.f : neg_inf();
    beam.token[r] = first ? d.bos_id : d.pad_id;
    beam.mask[r] = 0; beam.active[r] = -1; beam.len[r] = 0; beam.bank[r] = first ? 0 : -1; beam.backptr[r] = 0;
    if (first) open_list[r / d.k] = r;
    if (r == 0) { open_count[0] = d.B; open_count[1] = 0; open_count[2] = 0; open_count[3] = 0; }   // counts of open rows, the row scan's work counters
}

// Section 3.3: the completed hypothesis with the highest score (Section 4: optionally divided by its
// length); if none is completed, the best live slot of the highest occupied bank.  One thread per sentence.
__global__ void finalize_kernel(Dims d, Beam beam, const int32_t* __restrict__ hist_bp,
                                const int32_t* __restrict__ hist_tok, int steps, int max_steps,
                                int32_t* __restrict__ tokens, int32_t* __restrict__ len_out,
                                float* __restrict__ score_out, int32_t* __restrict__ flags_out) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= d.B) return;
    const int k = d.k, r0 = b * k;
    int pick = -1; float val = 0.f;
    for (int h = 0; h < k; ++h) {
        const float s = beam.score[r0 + h];
        if (s == neg_inf() || beam.token[r0 + h] != d.eos_id) continue;
        float v = s;
        const int L = beam.len[r0 + h];
        if ((d.flags & DBA_FLAG_LENGTH_NORM) && L > 0) v = __fdiv_rn(s, (float)L);
        if (pick < 0 || v > val) { pick = h; val = v; }
    }
    const bool completed = pick >= 0;
    if (!completed) {
        int best_bank = -1;
        for (int h = 0; h < k; ++h) {
            const float s = beam.score[r0 + h];
            if (s == neg_inf()) continue;
            const int bk = __popcll(beam.mask[r0 + h]);
            if (bk > best_bank || (bk == best_bank && s > val)) { best_bank = bk; pick = h; val = s; }
        }
    }
    int32_t* out = tokens + (int64_t)b * max_steps;
    for (int t = 0; t < max_steps; ++t) out[t] = d.pad_id;
    flags_out[b] = completed ? 1 : 0;
    score_out[b] = pick < 0 ? neg_inf() : val;
    if (pick < 0 || steps == 0) { len_out[b] = 0; return; }
    int slot = pick;
    for (int t = steps - 1; t >= 0; --t) {        // walk the back-pointers, writing tokens in place
        out[t] = hist_tok[(int64_t)t * d.R + r0 + slot];
        slot = min(max(hist_bp[(int64_t)t * d.R + r0 + slot], 0), k - 1);   // a record is a slot number; never trusted as an index
    }
    int n = 0;
    while (n < steps) { ++n; if (out[n - 1] == d.eos_id) break; }
    for (int t = n; t < steps; ++t) out[t] = d.pad_id;
    len_out[b] = n;
}

}  // namespace

cudaError_t launch_reset(const Dims& d, const Beam& beam, int32_t* open_list, int32_t* open_count,
                         const RowTop& top, cudaStream_t st, int* launches) {
    reset_kernel<<<(d.R + 255) / 256, 256, 0, st>>>(d, beam, open_list, open_count, top);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_finalize(const Dims& d, const Beam& beam, const int32_t* hist_bp, const int32_t* hist_tok,
                            int32_t steps, int32_t max_steps, int32_t* tokens, int32_t* len, float* score,
                            int32_t* flags, cudaStream_t st, int* launches) {
    finalize_kernel<<<(d.B + 127) / 128, 128, 0, st>>>(d, beam, hist_bp, hist_tok, steps, max_steps, tokens, len,
                                                       score, flags);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace dba
