// Allocation kernel (Section 3.2: ALLOCATE of Algorithm 2, then newBeam), one warp per sentence; plus the
// small kernels that reset the beam and pick / trace back the final hypothesis (Section 3.3).
#include "dba_device.cuh"
#include "dba_internal.h"

namespace dba {

namespace {

constexpr int kAllocWarps = 1;       // sentences per CTA
constexpr int kBanks = kMaxC + 1;

// Nearest bank above / below b whose bit is set in the 65-bit set (lo: banks 0..63, hi: bank 64); -1 if none.
__device__ __forceinline__ int next_above(uint64_t lo, bool hi, int b) {
    if (b < 63) {
        const uint64_t m = lo & ~((2ull << b) - 1ull);
        if (m) return __ffsll((long long)m) - 1;
    }
    return (hi && b < 64) ? 64 : -1;
}
__device__ __forceinline__ int next_below(uint64_t lo, int b) {
    const uint64_t m = b >= 64 ? lo : (lo & ((1ull << b) - 1ull));
    return m ? 63 - __clzll((long long)m) : -1;
}

__global__ void __launch_bounds__(kAllocWarps * 32)
allocate_kernel(Dims d, const SentCons* __restrict__ cons, Beam cur, Beam nxt, const Cand* __restrict__ cand,
                const int32_t* __restrict__ ncand, const int32_t* __restrict__ bank_count,
                const float* __restrict__ row_lse, dba_step_out out, int32_t* __restrict__ hist_bp,
                int32_t* __restrict__ hist_tok, int32_t* __restrict__ open_list, int32_t* __restrict__ open_count) {
    __shared__ int s_n[kAllocWarps][kBanks];
    __shared__ int s_alloc[kAllocWarps][kBanks];
    __shared__ int s_off[kAllocWarps][kBanks];
    __shared__ int s_sel[kAllocWarps][kMaxK];
    __shared__ float s_score[kAllocWarps][kMaxK];
    __shared__ int s_flat[kAllocWarps][kMaxK];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.x * kAllocWarps + warp;
    if (threadIdx.x == 0) allow_dependents();
    grid_dependency_wait();      // the candidates come from the kernel before
    if (b >= d.B) return;
    const int k = d.k, V = d.V;
    const int C = cons[b].C;
    int* n = s_n[warp]; int* alloc = s_alloc[warp]; int* off = s_off[warp]; int* sel = s_sel[warp];

    // Lane l looks after banks l, l + 32 and l + 64 (there are at most 65).
    // bank sizes; equal base share, remainder to the top bank C (Section 3.2); offsets of the banks inside the
    // bank-ordered candidate list
    const int share = k / (C + 1);
    int nq[3], aq[3];
#pragma unroll
    for (int j = 0; j < 3; ++j) {
        const int q = lane + 32 * j;
        nq[j] = q <= C ? bank_count[b * kBanks + q] : 0;
        aq[j] = q <= C ? share + (q == C ? k - share * (C + 1) : 0) : 0;
    }
    {
        int run = 0;                                  // exclusive prefix of n over banks, 32 at a time
#pragma unroll
        for (int j = 0; j < 3; ++j) {
            int incl = nq[j];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(kFullMask, incl, o); if (lane >= o) incl += t; }
            const int q = lane + 32 * j;
            if (q <= C) { off[q] = run + incl - nq[j]; n[q] = nq[j]; }
            run += __shfl_sync(kFullMask, incl, 31);
        }
    }
    if (d.flags & DBA_FLAG_ADJUST_OFF) {
#pragma unroll
        for (int j = 0; j < 3; ++j) { const int q = lane + 32 * j; if (q <= C) alloc[q] = min(aq[j], nq[j]); }
        __syncwarp();
    } else {
        // Adjustment: every bank with more slots than candidates passes the surplus to the nearest banks that
        // have more candidates than slots, the higher one first at equal distance.  The sets of such banks are
        // bit masks (banks 0..63 in a 64-bit word, bank 64 apart); the walk itself is short and serial.
        const unsigned o0 = __ballot_sync(kFullMask, aq[0] > nq[0]), o1 = __ballot_sync(kFullMask, aq[1] > nq[1]);
        const unsigned d0 = __ballot_sync(kFullMask, nq[0] > aq[0]), d1 = __ballot_sync(kFullMask, nq[1] > aq[1]);
        const bool over_hi = __any_sync(kFullMask, lane == 0 && aq[2] > nq[2]);
        bool need_hi = __any_sync(kFullMask, lane == 0 && nq[2] > aq[2]);
        const uint64_t over_lo = (uint64_t)o0 | ((uint64_t)o1 << 32);
        uint64_t need_lo = (uint64_t)d0 | ((uint64_t)d1 << 32);
#pragma unroll
        for (int j = 0; j < 3; ++j) { const int q = lane + 32 * j; if (q <= C) alloc[q] = aq[j]; }
        __syncwarp();
        if (lane == 0) {
            uint64_t todo = over_lo;
            bool todo_hi = over_hi;
            while (todo || todo_hi) {
                int q;
                if (todo) { q = __ffsll((long long)todo) - 1; todo &= todo - 1; } else { q = 64; todo_hi = false; }
                int surplus = alloc[q] - n[q];
                alloc[q] = n[q];
                while (surplus > 0) {
                    const int up = next_above(need_lo, need_hi, q);
                    const int dn = next_below(need_lo, q);
                    int r;
                    if (up < 0 && dn < 0) break;
                    if (up >= 0 && (dn < 0 || up - q <= q - dn)) r = up; else r = dn;
                    const int g = min(surplus, n[r] - alloc[r]);
                    alloc[r] += g; surplus -= g;
                    if (alloc[r] == n[r]) { if (r < 64) need_lo &= ~(1ull << r); else need_hi = false; }
                }
            }
        }
        __syncwarp();
    }
    // the best alloc[q] candidates of every bank (they are ordered inside the bank already)
    int ns_total;
    {
        int run = 0;
#pragma unroll
        for (int j = 0; j < 3; ++j) {
            const int q = lane + 32 * j;
            const int a = q <= C ? alloc[q] : 0;
            int incl = a;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(kFullMask, incl, o); if (lane >= o) incl += t; }
            const int first = run + incl - a;
            for (int i = 0; i < a; ++i) sel[first + i] = off[q] + i;
            run += __shfl_sync(kFullMask, incl, 31);
        }
        ns_total = run;
    }
    __syncwarp();
    if (lane == 0) off[0] = ns_total;   // (kept where the code below reads it)
    __syncwarp();
    const int ns = off[0];
    const Cand* cb = cand + (int64_t)b * d.max_cand;
    for (int i = lane; i < ns; i += 32) { s_score[warp][i] = cb[sel[i]].score; s_flat[warp][i] = cb[sel[i]].flat; }
    __syncwarp();
    // Section 4: threshold pruning.  Hypotheses scoring below (best completed score - threshold) are removed,
    // completed or not; they are the tail of the ordered beam, so their slots are simply left empty.
    float cut = neg_inf();
    if (d.prune > 0.f) {
        float best = neg_inf();
        for (int i = lane; i < ns; i += 32) {
            const int fi = s_flat[warp][i];
            if (fi - (fi / V) * V == d.eos_id) best = fmaxf(best, s_score[warp][i]);
        }
        best = warp_max(best);
        if (best != neg_inf()) cut = __fsub_rn(best, d.prune);
    }
    // new beam in decreasing score order, ties by lower flat index (Section 3.1), empty slots last
    const int r0 = b * k;
    int n_pruned = 0;
    for (int i0 = 0; i0 < ns; i0 += 32) n_pruned += __popc(__ballot_sync(kFullMask, i0 + lane < ns && s_score[warp][i0 + lane] < cut));
    for (int i = lane; i < k; i += 32) {
        if (i < ns && !(s_score[warp][i] < cut)) {
            const float si = s_score[warp][i]; const int fi = s_flat[warp][i];
            int rank = 0;
            for (int j = 0; j < ns; ++j) rank += cell_better(s_score[warp][j], s_flat[warp][j], si, fi);
            const Cand c = cb[sel[i]];
            const int h = fi / V, w = fi - h * V;
            const int r = r0 + rank;
            const int bank = __popcll(c.mask);
            const int plen = cur.len[r0 + h];
            const int len = cur.token[r0 + h] == d.eos_id ? plen : plen + 1;
            nxt.score[r] = si; nxt.token[r] = w; nxt.mask[r] = c.mask; nxt.active[r] = c.active; nxt.len[r] = len;
            nxt.bank[r] = bank; nxt.backptr[r] = h;
            hist_bp[r] = h; hist_tok[r] = w;
            if (out.backptr) out.backptr[r] = h;
            if (out.token) out.token[r] = w;
            if (out.score) out.score[r] = si;
            if (out.bank) out.bank[r] = bank;
            if (out.met_mask) out.met_mask[r] = c.mask;
            if (out.active) out.active[r] = c.active;
        }
    }
    for (int i = ns - n_pruned + lane; i < k; i += 32) {
        const int r = r0 + i;
        nxt.score[r] = neg_inf(); nxt.token[r] = d.pad_id; nxt.mask[r] = 0; nxt.active[r] = -1; nxt.len[r] = 0;
        nxt.bank[r] = -1; nxt.backptr[r] = 0;
        hist_bp[r] = 0; hist_tok[r] = d.pad_id;
        if (out.backptr) out.backptr[r] = 0;
        if (out.token) out.token[r] = d.pad_id;
        if (out.score) out.score[r] = neg_inf();
        if (out.bank) out.bank[r] = -1;
        if (out.met_mask) out.met_mask[r] = 0;
        if (out.active) out.active[r] = -1;
    }
    if (out.row_lse)
        for (int i = lane; i < k; i += 32) out.row_lse[r0 + i] = row_lse[r0 + i];
    // rows the next step has to scan: live slots that have not generated the end token
    __syncwarp();
    int n_live = 0, n_done = 0;
    for (int i0 = 0; i0 < k; i0 += 32) {
        const int i = i0 + lane;
        const bool live = i < k && nxt.score[r0 + i] != neg_inf();
        const bool open = live && nxt.token[r0 + i] != d.eos_id;
        n_live += __popc(__ballot_sync(kFullMask, live));
        n_done += __popc(__ballot_sync(kFullMask, live && !open));
        const unsigned bal = __ballot_sync(kFullMask, open);
        int base = 0;
        if (lane == 0 && bal) base = atomicAdd(open_count, __popc(bal));
        base = __shfl_sync(kFullMask, base, 0);
        if (open) open_list[base + __popc(bal & ((1u << lane) - 1u))] = r0 + i;
    }
    // Section 4's stopping rule (everything on the beam completed) and Section 6.4's early stopping (something is)
    if (out.stop && lane == 0)
        out.stop[b] = (n_live > 0 && n_done == n_live ? DBA_STOP_ALL_COMPLETED : 0) | (n_done > 0 ? DBA_STOP_SOME_COMPLETED : 0);
}

// Algorithm 1, DECODER-INIT: slot 0 holds the start symbol at score 0, the other slots are empty.
__global__ void reset_kernel(Dims d, Beam beam, int32_t* __restrict__ open_list, int32_t* __restrict__ open_count) {
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= d.R) return;
    const bool first = (r % d.k) == 0;
    beam.score[r] = first ? 0.f : neg_inf();
    beam.token[r] = first ? d.bos_id : d.pad_id;
    beam.mask[r] = 0; beam.active[r] = -1; beam.len[r] = 0; beam.bank[r] = first ? 0 : -1; beam.backptr[r] = 0;
    if (first) open_list[r / d.k] = r;
    if (r == 0) *open_count = d.B;
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
        slot = hist_bp[(int64_t)t * d.R + r0 + slot];
    }
    int n = 0;
    while (n < steps) { ++n; if (out[n - 1] == d.eos_id) break; }
    for (int t = n; t < steps; ++t) out[t] = d.pad_id;
    len_out[b] = n;
}

}  // namespace

cudaError_t launch_allocate(const Dims& d, const SentCons* cons, const Beam& cur, const Beam& next,
                            const Cand* cand, const int32_t* ncand, const int32_t* bank_count,
                            const float* row_lse, const dba_step_out& out, int32_t* hist_bp, int32_t* hist_tok,
                            int32_t* open_list, int32_t* open_count, cudaStream_t st, int* launches) {
    ++*launches;
    return launch_after(allocate_kernel, dim3((d.B + kAllocWarps - 1) / kAllocWarps), dim3(kAllocWarps * 32), 0, st,
                        d, cons, cur, next, cand, ncand, bank_count, row_lse, out, hist_bp, hist_tok, open_list, open_count);
}

cudaError_t launch_reset(const Dims& d, const Beam& beam, int32_t* open_list, int32_t* open_count,
                         cudaStream_t st, int* launches) {
    reset_kernel<<<(d.R + 255) / 256, 256, 0, st>>>(d, beam, open_list, open_count);
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
