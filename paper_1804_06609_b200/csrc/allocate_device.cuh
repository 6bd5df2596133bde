// Allocation (Section 3.2: ALLOCATE of Algorithm 2, then newBeam; Section 4's pruning and stopping rule), the
// last part of a step: one warp per sentence, called by the candidate kernel once the sentence's candidates,
// grouped by bank and ordered inside each bank, are in shared memory.
#pragma once
#include "dba_device.cuh"
#include "dba_internal.h"

namespace dba {

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

// What the allocation reads of the candidate kernel's shared memory.
struct AllocIn {
    const int* bank_cnt;       // [C + 1] candidates per bank
    const int* order;          // [n] candidate ids in (bank asc, score desc, flat index asc) order
    const float* c_score;      // by candidate id
    const int* c_flat;
    const uint64_t* c_mask;
    const int* c_active;
    const int* par_kind;       // [k] of the current beam: 0 empty, 1 open, 2 finished
    const int* par_len;        // [k] generated tokens so far
};

// One warp.  Writes the sentence's new beam (and the requested outputs, the history, the stop bits) and appends
// its open rows to the list the next step's row scan reads (the order of that list varies from run to run; no
// result depends on it).
__device__ __forceinline__ void allocate_sentence(const Dims& d, int b, int C, const AllocIn& in, const Beam& nxt,
                                                  const dba_step_out& out,
                                                  int32_t* __restrict__ hist_bp, int32_t* __restrict__ hist_tok,
                                                  int32_t* __restrict__ open_list, int32_t* __restrict__ open_count) {
    __shared__ int n[kBanks];
    __shared__ int alloc[kBanks];
    __shared__ int off[kBanks];
    __shared__ int sel[kMaxK];
    __shared__ float a_score[kMaxK];
    __shared__ int a_flat[kMaxK];
    __shared__ int a_tok[kMaxK];
    __shared__ int a_h[kMaxK];
    __shared__ float a_val[kMaxK];     // what a hypothesis enters the pruning comparison with
    const int lane = threadIdx.x & 31;
    const int k = d.k, V = d.V;
    const int* bank_cnt = in.bank_cnt; const int* order = in.order;
    const float* c_score = in.c_score; const int* c_flat = in.c_flat;
    const uint64_t* c_mask = in.c_mask; const int* c_active = in.c_active;
    const int* par_kind = in.par_kind; const int* par_len = in.par_len;

    // Lane l looks after banks l, l + 32 and l + 64 (there are at most 65).
    // bank sizes; equal base share, remainder to the top bank C (Section 3.2); offsets of the banks inside the
    // bank-ordered candidate list
    const int share = k / (C + 1);
    int nq[3], aq[3];
#pragma unroll
    for (int j = 0; j < 3; ++j) {
        const int q = lane + 32 * j;
        nq[j] = q <= C ? bank_cnt[q] : 0;
        aq[j] = q <= C ? share + (q == C ? k - share * (C + 1) : 0) : 0;
    }
    {
        int run = 0;                                  // exclusive prefix of n over banks, 32 at a time
#pragma unroll
        for (int j = 0; j < 3; ++j) {
            if (32 * j > C) break;                    // (no banks up there)
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
            if (32 * j > C) break;
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
    // the selected cells: score, flat index, and (one division per cell) the row it extends and its token
    for (int i = lane; i < ns; i += 32) {
        const int id = order[sel[i]];
        const int fi = c_flat[id];
        const int h = fi / V;
        sel[i] = id; a_score[i] = c_score[id]; a_flat[i] = fi; a_h[i] = h; a_tok[i] = fi - h * V;
    }
    __syncwarp();
    // Section 4: threshold pruning.  Hypotheses whose value is below (best completed value - threshold) are
    // removed, completed or not, and the ones behind them move up.  The value is the cumulative score; with
    // DBA_FLAG_PRUNE_NORMALISED a completed hypothesis enters with score / length on both sides of the comparison.
    float cut = neg_inf();
    if (d.prune > 0.f) {
        float best = neg_inf();
        for (int i = lane; i < ns; i += 32) {
            const int h = a_h[i];
            float v = a_score[i];
            if (a_tok[i] == d.eos_id) {
                if (d.flags & DBA_FLAG_PRUNE_NORMALISED) {
                    const int len = par_kind[h] == 2 ? par_len[h] : par_len[h] + 1;
                    if (len > 0) v = __fdiv_rn(v, (float)len);
                }
                best = fmaxf(best, v);
            }
            a_val[i] = v;
        }
        best = warp_max(best);
        if (best != neg_inf()) cut = __fsub_rn(best, d.prune);
        __syncwarp();
    }
    const int r0 = b * k;
    const bool pruning = cut != neg_inf();
    // Who stays, who of those is completed; the places of the open ones in the list the next step's row scan reads
    // are reserved now (a round trip to memory that the ordering and the writes below cover).
    int n_live = 0, n_done = 0, n_open = 0, list_base = 0;
    for (int i0 = 0; i0 < ns; i0 += 32) {
        const int i = i0 + lane;
        const bool live = i < ns && !(pruning && a_val[i] < cut);
        const bool done = live && a_tok[i] == d.eos_id;
        n_live += __popc(__ballot_sync(kFullMask, live));
        n_done += __popc(__ballot_sync(kFullMask, done));
    }
    n_open = n_live - n_done;
    if (lane == 0 && n_open) list_base = atomicAdd(open_count, n_open);
    // new beam in decreasing score order, ties by lower flat index (Section 3.1), empty slots last
    static_assert(kMaxK <= 64, "a lane looks after at most two slots");
    int slot_open[2] = {-1, -1};        // per round of the loop below: the row this lane's open cell went to, else -1
#pragma unroll
    for (int rd = 0; rd < 2; ++rd) {
        const int i0 = 32 * rd;
        if (i0 >= k) break;
        const int i = i0 + lane;
        const bool live = i < ns && !(pruning && a_val[i] < cut);
        int rank = 0, w = 0;
        if (live) {
            const float si = a_score[i]; const int fi = a_flat[i];
            // (branch-free and unrolled: the loads of several rounds are in flight together)
            if (pruning) {
#pragma unroll 8
                for (int j = 0; j < ns; ++j) rank += (int)cell_better(a_score[j], a_flat[j], si, fi) & (int)!(a_val[j] < cut);
            } else {
#pragma unroll 8
                for (int j = 0; j < ns; ++j) rank += (int)cell_better(a_score[j], a_flat[j], si, fi);
            }
            const int id = sel[i];
            const uint64_t cmask = c_mask[id]; const int cactive = c_active[id];
            const int h = a_h[i];
            w = a_tok[i];
            const int r = r0 + rank;
            const int bank = __popcll(cmask);
            const int len = par_kind[h] == 2 ? par_len[h] : par_len[h] + 1;      // a finished hypothesis stays as long as it was
            nxt.score[r] = si; nxt.token[r] = w; nxt.mask[r] = cmask; nxt.active[r] = cactive; nxt.len[r] = len;
            nxt.bank[r] = bank; nxt.backptr[r] = h;
            hist_bp[r] = h; hist_tok[r] = w;
            if (out.backptr) out.backptr[r] = h;
            if (out.token) out.token[r] = w;
            if (out.score) out.score[r] = si;
            if (out.bank) out.bank[r] = bank;
            if (out.met_mask) out.met_mask[r] = cmask;
            if (out.active) out.active[r] = cactive;
        }
        if (live && w != d.eos_id) slot_open[rd] = r0 + rank;
    }
    for (int i = n_live + lane; i < k; i += 32) {
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
    // rows the next step has to scan: live slots that have not generated the end token.  (Last, so that the reply
    // to the reservation made above has had the whole of the beam's writing to arrive in.)
    {
        const int base = __shfl_sync(kFullMask, list_base, 0);
        int open_before = 0;
#pragma unroll
        for (int rd = 0; rd < 2; ++rd) {
            const unsigned bal = __ballot_sync(kFullMask, slot_open[rd] >= 0);
            if (slot_open[rd] >= 0) open_list[base + open_before + __popc(bal & ((1u << lane) - 1u))] = slot_open[rd];
            open_before += __popc(bal);
        }
    }
    // Section 4's stopping rule (everything on the beam completed) and Section 6.4's early stopping (something is)
    if (out.stop && lane == 0)
        out.stop[b] = (n_live > 0 && n_done == n_live ? DBA_STOP_ALL_COMPLETED : 0) | (n_done > 0 ? DBA_STOP_SOME_COMPLETED : 0);
}

}  // namespace dba
