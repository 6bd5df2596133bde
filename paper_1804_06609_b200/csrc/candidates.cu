// Candidate kernel (Algorithm 2; Section 3.1; Section 3.3's end-token rule), ending with the allocation of
// Section 3.2 (allocate_device.cuh) by one of its warps.
// One CTA per sentence.  Builds the candidate set from (1) the k best cells of the k x V score matrix,
// (2) every token that advances an open hypothesis through its constraints and (3) every live
// hypothesis' best token, updates the constraint marks of each candidate (unwinding a broken phrase),
// removes duplicates, and hands the candidates over grouped by bank and ordered inside each bank.
#include "allocate_device.cuh"
#include "dba_device.cuh"
#include "dba_internal.h"

namespace dba {

namespace {

constexpr int kCandMaxThreads = 1024;      // the host picks 1024, 640, 512 or 256 threads: the most whose scratch fits

struct Layout {   // byte offsets into dynamic shared memory
    int cons, parent, lse, mask, active, kind, eos_ok, plen, s2_x, rt_score, rt_w, rt_n, rt_ptr, s1_h, s1_i, stage, merged,
        tmp_score, tmp_w, tmp_x, c_score, c_flat, c_mask, c_active, order, bank_cnt, sort, total;
};

__host__ __device__ inline int align_up(int x, int a) { return (x + a - 1) / a * a; }

__host__ __device__ inline Layout make_layout(int k, int K1, int S, int max_cand, int n_warps) {
    Layout L;
    int o = 0;
    L.cons = o;      o = align_up(o + (int)sizeof(SentCons), 16);
    L.mask = o;      o += 8 * k;
    L.parent = o;    o += 4 * k;
    L.lse = o;       o += 4 * k;
    L.active = o;    o += 4 * k;
    L.kind = o;      o += 4 * k;
    L.eos_ok = o;    o += 4 * k;
    L.plen = o;      o += 4 * k;
    L.s2_x = o;      o += 4 * k * kMaxC;
    L.rt_score = o;  o += 4 * k * k;
    L.rt_w = o;      o += 4 * k * k;
    L.rt_n = o;      o += 4 * k;
    L.rt_ptr = o;    o += 4 * k;
    L.s1_h = o;      o += 4 * k;
    L.s1_i = o;      o += 4 * k;
    o = align_up(o, 8);
    L.stage = o;     o += 8 * n_warps * (S > 1 ? S * K1 : 0);
    L.merged = o;    o += 8 * n_warps * K1;
    L.tmp_score = o; o += 4 * n_warps * K1;
    L.tmp_w = o;     o += 4 * n_warps * K1;
    L.tmp_x = o;     o += 4 * n_warps * K1;
    o = align_up(o, 8);
    L.c_mask = o;    o += 8 * max_cand;
    L.c_score = o;   o += 4 * max_cand;
    L.c_flat = o;    o += 4 * max_cand;
    L.c_active = o;  o += 4 * max_cand;
    L.order = o;     o += 4 * max_cand;
    L.bank_cnt = o;  o += 4 * (kMaxC + 1);
    o = align_up(o, 16);
    L.sort = o;      o += 12 * max_cand;            // ordering keys (8 bytes) and ids (4 bytes) by grouped place
    L.total = o;
    return L;
}

// Merge of descending key lists of at most 32 entries each (key 0 = empty), one entry per lane: with the second
// list reversed, the lane-wise maximum holds the 32 largest of both as a bitonic sequence, which five
// compare-exchange steps put in descending order.
constexpr int kMergeWays = 4;       // warps that share the merge of the row lists (source 1)

__device__ __forceinline__ uint64_t merge_top32(uint64_t a, uint64_t b, int lane) {
    const uint64_t br = __shfl_sync(kFullMask, b, 31 - lane);
    uint64_t acc = a > br ? a : br;
#pragma unroll
    for (int str = 16; str; str >>= 1) {
        const uint64_t o = __shfl_xor_sync(kFullMask, acc, str);
        const bool upper = (lane & str) == 0;             // this lane keeps the larger of the pair
        acc = (o > acc) == upper ? o : acc;
    }
    return acc;
}

// 48 registers: two CTAs of 640 threads (a warp per row at k = 20) fit an SM.
__global__ void __maxnreg__(48)
candidates_kernel(const void* __restrict__ logits, int64_t stride, Dims d, const SentCons* __restrict__ cons,
                  Beam cur, Beam nxt, RowTop top, ScanScratch part, const float* __restrict__ lse_in,
                  const float* __restrict__ s2_given, dba_step_out out, int32_t* __restrict__ hist_bp, int32_t* __restrict__ hist_tok,
                  uint32_t* __restrict__ status, int32_t* __restrict__ open_list, int32_t* __restrict__ open_count) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int k = d.k, V = d.V, K1 = d.K1;
    const int S = part.m ? d.S : 0;     // > 0: the streaming scan left one partial result per (row, segment) in `part`;
                                        // 0: the row's finished list and normaliser are in `top`
    float* row_lse = top.lse;      // written by the row scan for open rows; set to 0 here for the others
    const int n_threads = blockDim.x, n_warps = n_threads >> 5;
    const Layout L = make_layout(k, K1, d.S, d.max_cand, n_warps);
    SentCons& sc = *reinterpret_cast<SentCons*>(smem + L.cons);
    uint64_t* s_mask = reinterpret_cast<uint64_t*>(smem + L.mask);
    float* s_parent = reinterpret_cast<float*>(smem + L.parent);
    float* s_lse = reinterpret_cast<float*>(smem + L.lse);
    int* s_active = reinterpret_cast<int*>(smem + L.active);
    int* s_kind = reinterpret_cast<int*>(smem + L.kind);      // 0 empty, 1 open, 2 finished
    int* s_eos_ok = reinterpret_cast<int*>(smem + L.eos_ok);
    int* s_plen = reinterpret_cast<int*>(smem + L.plen);
    int* s_order = reinterpret_cast<int*>(smem + L.order);   // candidate ids in (bank, score, flat index) order
    float* s2_x = reinterpret_cast<float*>(smem + L.s2_x);    // logit of the token at constraint position j of row h, if it advances h
    float* rt_score = reinterpret_cast<float*>(smem + L.rt_score);
    int* rt_w = reinterpret_cast<int*>(smem + L.rt_w);
    int* rt_n = reinterpret_cast<int*>(smem + L.rt_n);
    int* rt_ptr = reinterpret_cast<int*>(smem + L.rt_ptr);
    int* s1_h = reinterpret_cast<int*>(smem + L.s1_h);
    int* s1_i = reinterpret_cast<int*>(smem + L.s1_i);
    float* c_score = reinterpret_cast<float*>(smem + L.c_score);
    int* c_flat = reinterpret_cast<int*>(smem + L.c_flat);
    uint64_t* c_mask = reinterpret_cast<uint64_t*>(smem + L.c_mask);
    int* c_active = reinterpret_cast<int*>(smem + L.c_active);
    int* bank_cnt = reinterpret_cast<int*>(smem + L.bank_cnt);
    unsigned char* ent = smem + L.sort;
    __shared__ int s_ncand, s_ns1;
    __shared__ uint64_t s_part[kMergeWays][32];       // partial merges of source 1

    const int b = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int r0 = b * k;
    if (tid == 0) allow_dependents();

    // ---- load the sentence: constraint table and beam state --------------------------------------------
    {
        const uint32_t* src = reinterpret_cast<const uint32_t*>(cons + b);
        uint32_t* dst = reinterpret_cast<uint32_t*>(&sc);
        for (int i = tid; i < (int)(sizeof(SentCons) / 4); i += n_threads) dst[i] = src[i];
    }
    if (tid < k) {
        const float ps = cur.score[r0 + tid];
        const int tk = cur.token[r0 + tid];
        s_parent[tid] = ps;
        s_mask[tid] = cur.mask[r0 + tid];
        s_active[tid] = cur.active[r0 + tid];
        s_plen[tid] = cur.len[r0 + tid];
        s_kind[tid] = ps == neg_inf() ? 0 : (tk == d.eos_id ? 2 : 1);
        rt_ptr[tid] = 0;
        rt_n[tid] = 0;
    }
    if (tid <= kMaxC) bank_cnt[tid] = 0;
    if (tid == 0) { s_ncand = 0; s_ns1 = 0; }
    // Source 2's logits, fetched early: which tokens advance a hypothesis depends on the beam alone, and the
    // logits were there before the row scan started.  These are scattered reads of a matrix that has left the
    // L2 cache, the longest single latency of this kernel; here it overlaps the end of the row scan.
    __syncthreads();
    {
        const int C0 = sc.C;
        for (int h = warp; h < k; h += n_warps) {
            if (s_kind[h] != 1) continue;
            const uint64_t m = s_mask[h]; const int a = s_active[h];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int j = lane + 32 * q;
                bool ok = j < C0;
                if (ok) {
                    if (a >= 0) ok = j == a + 1;
                    else {
                        ok = ((sc.first_mask >> j) & 1ull) && !((m >> j) & 1ull);
                        // the same token may open an earlier word/phrase that is still unmet: then that one is listed
                        for (int e = ok ? sc.prev_same[j] : 255; e != 255; e = sc.prev_same[e])
                            if (!((m >> e) & 1ull)) { ok = false; break; }
                    }
                }
                // (with the projection fused into the step there is no logit matrix: the logits of the constraint
                //  tokens were computed on their own and are read further down, once they are there)
                s2_x[h * kMaxC + j] = !ok ? neg_inf() : logits ? load_logit_dyn(logits, d.dtype, (int64_t)(r0 + h) * stride + sc.ctok[j]) : 0.f;
            }
        }
    }
    // Up to here only what earlier steps left behind was read (the row scan waited for them before it let
    // this kernel start); from here on the row scan's own results are needed.
    const int C = sc.C;
    if (tid < k) s_eos_ok[tid] = __popcll(s_mask[tid]) >= C;   // Section 3.3: end token only once all are met
    grid_dependency_wait();
    if (!logits) {
        __syncthreads();
        for (int q = tid; q < k * kMaxC; q += n_threads) {
            const int h = q >> 6, j = q & 63;
            if (s_kind[h] == 1 && j < C && s2_x[q] != neg_inf()) s2_x[q] = s2_given[(int64_t)(r0 + h) * kMaxC + j];
        }
    }
    __syncthreads();

    // ---- phase A: per row, the k best cells in (score desc, token asc) order ------------------------------
    uint64_t* stage = reinterpret_cast<uint64_t*>(smem + L.stage) + warp * (d.S > 1 ? d.S * K1 : 0);
    uint64_t* merged = reinterpret_cast<uint64_t*>(smem + L.merged) + warp * K1;
    float* tmp_score = reinterpret_cast<float*>(smem + L.tmp_score) + warp * K1;
    int* tmp_w = reinterpret_cast<int*>(smem + L.tmp_w) + warp * K1;
    float* tmp_x = reinterpret_cast<float*>(smem + L.tmp_x) + warp * K1;
    const unsigned lt_mask = (1u << lane) - 1u;

    for (int h = warp; h < k; h += n_warps) {
        const int r = r0 + h;
        const int kind = s_kind[h];
        if (kind == 0) { if (lane == 0) { row_lse[r] = 0.f; s_lse[h] = 0.f; if (out.row_lse) out.row_lse[r] = 0.f; } continue; }
        if (kind == 2) {                      // finished: repeats the end token at an unchanged score
            if (lane == 0) { rt_n[h] = 1; rt_score[h * k] = s_parent[h]; rt_w[h * k] = d.eos_id; row_lse[r] = 0.f; s_lse[h] = 0.f; if (out.row_lse) out.row_lse[r] = 0.f; }
            continue;
        }
        float lse;
        float parent;
        bool eos_ok;
        if (S > 0) {
            // every global load of this row first (they are independent), so that their latencies overlap
            const int n_ent = S * K1;
            const float mg = lane < S ? part.m[r * S + lane] : neg_inf();
            const float sg = lane < S ? part.s[r * S + lane] : 0.f;
            const float lse_given = lse_in ? lse_in[r] : 0.f;
            {   // four loads of each array in flight before the first key is stored (the stores would hold them back)
                uint64_t* dst = S == 1 ? merged : stage;
                const int32_t* gi = part.idx + (int64_t)r * n_ent;
                const float* gv = part.val + (int64_t)r * n_ent;
                for (int e0 = lane; e0 < n_ent; e0 += 128) {
                    int ix[4]; float xv[4];
    #pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int e = e0 + 32 * q;
                        ix[q] = e < n_ent ? __ldg(gi + e) : -1;
                        xv[q] = e < n_ent ? __ldg(gv + e) : 0.f;
                    }
    #pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int e = e0 + 32 * q;
                        if (e < n_ent) dst[e] = ix[q] >= 0 ? row_key(xv[q], ix[q]) : 0ull;
                    }
                }
            }
            // row normaliser from the segment partials: lane g holds segment g (S <= 8), fixed reduction order
            {
                const float M = warp_max(mg);
                const float sum = warp_sum(mg != neg_inf() ? sg * expf(mg - M) : 0.f);
                lse = M == neg_inf() ? neg_inf() : M + logf(sum);
            }
            if (lane == 0) { row_lse[r] = lse; if (out.row_lse) out.row_lse[r] = lse; }
            if (lse_in) lse = lse_given;
            if (lane == 0) s_lse[h] = lse;
            parent = s_parent[h];
            eos_ok = s_eos_ok[h] != 0;

            // the row's K1 largest raw logits, merged over segments, as keys in `merged`
            if (S > 1) {
                const int n = n_ent;
                for (int e = lane; e < K1; e += 32) merged[e] = 0ull;
                __syncwarp();
                if (K1 <= 32) {
                    uint64_t acc = lane < K1 ? stage[lane] : 0ull;
                    for (int g = 1; g < S; ++g) acc = merge_top32(acc, lane < K1 ? stage[g * K1 + lane] : 0ull, lane);
                    if (lane < K1) merged[lane] = acc;
                } else
                // every segment's list is in descending key order (empty entries, key 0, last): the place of an
                // entry in the merged order is its place in its own list plus, for every other list, the number of
                // keys above it, found by bisection
                for (int e = lane; e < n; e += 32) {
                    const uint64_t key = stage[e];
                    if (!key) continue;
                    const int g = e / K1;
                    int rank = e - g * K1;
                    for (int g2 = 0; g2 < S; ++g2) {
                        if (g2 == g) continue;
                        const uint64_t* lst = stage + g2 * K1;
                        int lo2 = 0, hi2 = K1;                      // first position whose key is not above `key`
                        while (lo2 < hi2) { const int mid = (lo2 + hi2) >> 1; if (lst[mid] > key) lo2 = mid + 1; else hi2 = mid; }
                        rank += lo2;
                    }
                    if (rank < K1) merged[rank] = key;
                }
            }
            __syncwarp();
        } else {
            // the row's K1 largest raw logits (the finished list) as keys in `merged`, and its normaliser
            lse = row_lse[r];
            if (lane == 0 && out.row_lse) out.row_lse[r] = lse;
            const float lse_given = lse_in ? lse_in[r] : 0.f;
            const int32_t* gi = top.idx + (int64_t)r * K1;
            const float* gv = top.val + (int64_t)r * K1;
            for (int e = lane; e < K1; e += 32) {
                const int ix = gi[e];
                const float xv = gv[e];
                merged[e] = ix >= 0 ? row_key(xv, ix) : 0ull;
            }
            if (lse_in) lse = lse_given;
            if (lane == 0) s_lse[h] = lse;
            parent = s_parent[h];
            eos_ok = s_eos_ok[h] != 0;
            __syncwarp();
        }

        // scores of the entries that may be generated, in list order
        int total_valid = 0, finite_entries = 0;
        for (int e0 = 0; e0 < K1; e0 += 32) {
            const int e = e0 + lane;
            bool valid = false, finite = false; float scv = neg_inf(), x = neg_inf(); int w = -1;
            if (e < K1) {
                const uint64_t key = merged[e];
                if (key) {
                    x = row_key_val(key);
                    w = row_key_idx(key);
                    finite = x != neg_inf();
                    valid = finite && !(w == d.eos_id && !eos_ok) && lse != neg_inf();
                    if (valid) scv = cell_score(x, lse, parent);
                }
            }
            const unsigned bal = __ballot_sync(kFullMask, valid);
            const int pos = total_valid + __popc(bal & lt_mask);
            if (valid) { tmp_score[pos] = scv; tmp_w[pos] = w; tmp_x[pos] = x; }
            total_valid += __popc(bal);
            finite_entries += __popc(__ballot_sync(kFullMask, finite));
        }
        __syncwarp();
        // The list is ordered by raw logit, the beam by score, and distinct logits can round to one score.
        // m = how many list entries compete for the row's k places: k, unless the k-th score continues
        // past the cut, in which case every entry of that run competes (lowest token ids win).
        int m = min(total_valid, k);
        if (total_valid > k && tmp_score[k] == tmp_score[k - 1]) {
            const float sb = tmp_score[k - 1];
            int g = k - 1, e = k;
            while (g > 0 && tmp_score[g - 1] == sb) --g;
            while (e + 1 < total_valid && tmp_score[e + 1] == sb) ++e;
            m = e + 1;
            // If the run reaches the end of a full list, cells outside the list may belong to it.  They
            // cannot precede the listed ones when the whole run is one logit value (the list holds that
            // value's lowest ids) and the next lower representable logit already scores below the run.
            const bool open_end = e == total_valid - 1 && finite_entries == K1;
            bool rescan = false;
            if (open_end) {
                const float xl = tmp_x[e];
                uint32_t bits = __float_as_uint(xl);
                const uint32_t ulp = d.dtype == DBA_BF16 ? 0x10000u : 1u;
                if ((bits << 1) == 0) bits = 0x80000000u | ulp;
                else bits = (bits & 0x80000000u) ? bits + ulp : bits - ulp;
                rescan = !(tmp_x[g] == xl && cell_score(__uint_as_float(bits), lse, parent) < sb);
            }
            if (rescan && !logits) {       // no logit matrix to look into: the listed entries stand (counted, see dba_counters)
                if (lane == 0) atomicAdd(status + kStatusWordUnresolved, 1u);
                rescan = false;
            }
            if (rescan) {      // whole row: the cells scoring exactly sb, lowest token ids first
                const int need = k - g;
                int found = 0;
                __syncwarp();
                for (int base = 0; base < V && found < need; base += 32) {
                    const int w = base + lane;
                    bool hit = false;
                    if (w < V) {
                        const float x = load_logit_dyn(logits, d.dtype, (int64_t)r * stride + w);
                        hit = x != neg_inf() && !(w == d.eos_id && !eos_ok) && cell_score(x, lse, parent) == sb;
                    }
                    const unsigned bal = __ballot_sync(kFullMask, hit);
                    const int pos = found + __popc(bal & lt_mask);
                    if (hit && pos < need) { tmp_score[g + pos] = sb; tmp_w[g + pos] = w; }
                    found += __popc(bal);
                }
                m = k;
                __syncwarp();
            }
        }
        // order by (score desc, token asc), keep the first k and publish
        const int nrow = min(m, k);
        bool ordered = m <= 32;                               // common case: already in (score desc, token asc) order
        if (ordered) {
            const bool bad = lane + 1 < m && !cell_better(tmp_score[lane], tmp_w[lane], tmp_score[lane + 1], tmp_w[lane + 1]);
            ordered = !__any_sync(kFullMask, bad);
        }
        if (ordered) {
            if (lane < nrow) { rt_score[h * k + lane] = tmp_score[lane]; rt_w[h * k + lane] = tmp_w[lane]; }
        } else
        for (int i = lane; i < m; i += 32) {
            const float si = tmp_score[i]; const int wi = tmp_w[i];
            int rank = 0;
            for (int j = 0; j < m; ++j) rank += cell_better(tmp_score[j], tmp_w[j], si, wi);
            if (rank < k) { rt_score[h * k + rank] = si; rt_w[h * k + rank] = wi; }
        }
        if (lane == 0) rt_n[h] = nrow;
        __syncwarp();
    }
    __syncthreads();

    // ---- phase B (source 1): the k best cells of the whole matrix -----------------------------------------------
    const int src1_warps = k <= 32 ? kMergeWays : 1;          // warps busy with source 1; the others take source 2
    if (warp < kMergeWays && k <= 32) {
        // Every row's list is in (score desc, token asc) order and at most 32 long: lists are merged, one entry
        // per lane, with the bitonic top-32 merge -- every kMergeWays-th row by one of kMergeWays warps, then the
        // partial results by the first of them; the first k of the result are the k best cells.
        // Keys: ordered score above, inverted flat index below (larger = better).
        uint64_t acc = 0;
        for (int h = warp; h < k; h += kMergeWays) {
            const uint64_t key = lane < rt_n[h]
                ? ((uint64_t)ord32(rt_score[h * k + lane]) << 32) | (uint32_t)(0xffffffffu - (uint32_t)(h * V + rt_w[h * k + lane]))
                : 0ull;
            acc = h == warp ? key : merge_top32(acc, key, lane);
        }
        s_part[warp][lane] = acc;
        asm volatile("bar.sync 1, %0;" ::"n"(kMergeWays * 32) : "memory");      // these warps only
        if (warp == 0) {
#pragma unroll
            for (int w = 1; w < kMergeWays; ++w) acc = merge_top32(acc, s_part[w][lane], lane);
            const bool have = lane < k && acc != 0ull;
            const unsigned sel_mask = __ballot_sync(kFullMask, have);
            const int flat = (int)(0xffffffffu - (uint32_t)acc);
            const int h = have ? flat / V : -1 - lane;                       // (lanes without a cell match nobody)
            // a row's cells are taken in its list's order: the cell's place in its row's list is the number of selected
            // cells of the same row before it
            const unsigned same = __match_any_sync(kFullMask, h) & sel_mask;
            if (have) {
                s1_h[lane] = h; s1_i[lane] = __popc(same & lt_mask);
                atomicMax(&rt_ptr[h], __popc(same));
            }
            if (lane == 0) s_ns1 = __popc(sel_mask);
        }
    } else if (warp == 0) {
        // (beams wider than 32: a k-round tournament of row heads)
        // lane l holds the heads of rows l and l + 32: ordered score key and flat index of the best unused cell
        uint32_t ks[2]; int fl[2], ptr[2] = {0, 0};
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const int h = lane + 32 * q;
            const bool has = h < k && rt_n[h] > 0;
            ks[q] = has ? ord32(rt_score[h * k]) : 0u;            // 0 is below every real key
            fl[q] = has ? h * V + rt_w[h * k] : 0x7fffffff;
        }
        int ns1 = 0;
        for (int round = 0; round < k; ++round) {
            // best head: highest score key, then lowest flat index
            const int q = (ks[1] > ks[0] || (ks[1] == ks[0] && fl[1] < fl[0])) ? 1 : 0;
            const uint32_t kmax = __reduce_max_sync(kFullMask, q ? ks[1] : ks[0]);
            if (kmax == 0u) break;
            const int mine = (q ? ks[1] : ks[0]) == kmax ? (q ? fl[1] : fl[0]) : 0x7fffffff;
            const int fmin = __reduce_min_sync(kFullMask, mine);
            if (mine == fmin) {                                    // exactly one lane: flat indices are distinct
                const int h = lane + 32 * q;
                s1_h[ns1] = h; s1_i[ns1] = q ? ptr[1] : ptr[0];
                const int np = (q ? ptr[1] : ptr[0]) + 1;
                const bool has = np < rt_n[h];
                const uint32_t nk = has ? ord32(rt_score[h * k + np]) : 0u;
                const int nf = has ? h * V + rt_w[h * k + np] : 0x7fffffff;
                if (q) { ptr[1] = np; ks[1] = nk; fl[1] = nf; } else { ptr[0] = np; ks[0] = nk; fl[0] = nf; }
                rt_ptr[h] = np;
            }
            ++ns1;
        }
        if (lane == 0) s_ns1 = ns1;
    } else {
        // ---- source 2, meanwhile, on the other warps (a row per warp): for every open hypothesis the tokens that
        //      raise its met count by one.  They all land in the same bank, so of one row at most k can ever be
        //      kept: with more, only the row's k best go on (the rest could not be selected; the bank still
        //      counts at least k candidates, which is all the allocation needs to know).
        for (int h = warp - src1_warps; h < k; h += n_warps - src1_warps) {
            if (s_kind[h] != 1) continue;
            const uint64_t m = s_mask[h];
            const float lse = s_lse[h], parent = s_parent[h];
            float sc2[2]; int w2[2], j2[2]; bool v2[2];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int j = lane + 32 * q;
                const float x = s2_x[h * kMaxC + j];          // -inf unless the token at position j advances h
                v2[q] = j < C && lse != neg_inf() && x != neg_inf();
                w2[q] = v2[q] ? sc.ctok[j] : 0x7fffffff;
                sc2[q] = v2[q] ? cell_score(x, lse, parent) : neg_inf();
                j2[q] = j;
            }
            const unsigned b0 = __ballot_sync(kFullMask, v2[0]), b1 = __ballot_sync(kFullMask, v2[1]);
            int cnt = __popc(b0) + __popc(b1);
            if (cnt > k) {                                    // keep the row's k best (score desc, token asc)
                int rank[2] = {0, 0};
                for (int o = 0; o < 32; ++o)
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        const float os = __shfl_sync(kFullMask, sc2[q], o); const int ow = __shfl_sync(kFullMask, w2[q], o);
                        rank[0] += cell_better(os, ow, sc2[0], w2[0]); rank[1] += cell_better(os, ow, sc2[1], w2[1]);
                    }
                v2[0] = v2[0] && rank[0] < k; v2[1] = v2[1] && rank[1] < k;
                cnt = k;
            }
            const unsigned k0 = __ballot_sync(kFullMask, v2[0]), k1 = __ballot_sync(kFullMask, v2[1]);
            int base = 0;
            if (lane == 0 && cnt) { base = atomicAdd(&s_ncand, cnt); atomicAdd(&bank_cnt[__popcll(m) + 1], cnt); }
            base = __shfl_sync(kFullMask, base, 0);
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int slot = base + (q ? __popc(k0) : 0) + __popc((q ? k1 : k0) & lt_mask);
                if (v2[q] && slot < d.max_cand) {
                    const int j = j2[q];
                    c_score[slot] = sc2[q]; c_flat[slot] = h * V + w2[q]; c_mask[slot] = m | (1ull << j);
                    c_active[slot] = ((sc.last_mask >> j) & 1ull) ? -1 : j;
                }
            }
        }
    }
    __syncthreads();

    // ---- sources 1 and 3 with their updated constraint marks; cells that advance a hypothesis through
    //      its constraints are left to source 2, which lists every such cell (no duplicates arise) ----------
    const int ns1 = s_ns1;
    // constraints[h].add(w) (Section 3.1, last paragraph) for these at most 2k cells: continue the begun phrase
    // if w is its next token; otherwise reset that phrase's marks and let w open the first wholly unmet
    // word/phrase it matches.  The scan over the constraint positions is spread over the CTA.
    // Step 1: continue the begun phrase, or unwind it; note the marks that remain.
    __shared__ uint64_t a_mask[2 * kMaxK];     // marks after a possible unwind (before w opens anything)
    __shared__ int a_w[2 * kMaxK];             // the token, -1: no cell / nothing to look for
    __shared__ int a_pos[2 * kMaxK];           // lowest position w can open (64: none)
    for (int t = tid; t < 2 * k; t += n_threads) {
        int h, i; bool have = true;
        if (t < k) { have = t < ns1; h = have ? s1_h[t] : 0; i = have ? s1_i[t] : 0; }
        else { h = t - k; i = 0; have = rt_n[h] != 0 && rt_ptr[h] == 0; }      // else: best cell already in source 1
        a_pos[t] = 64; a_w[t] = -1;
        if (have && s_kind[h] == 1) {
            const int w = rt_w[h * k + i];
            uint64_t m = s_mask[h]; const int a = s_active[h];
            if (a >= 0 && w != sc.ctok[a + 1]) {                                 // the begun phrase is broken: unwind
                const int p0 = sc.pstart[a];
                m &= ~(((2ull << a) - 1ull) & ~((1ull << p0) - 1ull));
            }
            a_mask[t] = m;
            if (!(a >= 0 && w == sc.ctok[a + 1])) a_w[t] = w;                    // otherwise it simply continues
        }
    }
    __syncthreads();
    // Step 2: the first wholly unmet word/phrase that w opens, if any.
    for (int q = tid; q < 2 * k * kMaxC; q += n_threads) {
        const int t = q >> 6, j = q & 63;
        const int w = a_w[t];
        if (w >= 0 && j < C && sc.ctok[j] == w && ((sc.first_mask & ~a_mask[t]) >> j) & 1ull) atomicMin(&a_pos[t], j);
    }
    __syncthreads();
    // Step 3: finish the update; cells that raise the met count belong to source 2 and are skipped here.
    for (int t = tid; t < 2 * k; t += n_threads) {
        int h, i;
        if (t < k) { if (t >= ns1) continue; h = s1_h[t]; i = s1_i[t]; }
        else { h = t - k; i = 0; if (rt_n[h] == 0 || rt_ptr[h] > 0) continue; }
        const int w = rt_w[h * k + i];
        uint64_t m = s_mask[h]; int a = s_active[h];
        if (s_kind[h] == 1) {
            const int before = __popcll(m);
            if (a >= 0 && w == sc.ctok[a + 1]) {
                const int nn = a + 1;
                m |= 1ull << nn; a = ((sc.last_mask >> nn) & 1ull) ? -1 : nn;
            } else {
                m = a_mask[t]; a = -1;
                const int j = a_pos[t];
                if (j < 64) { m |= 1ull << j; a = ((sc.last_mask >> j) & 1ull) ? -1 : j; }
            }
            if (__popcll(m) == before + 1) continue;
        }
        const int slot = atomicAdd(&s_ncand, 1);
        if (slot < d.max_cand) {
            c_score[slot] = rt_score[h * k + i]; c_flat[slot] = h * V + w; c_mask[slot] = m; c_active[slot] = a;
            atomicAdd(&bank_cnt[__popcll(m)], 1);
        }
    }
    __syncthreads();
    int n = s_ncand;
    if (n > d.max_cand) { if (tid == 0) atomicOr(status, kStatusOverflow); n = d.max_cand; }

    // ---- group by bank, order inside each bank (Section 3.1): order (bank asc, score desc, flat asc) ---------
    // Banks first (their sizes are known: a counting sort), then every candidate finds its place inside its bank
    // by counting the bank's candidates that precede it: the work grows with the size of the banks, not with the
    // number of candidates, and the result does not depend on the order in which the candidates were appended.
    __shared__ int bank_off[kMaxC + 1];        // where each bank starts in the grouped order
    __shared__ int bank_cur[kMaxC + 1];
    uint64_t* gkey = reinterpret_cast<uint64_t*>(ent);                 // by grouped place: ordering key (smaller = earlier)
    uint32_t* gid = reinterpret_cast<uint32_t*>(gkey + d.max_cand);    //                   candidate id | bank << 16
    if (warp == 0) {
        int run = 0;
#pragma unroll
        for (int j = 0; j < 3; ++j) {
            const int q = lane + 32 * j;
            const int c = q <= C ? bank_cnt[q] : 0;
            int incl = c;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(kFullMask, incl, o); if (lane >= o) incl += t; }
            if (q <= C) { bank_off[q] = run + incl - c; bank_cur[q] = 0; }
            run += __shfl_sync(kFullMask, incl, 31);
        }
    }
    __syncthreads();
    for (int i = tid; i < n; i += n_threads) {
        const int bk = __popcll(c_mask[i]);
        const int at = min(bank_off[bk] + atomicAdd(&bank_cur[bk], 1), d.max_cand - 1);
        gkey[at] = ((uint64_t)(0xffffffffu - ord32(c_score[i])) << 32) | (uint32_t)c_flat[i];
        gid[at] = (uint32_t)i | ((uint32_t)bk << 16);
    }
    __syncthreads();
    {
        // `split` neighbouring lanes share one candidate's count when there are threads to spare (chosen pass by
        // pass: the few candidates left for a last pass are counted by eight lanes each, not by one warp alone)
        for (int base = 0, per_pass = 0; base < n; base += per_pass) {
            int split = 1;
            while (split < 8 && 2 * split * (n - base) <= n_threads) split <<= 1;
            per_pass = n_threads / split;
            const int at = base + tid / split, part = tid & (split - 1);
            int rank = 0, lo = 0;
            uint32_t id = 0;
            if (at < n) {
                const uint64_t mine = gkey[at];
                id = gid[at];
                const int bk = (int)(id >> 16);
                lo = bank_off[bk];
                const int nb = min(bank_cnt[bk], n - lo);
                const int chunk = (nb + split - 1) / split;
                const int j1 = min(nb, (part + 1) * chunk);
#pragma unroll 4
                for (int j = part * chunk; j < j1; ++j) rank += gkey[lo + j] < mine;
            }
            for (int o = 1; o < split; o <<= 1) rank += __shfl_xor_sync(kFullMask, rank, o);
            if (at < n && part == 0) s_order[min(lo + rank, d.max_cand - 1)] = (int)(id & 0xffffu);
        }
    }
    // ---- ALLOCATE and the new beam (Section 3.2), by one warp ---------------------------------------------
    __syncthreads();
    if (warp == 0) {
        AllocIn in;
        in.bank_cnt = bank_cnt; in.order = s_order; in.c_score = c_score; in.c_flat = c_flat; in.c_mask = c_mask;
        in.c_active = c_active; in.par_kind = s_kind; in.par_len = s_plen;
        allocate_sentence(d, b, C, in, nxt, out, hist_bp, hist_tok, open_list, open_count);
    }
}

}  // namespace

// Threads per CTA: 1024 when every sentence gets an SM of its own (then only the latency of one CTA counts);
// otherwise two CTAs share an SM: 640 threads when the beam has more than 15 rows (a warp per row up to k = 20
// in the phase that works row by row), else 512; fewer if the per-warp scratch would not fit shared memory.
static int pick_threads(const Dims& d, size_t smem_limit, int sm_count) {
    const int first = d.B <= sm_count ? kCandMaxThreads : (d.k > 15 ? 640 : 512);
    for (int t = first; t > 256; t = t == 640 ? 512 : t >> 1)
        if ((size_t)make_layout(d.k, d.K1, d.S, d.max_cand, t / 32).total <= smem_limit) return t;
    return 256;
}

// The dynamic shared memory a block may ask for is the device's opt-in limit less what the kernel declares
// statically.  *fits = false (and nothing configured) when even the smallest block is over it.
cudaError_t configure_candidates(const Dims& d, CandLaunch* cl, bool* fits) {
    int dev = 0, lim = 0, sms = 1;
    *fits = false;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&lim, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaFuncAttributes fa{};
    if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa, candidates_kernel);
    if (e != cudaSuccess) return e;
    const size_t smem_limit = (size_t)lim > fa.sharedSizeBytes ? (size_t)lim - fa.sharedSizeBytes : 0;
    if ((size_t)make_layout(d.k, d.K1, d.S, d.max_cand, 256 / 32).total > smem_limit) return cudaSuccess;
    *fits = true;
    cl->threads = pick_threads(d, smem_limit, sms);
    cl->smem = (size_t)make_layout(d.k, d.K1, d.S, d.max_cand, cl->threads / 32).total;
    // The attribute belongs to the kernel, not to a handle: it is raised to the most any shape may ask for, so
    // that handles of different shapes can be alive together.
    return cudaFuncSetAttribute(candidates_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_limit);
}

cudaError_t launch_candidates(const void* logits, int64_t stride, const Dims& d, const SentCons* cons,
                              const Beam& cur, const Beam& next, const RowTop& top, const ScanScratch& part,
                              const float* lse_in, const float* s2_given, const dba_step_out& out, int32_t* hist_bp, int32_t* hist_tok, uint32_t* status,
                              int32_t* open_list, int32_t* open_count, const CandLaunch& cl, cudaStream_t st,
                              int* launches) {
    ++*launches;
    return launch_after(candidates_kernel, dim3(d.B), dim3(cl.threads), cl.smem, st, logits, stride, d, cons, cur, next,
                        top, part, lse_in, s2_given, out, hist_bp, hist_tok, status, open_list, open_count);
}

}  // namespace dba
