// Row scan, streaming version for sm_100a: one HBM pass per row.
//
// A persistent CTA per SM works through (row, segment) items.  Three roles, all synchronised with mbarriers:
//   producer   one thread issues bulk asynchronous copies (TMA, cp.async.bulk) of 8 KB chunks of the row into
//              a ring of shared-memory stages;
//   consumers  stream every chunk once: exp2 of (x - reference) summed per lane (Section 2's normaliser), and
//              a per-lane running maximum; no selection logic in this loop;
//   selectors  one item behind: from the consumers' lane maxima they take a lower bound of the K1-th largest
//              entry (the K1-th largest of 256 disjoint group maxima is one), pass over the item's chunks
//              again while they are still in shared memory, collect the few entries at or above the bound,
//              order them exactly (value descending, lower index first) and write the segment's partial
//              result; only then are the stages handed back to the producer.
// Every wait is bounded: a wait that runs out sets the timeout bit of the status word and the CTA winds down.
#include <cuda_bf16.h>

#include "dba_device.cuh"
#include "dba_internal.h"

namespace dba {

namespace {

constexpr int kChunkBytes = 8192;
constexpr int kStages = 24;                 // 192 KB of ring
constexpr int kMaxSegChunks = 8;            // a segment is at most 64 KB
constexpr int kNC = 8;                      // consumer warps
constexpr int kNS = 4;                      // selector warps
constexpr int kThreads = 32 * (1 + kNC + kNS);
constexpr int kConsThreads = 32 * kNC;
constexpr int kSelThreads = 32 * kNS;
constexpr int kSlots = 4;                   // items whose lane maxima may be pending at once
constexpr int kCandCap = 1024;              // entries at or above the bound that one item may hold
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr float kLog2e = 1.44269502162933349609375f;        // fl32(log2(e))
constexpr double kLn2 = 0.69314718055994530942;

struct Smem {
    alignas(128) unsigned char ring[kStages][kChunkBytes];
    alignas(8) uint64_t full[kStages];
    uint64_t empty[kStages];
    uint64_t item_done[kSlots];
    uint64_t slot_free[kSlots];
    uint64_t cand[kCandCap];
    float lane_max[kSlots][kConsThreads];
    float warp_sum[kSlots][kNC];
    float warp_ref[kSlots][kNC];            // the constant c of exp2(x*log2e - c) each warp ended with
    int hist1[256];
    int hist2[256];
    int sel_b1, sel_rank, sel_thr_ord;
    int cand_count;
    int abort_flag;
    uint64_t red[kNS];
};

struct Params {
    const void* logits;
    int64_t stride;             // elements
    int V, S, seg_len, K1;
    int R;
    const int32_t* open_list;   // rows to scan (null: all R rows)
    const int32_t* open_count;  // number of entries of open_list (device memory)
    float* part_m; float* part_s; float* top_val; int32_t* top_idx;
    uint32_t* status;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the CTA is winding down (this wait ran out, or another one did).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 255u) == 255u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void sel_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kSelThreads) : "memory"); }
// Barrier of the selector group that also ORs a flag over its threads: every thread gets the same answer.
__device__ __forceinline__ bool sel_barrier_or(int flag) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.s32 q, %1, 0;\n\tbar.red.or.pred p, 1, %2, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r) : "r"(flag), "n"(kSelThreads) : "memory");
    return r != 0;
}
__device__ __forceinline__ float ex2(float t) { float r; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(t)); return r; }
__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
    uint32_t r; asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b)); return r;
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

template <typename T> struct Vec;
template <> struct Vec<float> {
    static constexpr int kElems = 4;
    static __device__ __forceinline__ float vmax(const uint4& v) {
        return fmaxf(fmaxf(__uint_as_float(v.x), __uint_as_float(v.y)), fmaxf(__uint_as_float(v.z), __uint_as_float(v.w)));
    }
    static __device__ __forceinline__ void unpack(const uint4& v, float* x) {
        x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y); x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
    }
};
template <> struct Vec<__nv_bfloat16> {
    static constexpr int kElems = 8;
    static __device__ __forceinline__ float vmax(const uint4& v) {
        const uint32_t m = max_bf16x2(max_bf16x2(v.x, v.y), max_bf16x2(v.z, v.w));
        return fmaxf(bf16_lo(m), bf16_hi(m));
    }
    static __device__ __forceinline__ void unpack(const uint4& v, float* x) {
        x[0] = bf16_lo(v.x); x[1] = bf16_hi(v.x); x[2] = bf16_lo(v.y); x[3] = bf16_hi(v.y);
        x[4] = bf16_lo(v.z); x[5] = bf16_hi(v.z); x[6] = bf16_lo(v.w); x[7] = bf16_hi(v.w);
    }
};

// Walks the items of this CTA in the order all three roles agree on.
struct ItemIter {
    int item, n_items, S;
    const int32_t* open_list;
    __device__ ItemIter(const Params& p) : S(p.S), open_list(p.open_list) {
        const int rows = p.open_count ? *p.open_count : p.R;
        n_items = rows * p.S;
        item = blockIdx.x;
    }
    __device__ bool valid() const { return item < n_items; }
    __device__ void next() { item += gridDim.x; }
    __device__ int row() const { const int i = item / S; return open_list ? open_list[i] : i; }
    __device__ int seg() const { return item % S; }
};

template <typename T>
__global__ void __launch_bounds__(kThreads, 1) row_scan_tma_kernel(Params p) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
    constexpr int kElems = Vec<T>::kElems;
    constexpr int kChunkElems = kChunkBytes / (int)sizeof(T);
    constexpr int kChunkVecs = kChunkBytes / 16;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int* abort_flag = &sm.abort_flag;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&sm.full[s]), 1); mbar_init(smem_u32(&sm.empty[s]), kNS); }
        for (int s = 0; s < kSlots; ++s) { mbar_init(smem_u32(&sm.item_done[s]), kNC); mbar_init(smem_u32(&sm.slot_free[s]), 1); }
        sm.cand_count = 0; sm.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i < 256; i += kThreads) { sm.hist1[i] = 0; sm.hist2[i] = 0; }
    __syncthreads();

    const int seg_bytes_full = p.seg_len * (int)sizeof(T);
    const int row_bytes = p.V * (int)sizeof(T);

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t fills = 0;
            bool ok = true;
            for (ItemIter it(p); ok && it.valid(); it.next()) {
                const int seg = it.seg();
                const char* src = (const char*)p.logits + ((int64_t)it.row() * p.stride + (int64_t)seg * p.seg_len) * (int64_t)sizeof(T);
                int left = min(seg_bytes_full, row_bytes - seg * seg_bytes_full);
                while (left > 0) {
                    const int bytes = min(left, kChunkBytes);
                    const uint32_t st = fills % kStages, ph = (fills / kStages) & 1u;
                    if (!mbar_wait(smem_u32(&sm.empty[st]), ph ^ 1u, abort_flag)) { ok = false; break; }
                    mbar_expect_tx(smem_u32(&sm.full[st]), (uint32_t)bytes);
                    bulk_load(smem_u32(sm.ring[st]), src, (uint32_t)bytes, smem_u32(&sm.full[st]));
                    src += bytes; left -= bytes; ++fills;
                }
            }
            if (!ok) {   // winding down: let the copies already issued land before the CTA leaves
                const uint32_t first = fills > kStages ? fills - kStages : 0;
                for (uint32_t f = first; f < fills; ++f) {
                    const uint32_t st = f % kStages, ph = (f / kStages) & 1u;
                    for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(smem_u32(&sm.full[st]), ph); ++i) {}
                }
            }
        }
        __syncwarp();
    } else if (warp <= kNC) {
        // ------------------------------------------------------------------ consumers
        const int cw = warp - 1, ctid = cw * 32 + lane;
        uint32_t fills = 0, n_item = 0;
        bool ok = true;
        for (ItemIter it(p); ok && it.valid(); it.next(), ++n_item) {
            const int seg = it.seg();
            const int bytes_item = min(seg_bytes_full, row_bytes - seg * seg_bytes_full);
            const uint32_t slot = n_item % kSlots, slot_ph = (n_item / kSlots) & 1u;
            float ssum = 0.f, lmax = neg_inf();
            float ref = 0.f, negc = 0.f;          // exp2(x*log2e + negc); ref = the value negc was made from
            bool have_ref = false;
            for (int done = 0; done < bytes_item; done += kChunkBytes, ++fills) {
                const int bytes = min(kChunkBytes, bytes_item - done);
                const uint32_t st = fills % kStages, ph = (fills / kStages) & 1u;
                if (!__all_sync(kFullMask, mbar_wait(smem_u32(&sm.full[st]), ph, abort_flag))) { ok = false; break; }
                const uint4* vec = reinterpret_cast<const uint4*>(sm.ring[st]);
                const int nvec = bytes >> 4;
                uint4 v0 = make_uint4(0, 0, 0, 0), v1 = v0;
                const bool h0 = ctid < nvec, h1 = ctid + kConsThreads < nvec;
                if (h0) v0 = vec[ctid];
                if (h1) v1 = vec[ctid + kConsThreads];
                float m2 = neg_inf();
                if (h0) m2 = Vec<T>::vmax(v0);
                if (h1) m2 = fmaxf(m2, Vec<T>::vmax(v1));
                lmax = fmaxf(lmax, m2);
                // keep the exponent argument well inside fp32 range: move the reference up when needed
                if (__any_sync(kFullMask, have_ref ? m2 > ref + 32.f : m2 > neg_inf())) {
                    float nm = warp_max(m2);
                    if (have_ref) { nm = fmaxf(nm, ref); ssum *= ex2((ref - nm) * kLog2e); }
                    ref = nm; negc = -(nm * kLog2e); have_ref = true;
                }
                float x[kElems];
                if (h0) {
                    Vec<T>::unpack(v0, x);
#pragma unroll
                    for (int e = 0; e < kElems; ++e) ssum += ex2(fmaf(x[e], kLog2e, negc));
                }
                if (h1) {
                    Vec<T>::unpack(v1, x);
#pragma unroll
                    for (int e = 0; e < kElems; ++e) ssum += ex2(fmaf(x[e], kLog2e, negc));
                }
            }
            if (!ok) break;
            // hand the lane maxima and the warp's sum to the selectors
            if (!__all_sync(kFullMask, mbar_wait(smem_u32(&sm.slot_free[slot]), slot_ph ^ 1u, abort_flag))) break;
            sm.lane_max[slot][ctid] = lmax;
            const float wsum = warp_sum(ssum);
            if (lane == 0) { sm.warp_sum[slot][cw] = wsum; sm.warp_ref[slot][cw] = -negc; }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm.item_done[slot]));
        }
    } else {
        // ------------------------------------------------------------------ selectors
        const int sw = warp - 1 - kNC, stid = sw * 32 + lane;
        uint32_t fills = 0, n_item = 0;
        bool ok = true;
        for (ItemIter it(p); ok && it.valid(); it.next(), ++n_item) {
            const int row = it.row(), seg = it.seg();
            const int bytes_item = min(seg_bytes_full, row_bytes - seg * seg_bytes_full);
            const uint32_t slot = n_item % kSlots, slot_ph = (n_item / kSlots) & 1u;
            const int64_t out = (int64_t)row * p.S + seg;
            mbar_wait(smem_u32(&sm.item_done[slot]), slot_ph, abort_flag);
            if (sel_barrier_or(*abort_flag)) { ok = false; break; }      // one answer for the whole group

            // ---- bound: the K1-th largest of the 256 lane maxima, to 16 bits of the ordered key ----
            uint32_t key[kConsThreads / kSelThreads];
#pragma unroll
            for (int q = 0; q < kConsThreads / kSelThreads; ++q) {
                key[q] = ord32(sm.lane_max[slot][stid + q * kSelThreads]);
                atomicAdd(&sm.hist1[key[q] >> 24], 1);
            }
            if (stid == 0) {   // the segment's normaliser parts, combined in double
                double C = -1e300;
                for (int w = 0; w < kNC; ++w) C = fmax(C, (double)sm.warp_ref[slot][w]);
                double S = 0.0;
                for (int w = 0; w < kNC; ++w) S += (double)sm.warp_sum[slot][w] * exp2((double)sm.warp_ref[slot][w] - C);
                // sum_x 2^(x*log2e) = S * 2^C  ->  (m, s) with sum_x e^x = s * e^m
                float m = (float)(C * kLn2);
                float s = (float)(S * exp(C * kLn2 - (double)m));
                if (S == 0.0) { m = neg_inf(); s = 0.f; }
                p.part_m[out] = m; p.part_s[out] = s;
            }
            sel_barrier();
            if (sw == 0) {     // highest 8-bit digit whose suffix count reaches K1
                int c[8], tot = 0;
#pragma unroll
                for (int j = 0; j < 8; ++j) { c[j] = sm.hist1[lane * 8 + j]; tot += c[j]; }
                int suf = tot;                                  // inclusive suffix over lanes
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_down_sync(kFullMask, suf, o); if (lane + o < 32) suf += t; }
                const int above = suf - tot;                    // count in lanes above this one
                int run = above, b1 = -1, rank = 0;
#pragma unroll
                for (int j = 7; j >= 0; --j) { if (b1 < 0 && run + c[j] >= p.K1) { b1 = lane * 8 + j; rank = p.K1 - run; } run += c[j]; }
                const unsigned hit = __ballot_sync(kFullMask, b1 >= 0);
                const int src = hit ? 31 - __clz(hit) : 0;      // the highest lane that found it
                b1 = __shfl_sync(kFullMask, b1, src); rank = __shfl_sync(kFullMask, rank, src);
                if (lane == 0) { sm.sel_b1 = hit ? b1 : 0; sm.sel_rank = hit ? rank : 1; }
#pragma unroll
                for (int j = 0; j < 8; ++j) sm.hist1[lane * 8 + j] = 0;
            }
            sel_barrier();
            const int b1 = sm.sel_b1;
#pragma unroll
            for (int q = 0; q < kConsThreads / kSelThreads; ++q)
                if ((int)(key[q] >> 24) == b1) atomicAdd(&sm.hist2[(key[q] >> 16) & 255u], 1);
            sel_barrier();
            if (sw == 0) {
                const int want = sm.sel_rank;
                int c[8], tot = 0;
#pragma unroll
                for (int j = 0; j < 8; ++j) { c[j] = sm.hist2[lane * 8 + j]; tot += c[j]; }
                int suf = tot;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_down_sync(kFullMask, suf, o); if (lane + o < 32) suf += t; }
                int run = suf - tot, b2 = -1;
#pragma unroll
                for (int j = 7; j >= 0; --j) { if (b2 < 0 && run + c[j] >= want) b2 = lane * 8 + j; run += c[j]; }
                const unsigned hit = __ballot_sync(kFullMask, b2 >= 0);
                const int src = hit ? 31 - __clz(hit) : 0;
                b2 = __shfl_sync(kFullMask, b2, src);
                if (lane == 0) sm.sel_thr_ord = (int)(((uint32_t)b1 << 24) | ((uint32_t)(hit ? b2 : 0) << 16));
#pragma unroll
                for (int j = 0; j < 8; ++j) sm.hist2[lane * 8 + j] = 0;
            }
            sel_barrier();
            float thr = unord32((uint32_t)sm.sel_thr_ord);
            if (!(thr == thr)) thr = neg_inf();          // the bucket that holds -inf has no finite lower edge
            // the consumers may reuse this slot from here on
            if (stid == 0) mbar_arrive(smem_u32(&sm.slot_free[slot]));

            // ---- second look at the item's chunks: everything at or above the bound ----
            const int elem0 = seg * p.seg_len;
            int chunk = 0;
            for (int done = 0; done < bytes_item; done += kChunkBytes, ++fills, ++chunk) {
                const int bytes = min(kChunkBytes, bytes_item - done);
                const uint32_t st = fills % kStages, ph = (fills / kStages) & 1u;
                mbar_wait(smem_u32(&sm.full[st]), ph, abort_flag);   // complete already: the consumers waited on it
                const uint4* vec = reinterpret_cast<const uint4*>(sm.ring[st]);
                const int nvec = bytes >> 4;
#pragma unroll
                for (int q = 0; q < kChunkVecs / kSelThreads; ++q) {
                    const int vi = stid + q * kSelThreads;
                    if (vi < nvec) {
                        const uint4 v = vec[vi];
                        if (Vec<T>::vmax(v) >= thr) {
                            float x[kElems];
                            Vec<T>::unpack(v, x);
                            const int base = elem0 + chunk * kChunkElems + vi * kElems;
#pragma unroll
                            for (int e = 0; e < kElems; ++e)
                                if (x[e] >= thr) {
                                    const int pos = atomicAdd(&sm.cand_count, 1);
                                    if (pos < kCandCap) sm.cand[pos] = row_key(x[e], base + e);
                                }
                        }
                    }
                }
            }
            sel_barrier();       // the stages are released below, once it is known whether they are still needed
            const int n = sm.cand_count;
            const uint32_t fills_end = fills;
            const int n_chunks = chunk;
            float* tv = p.top_val + out * p.K1;
            int32_t* ti = p.top_idx + out * p.K1;
            if (n <= kCandCap) {
                // release the stages first, the ordering below only needs the candidate list
                if (lane == 0)
                    for (int c2 = 0; c2 < n_chunks; ++c2) mbar_arrive(smem_u32(&sm.empty[(fills_end - n_chunks + c2) % kStages]));
                for (int i = stid; i < p.K1; i += kSelThreads) if (i >= n) { tv[i] = neg_inf(); ti[i] = -1; }
                for (int i = stid; i < n; i += kSelThreads) {
                    const uint64_t ki = sm.cand[i];
                    int rank = 0;
                    for (int j = 0; j < n; ++j) rank += sm.cand[j] > ki;
                    if (rank < p.K1) { tv[rank] = row_key_val(ki); ti[rank] = row_key_idx(ki); }
                }
            } else {
                // too many entries at or above the bound (long runs of equal values, or an adversarial
                // layout): take the K1 best one at a time from the chunks, which are still resident
                uint64_t prev = ~0ull;
                for (int r2 = 0; r2 < p.K1; ++r2) {
                    uint64_t best = 0;
                    for (int c2 = 0; c2 < n_chunks; ++c2) {
                        const uint32_t st = (fills_end - n_chunks + c2) % kStages;
                        const int bytes = min(kChunkBytes, bytes_item - c2 * kChunkBytes);
                        const uint4* vec = reinterpret_cast<const uint4*>(sm.ring[st]);
                        for (int vi = stid; vi < (bytes >> 4); vi += kSelThreads) {
                            float x[kElems];
                            Vec<T>::unpack(vec[vi], x);
                            const int base = elem0 + c2 * kChunkElems + vi * kElems;
#pragma unroll
                            for (int e = 0; e < kElems; ++e) {
                                const uint64_t kk = row_key(x[e], base + e);
                                if (kk < prev && kk > best) best = kk;
                            }
                        }
                    }
                    best = warp_max_u64(best);
                    if (lane == 0) sm.red[sw] = best;
                    sel_barrier();
                    best = sm.red[0];
#pragma unroll
                    for (int w = 1; w < kNS; ++w) best = sm.red[w] > best ? sm.red[w] : best;
                    sel_barrier();
                    if (stid == 0) { tv[r2] = best ? row_key_val(best) : neg_inf(); ti[r2] = best ? row_key_idx(best) : -1; }
                    prev = best;      // 0 once exhausted: nothing is below it
                }
                if (lane == 0)
                    for (int c2 = 0; c2 < n_chunks; ++c2) mbar_arrive(smem_u32(&sm.empty[(fills_end - n_chunks + c2) % kStages]));
            }
            sel_barrier();
            if (stid == 0) sm.cand_count = 0;
            sel_barrier();
        }
    }
    __syncthreads();
    if (tid == 0 && sm.abort_flag) atomicOr(p.status, kStatusTimeout);
}

}  // namespace

bool row_scan_tma_usable(const void* logits, int64_t stride, const Dims& d) {
    const int es = d.dtype == DBA_F32 ? 4 : 2;
    if (((uintptr_t)logits & 15u) || ((stride * es) & 15) || ((d.V * es) & 15)) return false;
    if ((d.seg_len * es) % kChunkBytes != 0 || d.seg_len * es > kMaxSegChunks * kChunkBytes) return false;
    return true;
}

size_t row_scan_tma_smem() { return sizeof(Smem) + 128; }

cudaError_t configure_row_scan_tma() {
    cudaError_t e = cudaFuncSetAttribute(row_scan_tma_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)row_scan_tma_smem());
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(row_scan_tma_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)row_scan_tma_smem());
}

cudaError_t launch_row_scan_tma(const void* logits, int64_t stride, const Dims& d, const int32_t* open_list,
                                const int32_t* open_count, const ScanOut& out, uint32_t* status, int sm_count,
                                cudaStream_t st) {
    Params p;
    p.logits = logits; p.stride = stride; p.V = d.V; p.S = d.S; p.seg_len = d.seg_len; p.K1 = d.K1; p.R = d.R;
    p.open_list = open_list; p.open_count = open_count;
    p.part_m = out.m; p.part_s = out.s; p.top_val = out.top_val; p.top_idx = out.top_idx; p.status = status;
    const int64_t items = (int64_t)d.R * d.S;
    const int grid = (int)(items < sm_count ? items : sm_count);
    if (d.dtype == DBA_F32) row_scan_tma_kernel<float><<<grid, kThreads, row_scan_tma_smem(), st>>>(p);
    else row_scan_tma_kernel<__nv_bfloat16><<<grid, kThreads, row_scan_tma_smem(), st>>>(p);
    return cudaGetLastError();
}

}  // namespace dba
