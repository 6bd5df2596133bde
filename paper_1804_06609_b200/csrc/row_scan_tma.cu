// Row scan, streaming version for sm_100a: one HBM pass per row.
//
// A persistent CTA per SM works through (row, segment) items; a segment is up to eight 8 KB chunks.  Warps have
// fixed roles and talk through mbarriers only (no CTA-wide barrier inside the loop):
//   producer    one thread issues bulk asynchronous copies (TMA, cp.async.bulk) of the chunks into a ring of
//               shared-memory stages;
//   consumers   each warp streams half a chunk of the item: the maximum first, then exp2(x*log2e - c) summed per
//               lane (Section 2's normaliser) with c a whole number at or above the maximum; it leaves one
//               maximum per lane; no selection logic in this loop;
//   bound       every consumer warp also leaves its J largest lane maxima; a warp takes the K1-th largest of
//               these values as a lower bound of the K1-th largest entry of the item (maxima of disjoint lanes:
//               at least K1 entries reach it).  J = ceil(K1 / warps with data), 2 for the usual shapes;
//   pass B      warps look again only at the vectors of lanes whose maximum reaches the bound (a few dozen of
//               the 4096 vectors of an item), collect the entries at or above the bound, and hand the stages
//               back to the producer;
//   ranking     warps (alternating items) order the collected entries exactly (value descending, lower index first) and
//               writes the segment's partial result.
// Every wait is bounded: a wait that runs out sets the timeout bit of the status word and the CTA winds down.
// The code is kept small on purpose: the roles run different code at the same time and share one
// instruction cache.
#include <cuda_bf16.h>

#include "dba_device.cuh"
#include "dba_internal.h"

namespace dba {

namespace {

constexpr int kChunkBytes = 8192;
constexpr int kChunkVecs = kChunkBytes / 16;   // 512
constexpr int kHalfVecs = kChunkVecs / 2;      // vectors of half a chunk: 8 per lane
constexpr int kVecsPerLane = kHalfVecs / 32;   // 8
constexpr int kStages = 24;                    // 192 KB of ring
constexpr int kMaxSegChunks = 8;               // a segment is at most 64 KB
constexpr int kNC = 2 * kMaxSegChunks;         // consumer warps, half a chunk of the item each
constexpr int kNB = 1;                         // bound warps
constexpr int kNS = kMaxSegChunks;             // pass-B warps, one chunk of the item each
constexpr int kNR = 2;                         // ranking warps, alternating items
constexpr int kWarpBound = 1 + kNC;            // first bound warp
constexpr int kWarpPassB = kWarpBound + kNB;   // first pass-B warp
constexpr int kWarpRank = kWarpPassB + kNS;    // first ranking warp
constexpr int kThreads = 32 * (kWarpRank + kNR);
constexpr int kSlots = 4;                      // items in flight between consumers and ranking
constexpr int kCandCap = 256;                  // entries at or above the bound that one item may hold
constexpr uint32_t kSpinLimit = 1u << 20;
constexpr uint32_t kSuspendHint = 0x989680u;   // lets a waiting thread sleep in hardware until the phase completes
constexpr float kLog2e = 1.44269502162933349609375f;        // fl32(log2(e))

struct Smem {
    alignas(128) unsigned char ring[kStages][kChunkBytes];
    alignas(8) uint64_t full[kStages];
    uint64_t empty[kStages];
    uint64_t item_done[kSlots];
    uint64_t bound_ready[kSlots];
    uint64_t passb_done[kSlots];
    uint64_t slot_free[kSlots];
    uint64_t cand[kSlots][kCandCap];
    float lane_max[kSlots][kNC][32];
    float lane_top[kSlots][kNC * 32];       // the J largest lane maxima of consumer warp w at [w*J, w*J + J)
    float warp_sum[kSlots][kNC];
    float warp_ref[kSlots][kNC];            // the whole number c of exp2(x*log2e - c) each warp used (-inf: no data)
    float bound_lo[kSlots];                 // entries >= bound_lo are collected
    int cand_count[kSlots];                 // above kCandCap: the list overflowed
    int abort_flag;
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
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(kSuspendHint) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the CTA is winding down (this wait ran out, or another one did).
__device__ __noinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
// The same for a whole warp (every lane observes the phase itself); the answer is the same on all lanes.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    bool ok = mbar_try_wait(bar, parity);
    if (!ok) ok = mbar_wait(bar, parity, abort_flag);
    return __all_sync(kFullMask, ok);
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ float ex2(float t) { float r; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(t)); return r; }
// 2^d for an integer d <= 0, exact (0 below the normal range)
__device__ __forceinline__ float pow2i(int d) { return d < -126 ? 0.f : __int_as_float((d + 127) << 23); }
__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
    uint32_t r; asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b)); return r;
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
// two fp32 values in one 64-bit register, for the packed fma / add of sm_100
__device__ __forceinline__ uint64_t pack2(float lo, float hi) { uint64_t r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi)); return r; }
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) { uint64_t d; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c)); return d; }
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) { uint64_t d; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b)); return d; }
// acc += (2^(a*L + C), 2^(b*L + C)) for packed constants L2 = (L, L), C2 = (C, C)
__device__ __forceinline__ uint64_t exp_acc(uint64_t acc, float a, float b, uint64_t L2, uint64_t C2) {
    float t0, t1;
    unpack2(fma2(pack2(a, b), L2, C2), t0, t1);
    return add2(acc, pack2(ex2(t0), ex2(t1)));
}

template <typename T> struct Vec;
template <> struct Vec<float> {
    static constexpr int kElems = 4;
    static constexpr uint32_t kNegInfWord = 0xff800000u;
    // running maximum of vectors, kept in a form that is cheap to update
    typedef float Max;
    static __device__ __forceinline__ Max max_init() { return neg_inf(); }
    static __device__ __forceinline__ Max max_update(Max m, const uint4& v) {
        return fmaxf(fmaxf(m, fmaxf(__uint_as_float(v.x), __uint_as_float(v.y))), fmaxf(__uint_as_float(v.z), __uint_as_float(v.w)));
    }
    static __device__ __forceinline__ float max_value(Max m) { return m; }
    static __device__ __forceinline__ void unpack(const uint4& v, float* x) {
        x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y); x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
    }
    static __device__ __forceinline__ void exp_sum(const uint4& v, uint64_t L2, uint64_t C2, uint64_t& a0, uint64_t& a1) {
        a0 = exp_acc(a0, __uint_as_float(v.x), __uint_as_float(v.y), L2, C2);
        a1 = exp_acc(a1, __uint_as_float(v.z), __uint_as_float(v.w), L2, C2);
    }
};
template <> struct Vec<__nv_bfloat16> {
    static constexpr int kElems = 8;
    static constexpr uint32_t kNegInfWord = 0xff80ff80u;
    typedef uint32_t Max;       // two bf16 maxima
    static __device__ __forceinline__ Max max_init() { return kNegInfWord; }
    static __device__ __forceinline__ Max max_update(Max m, const uint4& v) {
        return max_bf16x2(max_bf16x2(m, max_bf16x2(v.x, v.y)), max_bf16x2(v.z, v.w));
    }
    static __device__ __forceinline__ float max_value(Max m) { return fmaxf(bf16_lo(m), bf16_hi(m)); }
    static __device__ __forceinline__ void unpack(const uint4& v, float* x) {
        x[0] = bf16_lo(v.x); x[1] = bf16_hi(v.x); x[2] = bf16_lo(v.y); x[3] = bf16_hi(v.y);
        x[4] = bf16_lo(v.z); x[5] = bf16_hi(v.z); x[6] = bf16_lo(v.w); x[7] = bf16_hi(v.w);
    }
    static __device__ __forceinline__ void exp_sum(const uint4& v, uint64_t L2, uint64_t C2, uint64_t& a0, uint64_t& a1) {
        a0 = exp_acc(a0, bf16_lo(v.x), bf16_hi(v.x), L2, C2);
        a1 = exp_acc(a1, bf16_lo(v.y), bf16_hi(v.y), L2, C2);
        a0 = exp_acc(a0, bf16_lo(v.z), bf16_hi(v.z), L2, C2);
        a1 = exp_acc(a1, bf16_lo(v.w), bf16_hi(v.w), L2, C2);
    }
};

// The items of this CTA, in the order all roles agree on, with the ring position of each item's first chunk.
// Items are numbered row-major over (position in the list of open rows, segment); this CTA takes every
// gridDim.x-th one.  The walk needs no division after the constructor.
struct ItemIter {
    int i, seg_, n_rows, S, step_i, step_seg, seg_bytes_full, row_bytes;
    int row_, bytes_, n_chunks_;        // of the current item
    uint32_t fills, n_item;
    const int32_t* open_list;
    __device__ ItemIter(const Params& p, int elem_bytes) : S(p.S), fills(0), n_item(0), open_list(p.open_list) {
        n_rows = p.open_count ? *p.open_count : p.R;
        i = blockIdx.x / S; seg_ = blockIdx.x - i * S;
        step_i = gridDim.x / S; step_seg = gridDim.x - step_i * S;
        seg_bytes_full = p.seg_len * elem_bytes;
        row_bytes = p.V * elem_bytes;
        load();
    }
    __device__ __forceinline__ void load() {
        if (i >= n_rows) return;
        row_ = open_list ? open_list[i] : i;
        bytes_ = min(seg_bytes_full, row_bytes - seg_ * seg_bytes_full);
        n_chunks_ = (bytes_ + kChunkBytes - 1) / kChunkBytes;
    }
    __device__ bool valid() const { return i < n_rows; }
    __device__ void next() {
        fills += (uint32_t)n_chunks_; n_item += 1;
        i += step_i; seg_ += step_seg;
        if (seg_ >= S) { seg_ -= S; ++i; }
        load();
    }
    __device__ int row() const { return row_; }
    __device__ int seg() const { return seg_; }
    __device__ int bytes() const { return bytes_; }
    __device__ int n_chunks() const { return n_chunks_; }
    __device__ uint32_t slot() const { return n_item % kSlots; }
    __device__ uint32_t slot_phase() const { return (n_item / kSlots) & 1u; }
    __device__ uint32_t stage(int c) const { return (fills + (uint32_t)c) % kStages; }
    __device__ uint32_t stage_phase(int c) const { return ((fills + (uint32_t)c) / kStages) & 1u; }
    __device__ int chunk_vecs(int c) const { return min(kChunkBytes, bytes_ - c * kChunkBytes) >> 4; }
    // consumer warps that get data (half a chunk each), and how many lane maxima each reports so that
    // together they report at least K1 (capped by the 32 lanes a warp has)
    __device__ int active_warps() const { return ((bytes_ >> 4) + kHalfVecs - 1) / kHalfVecs; }
    __device__ int report(int K1) const { return min(32, (K1 + active_warps() - 1) / active_warps()); }
};

// Ranking, rare path: more entries at or above the bound than the list holds (long runs of equal values at the
// bound, or an adversarial layout): take the K1 best one at a time, reading the segment again from global memory.
template <typename T>
__device__ __noinline__ void rank_from_global(const T* src, int e0, int e1, int K1, float* tv, int32_t* ti) {
    const int lane = threadIdx.x & 31;
    uint64_t prev = ~0ull;
#pragma unroll 1
    for (int r2 = 0; r2 < K1; ++r2) {
        uint64_t best = 0;
#pragma unroll 2
        for (int w = e0 + lane; w < e1; w += 32) {
            const uint64_t kk = row_key(load_logit<T>(src + w), w);
            if (kk < prev && kk > best) best = kk;
        }
        best = warp_max_u64(best);
        if (lane == 0) { tv[r2] = best ? row_key_val(best) : neg_inf(); ti[r2] = best ? row_key_idx(best) : -1; }
        prev = best;      // 0 once exhausted: nothing is below it
    }
}

template <typename T>
__global__ void __launch_bounds__(kThreads, 1) row_scan_tma_kernel(Params p) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
    constexpr int kElems = Vec<T>::kElems;
    constexpr int kChunkElems = kChunkBytes / (int)sizeof(T);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int* abort_flag = &sm.abort_flag;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&sm.full[s]), 1); mbar_init(smem_u32(&sm.empty[s]), 1); }
        for (int s = 0; s < kSlots; ++s) {
            mbar_init(smem_u32(&sm.item_done[s]), kNC); mbar_init(smem_u32(&sm.bound_ready[s]), 1);
            mbar_init(smem_u32(&sm.passb_done[s]), kNS); mbar_init(smem_u32(&sm.slot_free[s]), 1);
            sm.cand_count[s] = 0;
        }
        sm.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            ItemIter it(p, (int)sizeof(T));
            bool ok = true;
#pragma unroll 1
            for (; ok && it.valid(); it.next()) {
                const char* src = (const char*)p.logits + ((int64_t)it.row() * p.stride + (int64_t)it.seg() * p.seg_len) * (int64_t)sizeof(T);
                const int nc = it.n_chunks();
#pragma unroll 1
                for (int c = 0; c < nc; ++c) {
                    const uint32_t st = it.stage(c);
                    if (!mbar_try_wait(smem_u32(&sm.empty[st]), it.stage_phase(c) ^ 1u) &&
                        !mbar_wait(smem_u32(&sm.empty[st]), it.stage_phase(c) ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t bytes = (uint32_t)it.chunk_vecs(c) << 4;
                    mbar_expect_tx(smem_u32(&sm.full[st]), bytes);
                    bulk_load(smem_u32(sm.ring[st]), src + (int64_t)c * kChunkBytes, bytes, smem_u32(&sm.full[st]));
                }
            }
            if (!ok) {   // winding down: let the copies already issued land before the CTA leaves
                const uint32_t fills = it.fills + kMaxSegChunks;
                const uint32_t first = fills > kStages ? fills - kStages : 0;
#pragma unroll 1
                for (uint32_t f = first; f < fills; ++f)
                    for (uint32_t i = 0; i < 64 && !mbar_try_wait(smem_u32(&sm.full[f % kStages]), (f / kStages) & 1u); ++i) {}
            }
        }
        __syncwarp();
    } else if (warp <= kNC) {
        // ------------------------------------------------------------------ consumers
        const int cw = warp - 1, chunk = cw >> 1, half = cw & 1;
#pragma unroll 1
        for (ItemIter it(p, (int)sizeof(T)); it.valid(); it.next()) {
            float lmax = neg_inf(), ssum = 0.f, cref = neg_inf();
            const int nvec = chunk < it.n_chunks() ? it.chunk_vecs(chunk) - half * kHalfVecs : 0;
            if (nvec > 0) {
                if (!mbar_wait_warp(smem_u32(&sm.full[it.stage(chunk)]), it.stage_phase(chunk), abort_flag)) break;
                const uint4* vec = reinterpret_cast<const uint4*>(sm.ring[it.stage(chunk)]) + half * kHalfVecs + lane;
                uint4 v[kVecsPerLane];
                if (nvec >= kHalfVecs) {
#pragma unroll
                    for (int i = 0; i < kVecsPerLane; ++i) v[i] = vec[i * 32];
                } else {
#pragma unroll
                    for (int i = 0; i < kVecsPerLane; ++i) {
                        const uint32_t w = Vec<T>::kNegInfWord;
                        v[i] = i * 32 + lane < nvec ? vec[i * 32] : make_uint4(w, w, w, w);   // beyond the row: -inf
                    }
                }
                typename Vec<T>::Max pm = Vec<T>::max_init();
#pragma unroll
                for (int i = 0; i < kVecsPerLane; ++i) pm = Vec<T>::max_update(pm, v[i]);
                lmax = Vec<T>::max_value(pm);
                const float wm = warp_max(lmax);
                if (wm != neg_inf()) {
                    cref = ceilf(wm * kLog2e);            // a whole number: rescaling by powers of two is exact
                    const uint64_t L2 = pack2(kLog2e, kLog2e), C2 = pack2(-cref, -cref);
                    uint64_t a0 = 0, a1 = 0;
#pragma unroll
                    for (int i = 0; i < kVecsPerLane; ++i) Vec<T>::exp_sum(v[i], L2, C2, a0, a1);
                    float s0, s1, s2, s3;
                    unpack2(a0, s0, s1); unpack2(a1, s2, s3);
                    ssum = (s0 + s1) + (s2 + s3);
                }
            }
            // hand the lane maxima and the warp's sum over
            if (!mbar_wait_warp(smem_u32(&sm.slot_free[it.slot()]), it.slot_phase() ^ 1u, abort_flag)) break;
            sm.lane_max[it.slot()][cw][lane] = lmax;
            if (nvec > 0) {       // the warp's J largest lane maxima, one lane removed per round
                const int J = it.report(p.K1);
                float cur = lmax;
#pragma unroll 1
                for (int j = 0; j < J; ++j) {
                    const float m = warp_max(cur);
                    const unsigned who = __ballot_sync(kFullMask, cur == m);
                    if (lane == 0) sm.lane_top[it.slot()][cw * J + j] = m;
                    if (lane == __ffs(who) - 1) cur = neg_inf();
                }
            }
            const float wsum = warp_sum(ssum);
            if (lane == 0) { sm.warp_sum[it.slot()][cw] = wsum; sm.warp_ref[it.slot()][cw] = cref; }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm.item_done[it.slot()]));
        }
    } else if (warp < kWarpPassB) {
        // ------------------------------------------------------------------ bound
#pragma unroll 1
        for (ItemIter it(p, (int)sizeof(T)); it.valid(); it.next()) {
            const uint32_t slot = it.slot();
            if (!mbar_wait_warp(smem_u32(&sm.item_done[slot]), it.slot_phase(), abort_flag)) break;
            // The K1-th largest of the reported lane maxima, by counting for each value how many are larger
            // (equal values ordered by position, so that the ranks are all different).
            const int J = it.report(p.K1), n_top = it.active_warps() * J;
            float lo = neg_inf();                 // fewer than K1 values: everything is collected
            if (n_top >= p.K1) {
#pragma unroll 1
                for (int i0 = 0; i0 < n_top; i0 += 32) {
                    const int i = i0 + lane;
                    const float mine = i < n_top ? sm.lane_top[slot][i] : neg_inf();
                    int rank = 0;
#pragma unroll 4
                    for (int j = 0; j < n_top; ++j) {
                        const float o = sm.lane_top[slot][j];
                        rank += (o > mine) || (o == mine && j < i);
                    }
                    const unsigned hit = __ballot_sync(kFullMask, i < n_top && rank == p.K1 - 1);
                    if (hit) lo = __shfl_sync(kFullMask, mine, __ffs(hit) - 1);
                }
            }
            if (lane == 0) sm.bound_lo[slot] = lo;
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm.bound_ready[slot]));
        }
    } else if (warp < kWarpRank) {
        // ------------------------------------------------------------------ pass B
        // This warp owns chunk sw of every item, i.e. consumer warps 2*sw and 2*sw+1.  Only lanes
        // whose maximum reaches the bound can hold an entry at or above it; up to four such lanes are handled
        // at a time, eight lanes of this warp looking at the eight vectors of one of them.
        const int sw = warp - kWarpPassB, grp = lane >> 3, vrow = lane & 7;
#pragma unroll 1
        for (ItemIter it(p, (int)sizeof(T)); it.valid(); it.next()) {
            const uint32_t slot = it.slot();
            if (!mbar_wait_warp(smem_u32(&sm.bound_ready[slot]), it.slot_phase(), abort_flag)) break;
            // The chunks' bytes are visible here: their consumers observed the copies' completion before they
            // reported the item done, and that report is ordered before the bound this warp has just waited for.
            const float lo = sm.bound_lo[slot];
            const int nc = it.n_chunks();
            const int elem0 = it.seg() * p.seg_len;
            if (sw < nc) {
                // bit l of m0 / m1: lane l of the first / second half's consumer warp reaches the bound
                unsigned m0 = __ballot_sync(kFullMask, sm.lane_max[slot][2 * sw][lane] >= lo);
                unsigned m1 = __ballot_sync(kFullMask, sm.lane_max[slot][2 * sw + 1][lane] >= lo);
                const uint4* vec = reinterpret_cast<const uint4*>(sm.ring[it.stage(sw)]);
                const int nvec = it.chunk_vecs(sw);
                while (m0 | m1) {
                    // the grp-th of the remaining candidate lanes, first half before second
                    int half = 0; unsigned mm = m0;
                    int skip = grp;
                    const int c0 = __popc(m0);
                    if (skip >= c0) { half = 1; mm = m1; skip -= c0; }
                    for (int j = 0; j < skip; ++j) mm &= mm - 1;
                    const int src_lane = __ffs(mm) - 1;
                    const int vi = half * kHalfVecs + vrow * 32 + src_lane;
                    if (mm && vi < nvec) {
                        float x[kElems];
                        Vec<T>::unpack(vec[vi], x);
                        const int base = elem0 + sw * kChunkElems + vi * kElems;
#pragma unroll
                        for (int e = 0; e < kElems; ++e)
                            if (x[e] >= lo) {
                                const int pos = atomicAdd(&sm.cand_count[slot], 1);
                                if (pos < kCandCap) sm.cand[slot][pos] = row_key(x[e], base + e);
                            }
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) { if (m0) m0 &= m0 - 1; else m1 &= m1 - 1; }     // four lanes done
                    __syncwarp();
                }
            }
            __syncwarp();
            if (lane == 0) {
                if (sw < nc) mbar_arrive(smem_u32(&sm.empty[it.stage(sw)]));          // the producer may refill it
                mbar_arrive(smem_u32(&sm.passb_done[slot]));
            }
        }
    } else {
        // ------------------------------------------------------------------ ranking
#pragma unroll 1
        for (ItemIter it(p, (int)sizeof(T)); it.valid(); it.next()) {
            if ((int)(it.n_item % kNR) != warp - kWarpRank) continue;       // the other ranking warp's item
            const uint32_t slot = it.slot();
            if (!mbar_wait_warp(smem_u32(&sm.passb_done[slot]), it.slot_phase(), abort_flag)) break;
            const int n = sm.cand_count[slot];
            const int64_t out = (int64_t)it.row() * p.S + it.seg();
            {   // the segment's normaliser: sum_x 2^(x*log2e) = S * 2^C with a whole number C; lane w holds warp w's part
                const float cw2 = lane < kNC ? sm.warp_ref[slot][lane] : neg_inf();
                const float C = warp_max(cw2);
                const float S = warp_sum(cw2 != neg_inf() ? sm.warp_sum[slot][lane] * pow2i((int)(cw2 - C)) : 0.f);
                if (lane == 0) {
                    float m = neg_inf(), s2 = 0.f;
                    if (C != neg_inf()) {
                        // (m, s) with sum_x e^x = s * e^m: m = fl32(C ln2), the rounding of m folded into s
                        constexpr float kLn2Hi = 0.693147182464599609375f, kLn2Lo = -1.904654299957767e-9f;
                        m = C * kLn2Hi;
                        const float err = fmaf(C, kLn2Hi, -m) + C * kLn2Lo;
                        s2 = fmaf(S, err, S);
                    }
                    p.part_m[out] = m; p.part_s[out] = s2;
                }
            }
            float* tv = p.top_val + out * p.K1;
            int32_t* ti = p.top_idx + out * p.K1;
            if (n <= kCandCap) {
#pragma unroll 1
                for (int i = n + lane; i < p.K1; i += 32) { tv[i] = neg_inf(); ti[i] = -1; }
#pragma unroll 1
                for (int i = lane; i < n; i += 32) {
                    const uint64_t ki = sm.cand[slot][i];
                    int rank = 0;
#pragma unroll 2
                    for (int j = 0; j < n; ++j) rank += sm.cand[slot][j] > ki;
                    if (rank < p.K1) { tv[rank] = row_key_val(ki); ti[rank] = row_key_idx(ki); }
                }
            } else {
                rank_from_global<T>((const T*)p.logits + (int64_t)it.row() * p.stride, it.seg() * p.seg_len,
                                    it.seg() * p.seg_len + it.bytes() / (int)sizeof(T), p.K1, tv, ti);
            }
            __syncwarp();
            if (lane == 0) { sm.cand_count[slot] = 0; mbar_arrive(smem_u32(&sm.slot_free[slot])); }
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
