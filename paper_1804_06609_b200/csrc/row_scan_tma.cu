// Row scan, streaming version for sm_100a: one HBM pass per row.
//
// A persistent CTA per SM works through (row, segment) items; a segment is up to eleven 4 KB chunks.  Four
// items are in flight, each with a shared-memory buffer and a selector warp of its own.  Warps have fixed
// roles and talk through mbarriers only (no CTA-wide barrier inside the loop); a consumer never waits for
// another consumer:
//   producer    one thread refills a buffer as soon as the item's consumers are done with it: one bulk
//               asynchronous copy (TMA, cp.async.bulk) per item;
//   consumers   two teams of eleven warps, the teams taking alternate items.  A warp owns one chunk of its
//               item: it reads the chunk (eight 16-byte vectors per lane) once for the maxima and once more for
//               the sum of exp2(x*log2e - c) (Section 2's normaliser), c a whole number at or above the warp's
//               maximum.  The selection piggybacks on the maxima: the maxima of every pair of vectors (cells
//               of eight entries) and of every lane go to shared memory as they are, and the butterfly that
//               gives the warp's maximum is tapped midway, which yields the maxima of G groups of lanes
//               (G >= 4 and G * warps with data >= K1), the warp's reports;
//   selectors   four warps, selector s serving the items that use buffer s.  The K1-th largest report is a
//               lower bound of the K1-th largest entry of the item, because group maxima are distinct
//               entries.  The selector finds the lanes, then the cells, whose maximum reaches the bound (two
//               or three dozen of the 2816 cells of an item), reads those cells again (from L2: the buffer
//               may be gone), keeps the entries at or above the bound, orders them exactly (value
//               descending, lower index first) and writes the segment's partial result: the K1 best
//               entries and the normaliser.
// Every wait is bounded: a wait that runs out sets the timeout bit of the status word and the CTA winds down.
#include <climits>

#include <cuda_bf16.h>

#include "dba_device.cuh"
#include "dba_internal.h"

namespace dba {

namespace {

constexpr int kChunkBytes = 4096;
constexpr int kChunkVecs = kChunkBytes / 16;   // 256
constexpr int kVecsPerLane = kChunkVecs / 32;  // 8
constexpr int kPairs = kVecsPerLane / 2;       // pairs of vectors per lane and chunk
constexpr int kTeamWarps = 11;                 // consumer warps per team = most chunks in a segment (44 KB)
constexpr int kTeams = 2;                      // teams take alternate items
constexpr int kNC = kTeams * kTeamWarps;       // consumer warps
constexpr int kSlots = 4;                      // items in flight: buffers (176 KB in all) and selection state
constexpr int kNR = kSlots;                    // selector warps (and ranking warps), one per slot
constexpr int kWarpSel = 0;                    // first selector warp
constexpr int kWarpRank = kNR;                 // first ranking warp
constexpr int kWarpProd = 2 * kNR;             // the producer's warp
constexpr int kWarpCons = 2 * kNR + 1;         // first consumer warp
constexpr int kThreads = 32 * (kWarpCons + kNC);
constexpr int kHitCap = 192;                   // cells reaching the bound that one item may have (three per wanted entry at K1 = 66)
constexpr int kKeyCap = 256;                   // entries at or above the bound that one item may hold
constexpr int kRepCap = 192;                   // reports of one item (11 warps x 16 groups fit)
constexpr float kLog2e = 1.44269502162933349609375f;        // fl32(log2(e))

struct WaitCtl {
    int abort_flag;                         // a wait ran out: everybody winds down
    uint32_t n_issued;                      // items whose copy the producer has announced
    long long wait_clocks;                  // how long a wait may last
};

constexpr int kStaticItems = kSlots;         // a CTA's first items are fixed by its number, the rest drawn from a counter
constexpr int kItemRing = 4 * kSlots;        // item descriptors kept in shared memory
struct ItemDesc { int row; int seg; };       // what the producer tells the other roles about an item; row < 0: no more items

struct Smem {
    alignas(128) unsigned char ring[kSlots][kTeamWarps * kChunkBytes];
    alignas(16) uint4 cell_max[kSlots][kTeamWarps][32];     // per lane: the maxima of its four pairs of vectors
    alignas(16) uint32_t report[kSlots][kRepCap];           // group maxima as ordered integers, warp w's at [w*G, w*G + G)
    alignas(8) uint64_t key[kNR][kKeyCap];
    uint64_t full[kSlots];          // the item's bytes have landed
    uint64_t loaded[kSlots];        // every consumer warp of the team is done with the buffer (it has read its chunk twice)
    uint64_t reports_in[kSlots];    // every consumer warp of the team has left its maxima and reports
    uint64_t sums_in[kSlots][2];    // every consumer warp of the team has left its sum (alternate uses, alternate barriers)
    uint64_t slot_free[kSlots];     // the selector is done with the slot's shared state
    uint32_t lane_key[kSlots][kTeamWarps][32];              // lane maxima as ordered integers
    float warp_sum[kSlots][2][kTeamWarps];  // alternate uses of a slot take alternate halves
    float warp_ref[kSlots][2][kTeamWarps];  // the whole number c of exp2(x*log2e - c) each warp used (-inf: no data)
    uint64_t hits_ready[kSlots];            // the selector has left the item's cell list
    uint64_t ranked[kSlots];                // the ranking warp is done with the item
    int hit_lane[kNR][kHitCap];             // lanes that reach the bound: chunk * 32 + lane
    int hit[kSlots][2][kHitCap];            // cells that reach the bound: (first vector of the pair) * 2 + parity
    int hit_n[kSlots][2];                   // how many (above kHitCap: the list overflowed)
    float hit_bound[kSlots][2];
    ItemDesc item[kItemRing];               // by item number % kItemRing
    WaitCtl ctl;
};

struct Params {
    const void* logits;
    int64_t stride;             // elements
    int V, S, seg_len, K1;
    int R;
    const int32_t* open_list;   // rows to scan (null: all R rows)
    const int32_t* open_count;  // number of entries of open_list (device memory)
    int32_t* zero_count;        // set to zero here: the count of the list the step's last kernel builds (may be null)
    int32_t* ticket;            // zero at launch: the counter the CTAs draw their items from
    int32_t* zero_ticket;       // set to zero here: the next launch's counter (may be null)
    float* part_m; float* part_s; float* top_val; int32_t* top_idx;     // results, per (row, segment)
    uint32_t* status;
    long long wait_clocks;      // how long a wait may last
    int drop_item;              // testing: every CTA announces the copy of this item of its sequence but never issues it
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
__device__ __noinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile WaitCtl* ctl) {
    const long long t0 = clock64();
    const long long limit = ctl->wait_clocks;
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 32; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (ctl->abort_flag) return false;
        if (clock64() - t0 > limit) break;
    }
    ctl->abort_flag = 1;
    return false;
}
// The same for a whole warp (every lane observes the phase itself); the answer is the same on all lanes.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile WaitCtl* abort_flag) {
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

// A cell is what one stored maximum stands for: eight entries of a pair of vectors (2p, 2p+1) of a lane.
//   fp32   a vector has four entries; the cell is the whole pair; a lane stores four floats.
//   bf16   a vector has eight entries; packed maxima keep even and odd positions apart, so the pair has two
//          cells (parity 0 and 1); a lane stores four words of two bf16 maxima.
template <typename T> struct Vec;
template <> struct Vec<float> {
    static constexpr uint32_t kNegInfWord = 0xff800000u;
    typedef float Max;
    static __device__ __forceinline__ Max vec_max(const uint4& v) {
        return fmaxf(fmaxf(__uint_as_float(v.x), __uint_as_float(v.y)), fmaxf(__uint_as_float(v.z), __uint_as_float(v.w)));
    }
    static __device__ __forceinline__ Max max2(Max a, Max b) { return fmaxf(a, b); }
    static __device__ __forceinline__ float max_value(Max m) { return m; }
    static __device__ __forceinline__ uint32_t word(Max m) { return __float_as_uint(m); }
    // bit p: the cell of pair p reaches tau
    static __device__ __forceinline__ unsigned reach_mask(const uint4& cm, float tau) {
        return (__uint_as_float(cm.x) >= tau ? 1u : 0u) | (__uint_as_float(cm.y) >= tau ? 2u : 0u) |
               (__uint_as_float(cm.z) >= tau ? 4u : 0u) | (__uint_as_float(cm.w) >= tau ? 8u : 0u);
    }
    static __device__ __forceinline__ int cell_pair(int cell) { return cell; }
    static __device__ __forceinline__ int cell_parity(int) { return 0; }
    // the eight entries of a cell and the position of each within the item, given the pair's two vectors
    static __device__ __forceinline__ void cell_entries(const uint4& a, const uint4& b, int vec_a, int, float* x, int* at) {
        x[0] = __uint_as_float(a.x); x[1] = __uint_as_float(a.y); x[2] = __uint_as_float(a.z); x[3] = __uint_as_float(a.w);
        x[4] = __uint_as_float(b.x); x[5] = __uint_as_float(b.y); x[6] = __uint_as_float(b.z); x[7] = __uint_as_float(b.w);
#pragma unroll
        for (int j = 0; j < 4; ++j) { at[j] = vec_a * 4 + j; at[4 + j] = (vec_a + 32) * 4 + j; }
    }
    static __device__ __forceinline__ void exp_sum(const uint4& v, uint64_t L2, uint64_t C2, uint64_t& a0, uint64_t& a1) {
        a0 = exp_acc(a0, __uint_as_float(v.x), __uint_as_float(v.y), L2, C2);
        a1 = exp_acc(a1, __uint_as_float(v.z), __uint_as_float(v.w), L2, C2);
    }
};
template <> struct Vec<__nv_bfloat16> {
    static constexpr uint32_t kNegInfWord = 0xff80ff80u;
    typedef uint32_t Max;       // two bf16 maxima: of the entries at even and at odd positions
    static __device__ __forceinline__ Max vec_max(const uint4& v) { return max_bf16x2(max_bf16x2(v.x, v.y), max_bf16x2(v.z, v.w)); }
    static __device__ __forceinline__ Max max2(Max a, Max b) { return max_bf16x2(a, b); }
    static __device__ __forceinline__ float max_value(Max m) { return fmaxf(bf16_lo(m), bf16_hi(m)); }
    static __device__ __forceinline__ uint32_t word(Max m) { return m; }
    // bit 2p + parity: that cell reaches tau (tau is a group maximum, hence a bf16 value: its upper half is exact)
    static __device__ __forceinline__ unsigned reach_mask(const uint4& cm, float tau) {
        const uint32_t u = __float_as_uint(tau), t2 = (u & 0xffff0000u) | (u >> 16);
        uint32_t r0, r1, r2, r3;    // 0xffff in each half where the maximum reaches tau
        asm("set.ge.u32.bf16x2 %0, %1, %2;" : "=r"(r0) : "r"(cm.x), "r"(t2));
        asm("set.ge.u32.bf16x2 %0, %1, %2;" : "=r"(r1) : "r"(cm.y), "r"(t2));
        asm("set.ge.u32.bf16x2 %0, %1, %2;" : "=r"(r2) : "r"(cm.z), "r"(t2));
        asm("set.ge.u32.bf16x2 %0, %1, %2;" : "=r"(r3) : "r"(cm.w), "r"(t2));
        return ((r0 & 1u) | ((r0 >> 15) & 2u)) | (((r1 & 1u) | ((r1 >> 15) & 2u)) << 2) |
               (((r2 & 1u) | ((r2 >> 15) & 2u)) << 4) | (((r3 & 1u) | ((r3 >> 15) & 2u)) << 6);
    }
    static __device__ __forceinline__ int cell_pair(int cell) { return cell >> 1; }
    static __device__ __forceinline__ int cell_parity(int cell) { return cell & 1; }
    static __device__ __forceinline__ void cell_entries(const uint4& a, const uint4& b, int vec_a, int parity, float* x, int* at) {
        const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
        for (int j = 0; j < 8; ++j) x[j] = parity ? bf16_hi(w[j]) : bf16_lo(w[j]);
#pragma unroll
        for (int j = 0; j < 4; ++j) { at[j] = vec_a * 8 + 2 * j + parity; at[4 + j] = (vec_a + 32) * 8 + 2 * j + parity; }
    }
    static __device__ __forceinline__ void exp_sum(const uint4& v, uint64_t L2, uint64_t C2, uint64_t& a0, uint64_t& a1) {
        a0 = exp_acc(a0, bf16_lo(v.x), bf16_hi(v.x), L2, C2);
        a1 = exp_acc(a1, bf16_lo(v.y), bf16_hi(v.y), L2, C2);
        a0 = exp_acc(a0, bf16_lo(v.z), bf16_hi(v.z), L2, C2);
        a1 = exp_acc(a1, bf16_lo(v.w), bf16_hi(v.w), L2, C2);
    }
};

// Which item is whose.  Items are numbered row-major over (position in the list of open rows, segment).  A CTA's
// first kStaticItems items are fixed by its number (item c + n * gridDim.x for its n-th), so that it can start
// without asking; the rest are drawn one at a time from a counter in global memory, so that a CTA that gets ahead
// (the memory system does not serve all SMs alike from one launch to the next: CTAs given equal shares finish up
// to 10 us apart) takes more.  The producer draws (kStaticItems items ahead of the copy it issues), looks the row up and
// leaves (row, segment) in a ring of descriptors in shared memory, where the other roles find it after the wait
// that orders them behind the producer; a descriptor without a row says that there are no more items.  It is
// written for the item of each of the kSlots buffers after the last, passes through all roles like an item
// without data, and each role stops when it has met as many as it serves buffers.
// A descriptor is overwritten kItemRing items later, which the copy into the same buffer three uses later waits
// for: by then the buffer's ranking warp, the last to look at it, has finished the buffer's next item.

// A role's place in its CTA's sequence of items, and the geometry of the item it is at.
// (Only a row's last segment differs from the others in length: what depends on the length alone -- bytes, chunks,
// the tap of the reports -- is worked out once for the two kinds, and an item picks one.)
struct ItemIter {
    int S, seg_, row_;
    int bytes_kind[2], chunks_kind[2], tap_kind[2];     // [0]: a full segment, [1]: the row's last segment
    int bytes_, n_chunks_, tap_;  // of the current item
    uint32_t n_item;
    __device__ ItemIter(const Params& p, int elem_bytes) : S(p.S), seg_(0), row_(-1), n_item(0) {
        const int seg_bytes_full = p.seg_len * elem_bytes, row_bytes = p.V * elem_bytes;
        bytes_kind[0] = seg_bytes_full;
        bytes_kind[1] = row_bytes - (S - 1) * seg_bytes_full;
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            chunks_kind[q] = (bytes_kind[q] + kChunkBytes - 1) / kChunkBytes;
            tap_kind[q] = tap_for(bytes_kind[q], p.K1);
        }
        set(-1, 0);
    }
    __device__ __forceinline__ void set(int row, int seg) {
        row_ = row; seg_ = seg;
        const bool last = seg_ == S - 1;
        bytes_ = last ? bytes_kind[1] : bytes_kind[0];
        n_chunks_ = last ? chunks_kind[1] : chunks_kind[0];
        tap_ = last ? tap_kind[1] : tap_kind[0];
    }
    // the descriptor the producer left for this item (call after the wait that orders this role behind it)
    __device__ __forceinline__ void fetch(const ItemDesc* ring) { const ItemDesc d = ring[n_item % kItemRing]; set(d.row, d.seg); }
    __device__ bool valid() const { return row_ >= 0; }
    __device__ void skip(int k) { n_item += (uint32_t)k; }
    __device__ int row() const { return row_; }
    __device__ int seg() const { return seg_; }
    __device__ int bytes() const { return bytes_; }
    __device__ int n_chunks() const { return n_chunks_; }
    __device__ uint32_t slot() const { return n_item % kSlots; }
    __device__ uint32_t use() const { return n_item / kSlots; }            // how often the slot was used before
    __device__ uint32_t slot_phase() const { return use() & 1u; }
    __device__ int chunk_vecs(int c) const { return min(kChunkBytes, bytes_ - c * kChunkBytes) >> 4; }
    // Warps whose 32 lanes all hold data report (they are the first report_warps() of the team).  Each reports
    // the maxima of G = 32 >> tap groups of lanes, where tap is the number of butterfly steps taken before the
    // values are recorded; G is the largest of 4, 8, 16, 32 that keeps the item at 64 reports or fewer, or, if
    // that is fewer than K1, the smallest that gives K1.
    // tap < 0: no usable bound, every entry is kept.
    static __device__ int warps_reporting(int bytes) {
        const int nvec = bytes >> 4;
        return nvec / kChunkVecs + ((nvec % kChunkVecs) >= 32 ? 1 : 0);
    }
    __device__ int report_warps() const { return warps_reporting(bytes_); }
    __device__ int report_tap(int) const { return tap_; }
    static __device__ int tap_for(int bytes, int K1) {
        const int warps = warps_reporting(bytes);
        if (warps == 0) return -1;
        // as many reports as the selector's fast path takes (64): the more reports, the tighter the bound
        for (int tap = 0; tap <= 3; ++tap)             // G = 32, 16, 8, 4
            if ((32 >> tap) * warps <= 64) { if ((32 >> tap) * warps >= K1) return tap; break; }
        for (int tap = 3; tap >= 0; --tap)             // more than 64 reports are needed: G = 4, 8, 16, 32
            if ((32 >> tap) * warps >= K1) return (32 >> tap) * warps <= kRepCap ? tap : -1;
        return -1;
    }
};

// Ranking, rare path: more entries at or above the bound than the lists hold (long runs of equal values at the
// bound, or an adversarial layout): take the K1 best one at a time, reading the segment again from global memory.
template <typename T>
__device__ __noinline__ void rank_from_global(const T* src, int e0, int e1, int K1, float* tv, int32_t* ti) {
    const int lane = threadIdx.x & 31;
    uint64_t prev = ~0ull;
#pragma unroll 1
    for (int r2 = 0; r2 < K1; ++r2) {
        uint64_t best = 0;
#pragma unroll 8
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
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile WaitCtl* abort_flag = &sm.ctl;

    if (tid == 0) {
        for (int s = 0; s < kSlots; ++s) {
            mbar_init(smem_u32(&sm.full[s]), 1); mbar_init(smem_u32(&sm.loaded[s]), kTeamWarps);
            mbar_init(smem_u32(&sm.reports_in[s]), kTeamWarps); mbar_init(smem_u32(&sm.slot_free[s]), 1);
            mbar_init(smem_u32(&sm.sums_in[s][0]), kTeamWarps); mbar_init(smem_u32(&sm.sums_in[s][1]), kTeamWarps);
            mbar_init(smem_u32(&sm.hits_ready[s]), 1); mbar_init(smem_u32(&sm.ranked[s]), 1);
        }
        sm.ctl.abort_flag = 0; sm.ctl.n_issued = 0; sm.ctl.wait_clocks = p.wait_clocks;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    grid_dependency_wait();      // the list of open rows comes from the previous step's last kernel
    if (tid == 0) {
        if (blockIdx.x == 0 && p.zero_count) *p.zero_count = 0;     // before the next kernel can start
        if (blockIdx.x == 0 && p.zero_ticket) *p.zero_ticket = 0;
        allow_dependents();
    }

    if (warp == kWarpProd) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            ItemIter it(p, (int)sizeof(T));
            bool ok = true;
            // Items are drawn 2 * kAhead items ahead and their rows looked up kAhead ahead (the list of open rows is in
            // global memory), so that no copy waits for either, and no further, so that a CTA is committed to few
            // items when the counter runs out: g_far[q] is the number of the item 2 * kAhead from now, g_near[q] /
            // row_near[q] number and row of the item kAhead from now (q = item number % kAhead).  The first loads
            // overlap the load of the list's length: a place beyond the length is still a place of the list, its
            // value is just not used.
            const int S = p.S;
            auto row_of = [&](int g) { const int i = g / S; return i < p.R ? (p.open_list ? __ldg(p.open_list + i) : i) : 0; };
            constexpr int kAhead = kStaticItems / 2;
            static_assert(kSlots % kAhead == 0, "the queues are indexed by the buffer number");
            int g_near[kAhead], row_near[kAhead], g_far[kAhead];
#pragma unroll
            for (int q = 0; q < kAhead; ++q) {
                g_near[q] = (int)blockIdx.x + q * (int)gridDim.x; row_near[q] = row_of(g_near[q]);
                g_far[q] = (int)blockIdx.x + (kAhead + q) * (int)gridDim.x;
            }
            const int n_rows = p.open_count ? *p.open_count : p.R;
            const int total = n_rows * S;                 // items of this launch
            int n_end = 0;                                // descriptors without a row written so far
#pragma unroll 1
            while (ok && n_end < kSlots) {
#pragma unroll
                for (int j = 0; j < kSlots; ++j) {          // item n uses slot n % kSlots = j
                    if (n_end == kSlots) break;
                    const uint32_t slot = j;
                    const int q = j % kAhead;              // (a constant once the loop is unrolled)
                    const int g = g_near[q], row = row_near[q];
                    g_near[q] = g_far[q]; row_near[q] = row_of(g_far[q]);
                    g_far[q] = kStaticItems * (int)gridDim.x + atomicAdd(p.ticket, 1);
                    const uint32_t phase = (it.n_item / kSlots) & 1u;
                    if (!mbar_try_wait(smem_u32(&sm.loaded[slot]), phase ^ 1u) &&
                        !mbar_wait(smem_u32(&sm.loaded[slot]), phase ^ 1u, abort_flag)) { ok = false; break; }
                    ItemDesc* desc = &sm.item[it.n_item % kItemRing];
                    if (g < total) {
                        const int seg = g - (g / S) * S;
                        it.set(row, seg);
                        desc->row = row; desc->seg = seg;
                        const char* src = (const char*)p.logits + ((int64_t)row * p.stride + (int64_t)seg * p.seg_len) * (int64_t)sizeof(T);
                        mbar_expect_tx(smem_u32(&sm.full[slot]), (uint32_t)it.bytes());
                        if ((int)it.n_item != p.drop_item)
                            bulk_load(smem_u32(sm.ring[slot]), src, (uint32_t)it.bytes(), smem_u32(&sm.full[slot]));
                        it.skip(1);
                        sm.ctl.n_issued = it.n_item;
                    } else {            // no more items: an item without data, for the roles that serve this buffer to stop at
                        desc->row = -1; desc->seg = 0;
                        mbar_arrive(smem_u32(&sm.full[slot]));
                        it.skip(1);
                        ++n_end;
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp >= kWarpCons) {
        // ------------------------------------------------------------------ consumers
        const int team = (warp - kWarpCons) / kTeamWarps, chunk = (warp - kWarpCons) - team * kTeamWarps;
        ItemIter it(p, (int)sizeof(T));
        int n_ends = 0;                            // items without data met: one for each of the team's kSlots / kTeams buffers
#pragma unroll 1
        for (it.skip(team);; it.skip(kTeams)) {
            const uint32_t slot = it.slot(), half = it.use() & 1u;
            uint4 v[kVecsPerLane];
            typename Vec<T>::Max pmax[kPairs];
            uint32_t key = 0;                      // below the key of every value, -inf included
            // A warp without a chunk in this item waits for the copy all the same: it must not run ahead and sign
            // the buffer off (`loaded`) for this use while a slower warp has yet to do so for the previous one.
            if (!mbar_wait_warp(smem_u32(&sm.full[slot]), it.slot_phase(), abort_flag)) break;
            it.fetch(sm.item);
            if (!it.valid()) {
                // no more items: the word is passed on to the buffer's selector, in turn like any item's reports
                if (!mbar_wait_warp(smem_u32(&sm.slot_free[slot]), it.slot_phase() ^ 1u, abort_flag)) break;
                if (lane == 0) mbar_arrive(smem_u32(&sm.reports_in[slot]));
                if (++n_ends == kSlots / kTeams) break;
                continue;
            }
            const int nvec = chunk < it.n_chunks() ? it.chunk_vecs(chunk) : 0;
            if (nvec > 0) {
                const uint4* vec = reinterpret_cast<const uint4*>(sm.ring[slot]) + chunk * kChunkVecs + lane;
                if (nvec >= kChunkVecs) {
#pragma unroll
                    for (int i = 0; i < kVecsPerLane; ++i) v[i] = vec[i * 32];
                } else {
#pragma unroll
                    for (int i = 0; i < kVecsPerLane; ++i) {
                        const uint32_t w = Vec<T>::kNegInfWord;
                        v[i] = i * 32 + lane < nvec ? vec[i * 32] : make_uint4(w, w, w, w);   // beyond the row: -inf
                    }
                }
            }
            if (nvec > 0) {
#pragma unroll
                for (int q = 0; q < kPairs; ++q) pmax[q] = Vec<T>::max2(Vec<T>::vec_max(v[2 * q]), Vec<T>::vec_max(v[2 * q + 1]));
                key = ord32(Vec<T>::max_value(Vec<T>::max2(Vec<T>::max2(pmax[0], pmax[1]), Vec<T>::max2(pmax[2], pmax[3]))));
            }
            // the slot's shared selection state belongs to this item from here on
            if (!mbar_wait_warp(smem_u32(&sm.slot_free[slot]), it.slot_phase() ^ 1u, abort_flag)) break;
            if (nvec > 0) {
                sm.cell_max[slot][chunk][lane] = make_uint4(Vec<T>::word(pmax[0]), Vec<T>::word(pmax[1]), Vec<T>::word(pmax[2]), Vec<T>::word(pmax[3]));
                sm.lane_key[slot][chunk][lane] = key;
            }
            // butterfly maximum over the lanes; the group maxima met on the way are the warp's reports
            const int tap = nvec >= 32 ? it.report_tap(p.K1) : -1;
#pragma unroll
            for (int st = 0; st < 5; ++st) {
                if (st == tap && (lane & ((1 << st) - 1)) == 0) sm.report[slot][(chunk << (5 - st)) + (lane >> st)] = key;
                key = max(key, __shfl_xor_sync(kFullMask, key, 1 << st));
            }
            const float wm = nvec > 0 ? unord32(key) : neg_inf();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm.reports_in[slot]));

            float ssum = 0.f, cref = neg_inf();
            if (wm != neg_inf()) {
                cref = ceilf(wm * kLog2e);            // a whole number: rescaling by powers of two is exact
                const uint64_t L2 = pack2(kLog2e, kLog2e), C2 = pack2(-cref, -cref);
                uint64_t a0 = 0, a1 = 0;
                // the chunk is read from the buffer a second time: held in registers since the maxima, it would
                // leave the exponentials too few registers to overlap one another
                const uint4* vec = reinterpret_cast<const uint4*>(sm.ring[slot]) + chunk * kChunkVecs + lane;
                if (nvec >= kChunkVecs) {
#pragma unroll
                    for (int i = 0; i < kVecsPerLane; ++i) Vec<T>::exp_sum(vec[i * 32], L2, C2, a0, a1);
                } else {
#pragma unroll
                    for (int i = 0; i < kVecsPerLane; ++i) {
                        const uint32_t w = Vec<T>::kNegInfWord;
                        const uint4 vv = i * 32 + lane < nvec ? vec[i * 32] : make_uint4(w, w, w, w);
                        Vec<T>::exp_sum(vv, L2, C2, a0, a1);
                    }
                }
                float s0, s1, s2, s3;
                unpack2(a0, s0, s1); unpack2(a1, s2, s3);
                ssum = (s0 + s1) + (s2 + s3);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm.loaded[slot]));         // this warp is done with the buffer
            const float wsum = warp_sum(ssum);
            if (lane == 0) {
                sm.warp_sum[slot][half][chunk] = wsum; sm.warp_ref[slot][half][chunk] = cref;
                mbar_arrive(smem_u32(&sm.sums_in[slot][half]));
            }
        }
    } else if (warp < kWarpRank) {
        // ------------------------------------------------------------------ selector of slot rk
        const int rk = warp - kWarpSel;
        const uint32_t slot = (uint32_t)rk;
        ItemIter it(p, (int)sizeof(T));
        it.skip(rk);                                      // this selector's first item
#pragma unroll 1
        for (;;) {
            if (!mbar_wait_warp(smem_u32(&sm.reports_in[slot]), it.slot_phase(), abort_flag)) break;
            it.fetch(sm.item);
            if (!it.valid()) {                            // no more items: tell the ranking warp, in turn
                if (!mbar_wait_warp(smem_u32(&sm.ranked[slot]), it.slot_phase() ^ 1u, abort_flag)) break;
                if (lane == 0) mbar_arrive(smem_u32(&sm.hits_ready[slot]));
                break;
            }
            // The bound: the K1-th largest report, i.e. the largest report that at least K1 reports reach.
            const uint32_t half = it.use() & 1u;
            int* hits = sm.hit[slot][half];
            const int tap = it.report_tap(p.K1);
            const int n_rep = tap < 0 ? 0 : it.report_warps() << (5 - tap);     // a multiple of four
            uint32_t best = 0;
            if (n_rep <= 64) {
                // Radix selection over the upper 16 bits of the keys, one bit at a time: the largest t with at
                // least K1 reports >= t.  (Exact for bf16 values; for fp32 the bound ends up a little lower.)
                const uint32_t m0 = lane < n_rep ? sm.report[slot][lane] : 0u;
                const uint32_t m1 = 32 + lane < n_rep ? sm.report[slot][32 + lane] : 0u;
                if (n_rep >= p.K1) {
#pragma unroll 4
                    for (uint32_t bit = 0x80000000u; bit >= 0x00010000u; bit >>= 1) {
                        const uint32_t t = best | bit;
                        const int cnt = __popc(__ballot_sync(kFullMask, m0 >= t)) + __popc(__ballot_sync(kFullMask, m1 >= t));
                        if (cnt >= p.K1) best = t;
                    }
                }
            } else {
                const uint4* rep4 = reinterpret_cast<const uint4*>(sm.report[slot]);
                uint32_t mine[kRepCap / 32];
                int reach[kRepCap / 32];
#pragma unroll
                for (int q = 0; q < kRepCap / 32; ++q) {
                    mine[q] = q * 32 + lane < n_rep ? sm.report[slot][q * 32 + lane] : 0xffffffffu;
                    reach[q] = 0;
                }
#pragma unroll 2
                for (int j = 0; j < (n_rep >> 2); ++j) {
                    const uint4 o = rep4[j];
#pragma unroll
                    for (int q = 0; q < kRepCap / 32; ++q)
                        reach[q] += (o.x >= mine[q]) + (o.y >= mine[q]) + (o.z >= mine[q]) + (o.w >= mine[q]);
                }
#pragma unroll
                for (int q = 0; q < kRepCap / 32; ++q) best = max(best, reach[q] >= p.K1 ? mine[q] : 0u);
            }
            best = __reduce_max_sync(kFullMask, best);
            if (best <= 0x007fffffu) best = 0;                       // nothing above -inf: no bound
            const float tau = best ? unord32(best) : neg_inf();      // no bound: everything is collected
            const uint32_t tau_key = best ? best : 1u;               // every lane key is above 0

            // the lanes that reach the bound, in (chunk, lane) order
            const int nc = it.n_chunks();
            int* hit_lanes = sm.hit_lane[rk];
            int n_hl = 0;
            {
                unsigned bal[kTeamWarps];
#pragma unroll
                for (int w = 0; w < kTeamWarps; ++w)
                    bal[w] = __ballot_sync(kFullMask, w < nc && sm.lane_key[slot][w][lane] >= tau_key);
                const unsigned below = (1u << lane) - 1u;
#pragma unroll
                for (int w = 0; w < kTeamWarps; ++w) {
                    const int at = n_hl + __popc(bal[w] & below);
                    if (((bal[w] >> lane) & 1u) && at < kHitCap) hit_lanes[at] = w * 32 + lane;
                    n_hl += __popc(bal[w]);
                }
            }
            __syncwarp();
            // their cells that reach the bound
            bool listed = n_hl <= kHitCap;
            int nh = 0;
            if (listed) {
#pragma unroll 1
                for (int h0 = 0; h0 < n_hl; h0 += 32) {
                    const int h = h0 + lane;
                    unsigned m = 0;
                    int w = 0, l = 0;
                    if (h < n_hl) {
                        const int wl = hit_lanes[h];
                        w = wl >> 5; l = wl & 31;
                        m = Vec<T>::reach_mask(sm.cell_max[slot][w][l], tau);
                        const int nvec_w = it.chunk_vecs(w);
                        if (nvec_w < kChunkVecs) {          // cells whose first vector lies beyond the row
#pragma unroll
                            for (int c = 0; c < 8; ++c)
                                if (Vec<T>::cell_pair(c) * 64 + l >= nvec_w) m &= ~(1u << c);
                        }
                    }
                    int incl = __popc(m);
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const int t = __shfl_up_sync(kFullMask, incl, o);
                        if (lane >= o) incl += t;
                    }
                    int pos = nh + incl - __popc(m);
                    while (m) {
                        const int cell = __ffs(m) - 1;
                        m &= m - 1;
                        if (pos < kHitCap) hits[pos] = ((w * kChunkVecs + Vec<T>::cell_pair(cell) * 64 + l) << 1) | Vec<T>::cell_parity(cell);
                        ++pos;
                    }
                    nh += __shfl_sync(kFullMask, incl, 31);
                }
                listed = nh <= kHitCap;
            }
            if (lane == 0) { sm.hit_n[slot][half] = listed ? nh : kHitCap + 1; sm.hit_bound[slot][half] = tau; }
            // The ranking warp must be done with the slot's previous item: then it has seen the previous list
            // being announced, and has read the sums that the team's next item will overwrite.
            if (!mbar_wait_warp(smem_u32(&sm.ranked[slot]), it.slot_phase() ^ 1u, abort_flag)) break;
            // nothing of the slot's shared maxima and reports is needed any more: let the team's next item in
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(&sm.slot_free[slot]));
                mbar_arrive(smem_u32(&sm.hits_ready[slot]));
            }
            it.skip(kSlots);
        }
    } else {
        // ------------------------------------------------------------------ ranking warp of slot rk
        const int rk = warp - kWarpRank;
        const uint32_t slot = (uint32_t)rk;
        uint64_t* keys = sm.key[rk];
        ItemIter it(p, (int)sizeof(T));
        it.skip(rk);
#pragma unroll 1
        for (;;) {
            if (!mbar_wait_warp(smem_u32(&sm.hits_ready[slot]), it.slot_phase(), abort_flag)) break;
            it.fetch(sm.item);
            if (!it.valid()) break;                       // no more items
            const int row = it.row();
            const uint32_t half = it.use() & 1u, use_phase = (it.use() >> 1) & 1u;
            const int nc = it.n_chunks();
            const int* hits = sm.hit[slot][half];
            const int nh = sm.hit_n[slot][half];
            const float tau = sm.hit_bound[slot][half];
            bool listed = nh <= kHitCap;
            const int elem0 = it.seg() * p.seg_len, n_elem = it.bytes() / (int)sizeof(T);
            const T* src = (const T*)p.logits + (int64_t)row * p.stride + elem0;
            int n = 0;
            if (listed) {
                // read the cells again, one per lane, and append the entries at or above the bound to `keys`
                const uint4* vec = reinterpret_cast<const uint4*>(src);
                const int nvec_item = it.bytes() >> 4;
#pragma unroll 1
                for (int h0 = 0; h0 < nh; h0 += 32) {
                    const int h = h0 + lane;
                    float x[8];
                    int at[8];
                    unsigned take = 0;
                    if (h < nh) {
                        const int d = hits[h], va = d >> 1;
                        const uint32_t ninf = Vec<T>::kNegInfWord;
                        const uint4 a = __ldg(vec + va);
                        const uint4 b = va + 32 < nvec_item ? __ldg(vec + va + 32) : make_uint4(ninf, ninf, ninf, ninf);
                        Vec<T>::cell_entries(a, b, va, d & 1, x, at);
#pragma unroll
                        for (int e = 0; e < 8; ++e) take |= (x[e] >= tau && at[e] < n_elem ? 1u : 0u) << e;
                    }
                    int incl = __popc(take);
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const int t = __shfl_up_sync(kFullMask, incl, o);
                        if (lane >= o) incl += t;
                    }
                    int pos = n + incl - __popc(take);
                    while (take) {                     // one entry, as a rule
                        const int e = __ffs(take) - 1;
                        take &= take - 1;
                        const float xa = e & 1 ? x[1] : x[0], xb = e & 1 ? x[3] : x[2], xc = e & 1 ? x[5] : x[4], xd = e & 1 ? x[7] : x[6];
                        const float xe = e & 2 ? xb : xa, xf = e & 2 ? xd : xc;
                        if (pos < kKeyCap) keys[pos] = row_key(e & 4 ? xf : xe, elem0 + at[0] + (at[1] - at[0]) * (e & 3) + (e & 4 ? at[4] - at[0] : 0));
                        ++pos;
                    }
                    n += __shfl_sync(kFullMask, incl, 31);
                }
                listed = n <= kKeyCap;
            }
            __syncwarp();

            // the segment's normaliser: sum_x 2^(x*log2e) = S * 2^C with a whole number C (fixed order of addition)
            const int64_t out = (int64_t)row * p.S + it.seg();
            if (!mbar_wait_warp(smem_u32(&sm.sums_in[slot][half]), use_phase, abort_flag)) break;
            {   // lane w holds warp w's part; whole-number references compare as integers
                const float cw2 = lane < nc ? sm.warp_ref[slot][half][lane] : neg_inf();
                const int ci = cw2 != neg_inf() ? __float2int_rn(cw2) : INT_MIN;
                const int Ci = __reduce_max_sync(kFullMask, ci);
                float part = ci != INT_MIN ? sm.warp_sum[slot][half][lane] * pow2i(ci - Ci) : 0.f;
#pragma unroll
                for (int o = 8; o; o >>= 1) part += __shfl_xor_sync(kFullMask, part, o);     // lanes 0..15 hold it all
                if (lane == 0) {
                    float m = neg_inf(), s2 = 0.f;
                    if (Ci != INT_MIN) {
                        // (m, s) with sum_x e^x = s * e^m: m = fl32(C ln2), the rounding of m folded into s
                        constexpr float kLn2Hi = 0.693147182464599609375f, kLn2Lo = -1.904654299957767e-9f;
                        const float C = (float)Ci;
                        m = C * kLn2Hi;
                        const float err = fmaf(C, kLn2Hi, -m) + C * kLn2Lo;
                        s2 = fmaf(part, err, part);
                    }
                    p.part_m[out] = m; p.part_s[out] = s2;
                }
            }

            float* tv = p.top_val + out * p.K1;
            int32_t* ti = p.top_idx + out * p.K1;
            if (listed) {
#pragma unroll 1
                for (int i = n + lane; i < p.K1; i += 32) { tv[i] = neg_inf(); ti[i] = -1; }
#pragma unroll 1
                for (int i = lane; i < n; i += 32) {
                    const uint64_t ki = keys[i];
                    int rank = 0;
#pragma unroll 8
                    for (int j = 0; j < n; ++j) rank += keys[j] > ki;
                    if (rank < p.K1) { tv[rank] = row_key_val(ki); ti[rank] = row_key_idx(ki); }
                }
            } else {
                if (lane == 0) atomicAdd(p.status + kStatusWordRescans, 1u);
                rank_from_global<T>((const T*)p.logits + (int64_t)row * p.stride, elem0, elem0 + n_elem, p.K1, tv, ti);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm.ranked[slot]));
            it.skip(kSlots);
        }
    }
    __syncthreads();
    if (tid == 0 && sm.ctl.abort_flag) {
        // winding down, whoever gave up: let the copies already issued land (bounded) before the CTA leaves
        const uint32_t n = sm.ctl.n_issued;
#pragma unroll 1
        for (uint32_t f = n > kSlots ? n - kSlots : 0; f < n; ++f)
            if ((int)f != p.drop_item)
                for (uint32_t i = 0; i < 100000 && !mbar_try_wait(smem_u32(&sm.full[f % kSlots]), (f / kSlots) & 1u); ++i) {}
        atomicOr(p.status, kStatusTimeout);
    }
}

}  // namespace

bool row_scan_tma_usable(const void* logits, int64_t stride, const Dims& d) {
    const int es = d.dtype == DBA_F32 ? 4 : 2;
    if (((uintptr_t)logits & 15u) || ((stride * es) & 15) || ((d.V * es) & 15)) return false;
    if ((d.seg_len * es) % kChunkBytes != 0 || d.seg_len * es > kTeamWarps * kChunkBytes) return false;
    return true;
}

size_t row_scan_tma_smem() { return sizeof(Smem) + 128; }

cudaError_t configure_row_scan_tma() {
    cudaError_t e = cudaFuncSetAttribute(row_scan_tma_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)row_scan_tma_smem());
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(row_scan_tma_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)row_scan_tma_smem());
}

cudaError_t launch_row_scan_tma(const void* logits, int64_t stride, const Dims& d, const int32_t* open_list,
                                const int32_t* open_count, int32_t* zero_count, const ScanScratch& part,
                                uint32_t* status, int sm_count, const ScanDebug& dbg, cudaStream_t st) {
    Params p;
    p.logits = logits; p.stride = stride; p.V = d.V; p.S = d.S; p.seg_len = d.seg_len; p.K1 = d.K1; p.R = d.R;
    p.open_list = open_list; p.open_count = open_count; p.zero_count = zero_count;
    // the work counter: with a list of open rows, the word two places after its count (the step alternates between
    // two counts, and so between two counters: each launch clears the other's); else a word of the status block,
    // which the caller has just cleared
    p.ticket = open_count ? const_cast<int32_t*>(open_count) + 2 : reinterpret_cast<int32_t*>(status) + kStatusWordTicket;
    p.zero_ticket = open_count && zero_count ? zero_count + 2 : nullptr;
    p.part_m = part.m; p.part_s = part.s; p.top_val = part.val; p.top_idx = part.idx; p.status = status;
    p.wait_clocks = dbg.wait_clocks > 0 ? dbg.wait_clocks : 2000000000LL;       // about a second: a wait this long has failed
    p.drop_item = dbg.drop_item;
    const int64_t items = (int64_t)d.R * d.S;
    const int grid = (int)(items < sm_count ? items : sm_count);
    if (d.dtype == DBA_F32) return launch_after(row_scan_tma_kernel<float>, dim3(grid), dim3(kThreads), row_scan_tma_smem(), st, p);
    return launch_after(row_scan_tma_kernel<__nv_bfloat16>, dim3(grid), dim3(kThreads), row_scan_tma_smem(), st, p);
}

}  // namespace dba
