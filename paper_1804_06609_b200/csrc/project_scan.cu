// Output projection fused with the row scan (Section 2: DECODER-STEP's last stage produces the k x |V_T| matrix
// that Algorithm 2 reads): logits[r, w] = <hidden[r, :], embed[w, :]> are computed on the tensor cores and
// consumed where they appear, so the R x V matrix never exists in HBM.
//
// Persistent CTAs in pairs (a cluster of two, one CTA per SM).  A pair works on tiles of 256 rows of hidden states
// x 256 words: each CTA holds its 128 rows of the hidden states and its 128 words of the embedding slice in shared
// memory, and one tcgen05.mma of the pair (cta_group::2, issued by the pair's first CTA) multiplies the 256 x 256
// tile, each CTA receiving the accumulator of its own 128 rows in its tensor memory.  That halves what each SM
// has to fetch of the embedding, which is what bounds a single CTA on a 128 x 256 tile.  The tiles are numbered row
// block by row block and dealt out to the pairs in equal contiguous runs, so a pair works through part of one row
// block's vocabulary (and possibly the start of the next row block's).  Roles in each CTA, talking through mbarriers:
//   warp 0    one thread issues the TMA loads (cp.async.bulk.tensor, cta_group::2, each CTA for itself) of the 64-deep
//             slices of this CTA's halves of both operands into a ring of shared-memory stages (128-byte swizzle);
//             the bytes of both CTAs are counted on the first CTA's barrier;
//   warp 1    allocates tensor memory (both CTAs); in the first CTA one thread issues the pair's tcgen05.mma
//             (256 x 256 x 16, bf16 in, fp32 out) into one of two accumulators and commits the stage back to both
//             loaders, and the finished accumulator to both epilogues;
//   warps 4-11 the epilogue: two warpgroups, one per accumulator, each taking every other tile of the run.  A thread
//             owns one row of the tile (the four warps of a group reach the four quarters of the CTA's rows).  It
//             reads its 256 logits from tensor memory, 32 at a time, and keeps, over all its tiles of the run:
//             the sum of 2^(x log2e - c) against a whole-number
//             reference c (raised with an exact rescaling when a logit exceeds it), and the candidates for the row's
//             K1 largest logits.  Selection: logits at or above a bound tau (none at first) go to the thread's list
//             in shared memory (found as a bit mask over the 32 columns); when a list is full, every thread of the
//             warp raises its tau to the K1-th largest entry of its list (to 16 bits, by a radix selection over the
//             list held in registers) and drops what fell below, so a list settles at K1 entries plus whatever
//             arrived since.  The bound is shared among all threads working on the same row (an atomic maximum in
//             global memory, read again before every tile).
// At the end of its part of a row block the thread writes its sum and its list (at least K1 entries, all that reach
// the final tau) as one piece of the row; project_merge_kernel
// orders the pieces of a row exactly and writes the row's normaliser and its K1 best entries in the row scan's format.
// Every wait on an mbarrier is bounded: a wait that runs out sets the timeout bit of the status word and the
// CTA winds down (the tensor memory is freed on every path); the two CTAs of a pair leave together.
#include <climits>

#include <cuda.h>
#include <cuda_bf16.h>

#include "dba_device.cuh"
#include "dba_internal.h"

namespace dba {

namespace {

constexpr int kBM = 128;                 // rows of hidden states per CTA and tile (= lanes of tensor memory)
constexpr int kPairM = 2 * kBM;          // rows of a pair's tile
constexpr int kBN = 256;                 // words per tile (= columns of one accumulator)
constexpr int kHalfN = kBN / 2;          // words of the tile whose embedding rows this CTA holds
constexpr int kBK = 64;                  // depth of a stage: 64 bf16 = 128 bytes, one swizzle row
constexpr int kPStages = 4;
constexpr int kStageA = kBM * kBK * 2;   // 16 KB
constexpr int kStageB = kHalfN * kBK * 2; // 16 KB
constexpr int kListCap = 48;             // candidates a thread may hold (K1 <= 32 of them settled, the rest arrivals)
constexpr int kEpiGroups = 2;            // epilogue warpgroups: one per accumulator, each taking every other tile
constexpr int kEpiThreads = 128 * kEpiGroups;
constexpr int kRefreshSlack = 8;         // arrivals beyond K1 after which a list is tidied at the next tile
constexpr int kMaxRunTiles = 256;        // tiles a CTA may work through: columns are kept relative to its first one, in 16 bits
constexpr int kProjThreads = 128 + kEpiThreads;
constexpr int kTmemCols = 512;           // two accumulators of 256 columns
constexpr long long kProjWaitClocks = 4000000000LL;      // about two seconds: a wait this long has failed (the default)

struct ProjWait {
    int abort_flag;                  // a wait has run out: every role leaves at its next wait
    long long wait_clocks;           // how long a wait may last
};

struct ProjSmem {
    alignas(1024) unsigned char a[kPStages][kStageA];
    alignas(1024) unsigned char b[kPStages][kStageB];
    uint32_t list_key[kListCap][kEpiThreads];   // entry e of thread t at [e][t] (no bank conflicts): the logit as an ordered integer
    uint16_t list_col[kListCap][kEpiThreads];  // its column, counted from the first column of the CTA's part of the row block
    uint64_t full[kPStages];         // (first CTA's) the stage's operands have landed in both CTAs
    uint64_t empty[kPStages];        // the stage's MMAs are done
    uint64_t acc_full[2];            // the accumulator holds a finished tile
    uint64_t acc_empty[2];           // (first CTA's) the epilogues of both CTAs have read the accumulator
    uint32_t tmem_base;
    ProjWait ctl;
};

struct ProjParams {
    int R, V, D, K1;
    int tiles_m, tiles_n;            // tiles (of a pair) along rows and along the vocabulary
    int pieces;                      // most pieces a row may have (stride of the per-piece arrays)
    ProjPieces out;
    uint32_t* row_tau;               // [R] zero before the launch: the highest bound any piece of the row has reached so far
    uint32_t* status;
    long long wait_clocks;           // how long a wait may last
    int drop_item;                   // testing: the first CTA of every pair announces the copies of this slice of its sequence but never issues them
};

__device__ __forceinline__ uint32_t psmem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void pbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void pbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool pbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  False: the CTA is winding down (this wait ran out, or another one did).
__device__ __noinline__ bool pbar_wait(uint32_t bar, uint32_t parity, volatile ProjWait* ctl) {
    const long long limit = ctl->wait_clocks;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 32; ++i)
            if (pbar_try_wait(bar, parity)) return true;
        if (ctl->abort_flag) return false;
        if (clock64() - t0 > limit) break;
    }
    ctl->abort_flag = 1;
    return false;
}
// 2-D tiled TMA load for this CTA alone: box at (x = element along the row, y = row) of the tensor map, into this CTA's
// shared memory; the bytes are counted on `bar`, a shared::cluster address that may be the other CTA of the pair's
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
// shared::cluster address of this CTA's shared-memory address `local` in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t cluster_addr(uint32_t local, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
    return r;
}
__device__ __forceinline__ void pbar_arrive_cluster(uint32_t bar_cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Shared-memory operand descriptor of a K-major tile stored as rows of 128 bytes with the 128-byte swizzle:
// start address, leading offset 1 (unused with a swizzle), 1024 bytes from one group of eight rows to the next,
// descriptor version 1, layout type "128-byte swizzle".
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3fffu);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, N = 256, M = 256 (the pair's), dense, no negation.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(kPairM >> 4) << 24);

// one MMA of the pair: the descriptors name the same shared-memory places in both CTAs, the accumulator the same
// columns of both tensor memories; no output lane is masked
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t accumulate) {
    const uint32_t zero = 0;
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(kIdesc), "r"(accumulate), "r"(zero) : "memory");
}
// arrives on the mbarrier at this place in both CTAs of the pair once every MMA issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    const uint16_t both = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(both) : "memory");
}
__device__ __forceinline__ void tmem_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// 32 consecutive columns of this thread's lane of tensor memory
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* r) {
    uint32_t u[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]),
          "=r"(u[8]), "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15]),
          "=r"(u[16]), "=r"(u[17]), "=r"(u[18]), "=r"(u[19]), "=r"(u[20]), "=r"(u[21]), "=r"(u[22]), "=r"(u[23]),
          "=r"(u[24]), "=r"(u[25]), "=r"(u[26]), "=r"(u[27]), "=r"(u[28]), "=r"(u[29]), "=r"(u[30]), "=r"(u[31])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) r[i] = __uint_as_float(u[i]);
}
__device__ __forceinline__ float pex2(float t) { float r; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(t)); return r; }
__device__ __forceinline__ float ppow2i(int d) { return d < -126 ? 0.f : __int_as_float((d + 127) << 23); }

constexpr float kPLog2e = 1.44269502162933349609375f;
constexpr float kPNoRef = -1.0e30f;
constexpr float kTauNone = -3.402823466e38f;     // no bound yet: every finite logit reaches it, -inf does not

__global__ void __launch_bounds__(kProjThreads, 1)
project_scan_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, ProjParams p) {
    extern __shared__ __align__(1024) unsigned char psmem_raw[];
    // the operand tiles want 1024-byte alignment (the swizzle pattern repeats every 1024 bytes)
    ProjSmem& sm = *reinterpret_cast<ProjSmem*>(psmem_raw + ((1024u - (psmem_u32(psmem_raw) & 1023u)) & 1023u));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile ProjWait* abort_flag = &sm.ctl;

    // the pair, this CTA's place in it (0: the CTA that issues the MMAs and whose barriers count for both), and
    // the pair's run of tiles
    const uint32_t rank = cluster_rank();
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const long long n_tiles = (long long)p.tiles_m * p.tiles_n;
    const int t_begin = (int)((long long)pair * n_tiles / n_pairs);
    const int t_end = (int)((long long)(pair + 1) * n_tiles / n_pairs);
    const int k_blocks = (p.D + kBK - 1) / kBK;

    if (tid == 0) {
        for (int s = 0; s < kPStages; ++s) { pbar_init(psmem_u32(&sm.full[s]), 1); pbar_init(psmem_u32(&sm.empty[s]), 1); }
        for (int a = 0; a < 2; ++a) { pbar_init(psmem_u32(&sm.acc_full[a]), 1); pbar_init(psmem_u32(&sm.acc_empty[a]), 2 * 4); }   // the four warps of one group in each CTA
        sm.ctl.abort_flag = 0; sm.ctl.wait_clocks = p.wait_clocks;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {       // tensor memory: the whole of it in both CTAs (the same warp of each asks), for two accumulators
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(psmem_u32(&sm.tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tmem_fence_before();
    __syncthreads();
    cluster_sync_all();        // the other CTA's barriers exist before anything is signalled on them
    tmem_fence_after();
    const uint32_t tmem_base = sm.tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ loader
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
            uint32_t n = 0;
            bool ok = true;
#pragma unroll 1
            for (int t = t_begin; t < t_end && ok; ++t) {
                const int m = t / p.tiles_n, nn = t - m * p.tiles_n;
#pragma unroll 1
                for (int kb = 0; kb < k_blocks; ++kb, ++n) {
                    const uint32_t s = n % kPStages, use = n / kPStages;
                    if (use > 0 && !pbar_wait(psmem_u32(&sm.empty[s]), (use - 1) & 1u, abort_flag)) { ok = false; break; }
                    // both CTAs' bytes are counted on the first CTA's barrier, which that CTA arms
                    if (rank == 0) pbar_expect_tx(psmem_u32(&sm.full[s]), 2 * (kStageA + kStageB));
                    const uint32_t bar = cluster_addr(psmem_u32(&sm.full[s]), 0);
                    if (rank == 0 && (int)n == p.drop_item) continue;
                    tma_load_2d(psmem_u32(sm.a[s]), &map_a, kb * kBK, m * kPairM + (int)rank * kBM, bar);
                    tma_load_2d(psmem_u32(sm.b[s]), &map_b, kb * kBK, nn * kBN + (int)rank * kHalfN, bar);
                }
            }
            // winding down: let the loads already issued (by both CTAs: the pair leaves together, after this) land
            if (!ok && rank == 0) {
                for (uint32_t f = n > kPStages ? n - kPStages : 0; f < n; ++f) {
                    if ((int)f == p.drop_item) continue;
                    for (uint32_t i = 0; i < 100000 && !pbar_try_wait(psmem_u32(&sm.full[f % kPStages]), (f / kPStages) & 1u); ++i) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (first CTA of the pair)
        if (lane == 0 && rank == 0) {
            uint32_t n = 0, tile_no = 0;
            bool ok = true;
#pragma unroll 1
            for (int t = t_begin; t < t_end && ok; ++t, ++tile_no) {
                const uint32_t acc = tile_no & 1u, acc_use = tile_no >> 1;
                if (acc_use > 0 && !pbar_wait(psmem_u32(&sm.acc_empty[acc]), (acc_use - 1) & 1u, abort_flag)) { ok = false; break; }
                tmem_fence_after();
                const uint32_t d_addr = tmem_base + acc * kBN;
#pragma unroll 1
                for (int kb = 0; kb < k_blocks; ++kb, ++n) {
                    const uint32_t s = n % kPStages, use = n / kPStages;
                    if (!pbar_wait(psmem_u32(&sm.full[s]), use & 1u, abort_flag)) { ok = false; break; }
                    tmem_fence_after();
                    const uint64_t da = umma_desc_sw128(psmem_u32(sm.a[s])), db = umma_desc_sw128(psmem_u32(sm.b[s]));
#pragma unroll
                    for (int k4 = 0; k4 < kBK / 16; ++k4)      // 16 bf16 = 32 bytes further along the swizzled row
                        umma_bf16(d_addr, da + (uint64_t)(k4 * 2), db + (uint64_t)(k4 * 2), (kb | k4) != 0 ? 1u : 0u);
                    umma_commit(psmem_u32(&sm.empty[s]));       // the stage may be refilled when these are done
                }
                if (ok) umma_commit(psmem_u32(&sm.acc_full[acc]));
            }
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ epilogue: a row of every other tile per thread
        const int et = tid - 128;                          // 0..255: place of this thread's list
        const int grp = (warp - 4) >> 2;                   // takes the tiles in accumulator grp (every other tile of the run)
        const int trow = et & 127;                         // row of this CTA's half of the tile = lane of tensor memory
        const int row_in_tile = (int)rank * kBM + trow;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        float cref = kPNoRef, sum = 0.f, tau = kTauNone;
        uint32_t tau_key = 0;              // tau as an ordered integer (0: none yet)
        int n_list = 0;
        bool lost = false;                 // a candidate found no room in the list: the piece cannot be trusted
        int cur_m = -1, col_first = 0;     // row block being worked on, and the first column of this CTA's part of it
        bool ok = true;
        uint32_t tile_no = 0;

        auto compact = [&]() {         // raise tau to the K1-th largest entry of the list (to 16 bits) and drop what is below
            if (n_list < p.K1) return;
            // the keys come into registers once (empty places as key 0, below every real key); the selection
            // then runs on registers alone
            uint32_t key[kListCap];
#pragma unroll
            for (int e = 0; e < kListCap; ++e) key[e] = e < n_list ? sm.list_key[e][et] : 0u;
            uint32_t best = 0;         // the largest t, a multiple of 2^16, that at least K1 keys reach
#pragma unroll 1
            for (uint32_t bit = 0x80000000u; bit >= 0x00010000u; bit >>= 1) {
                const uint32_t t = best | bit;
                int cnt = 0;
#pragma unroll
                for (int e = 0; e < kListCap; ++e) cnt += key[e] >= t;
                if (cnt >= p.K1) best = t;
            }
            if (best <= 0x007fffffu) best = 0;
            // A row's pieces are worked on at the same time by other threads (of this CTA and of others): the K1-th
            // largest entry of any piece bounds the row's K1-th largest from below, so the pieces share the highest
            // bound found.
            if (best > tau_key) {
                tau_key = best;
                if (cur_m * kPairM + row_in_tile < p.R) atomicMax(p.row_tau + cur_m * kPairM + row_in_tile, best);
            }
            best = tau_key;
            tau = tau_key ? unord32(tau_key) : kTauNone;
            int kept = 0;
#pragma unroll
            for (int e = 0; e < kListCap; ++e)
                if (e < n_list && key[e] >= best) {
                    const uint16_t c = sm.list_col[e][et];     // (kept <= e: nothing unread is overwritten)
                    sm.list_key[kept][et] = key[e]; sm.list_col[kept][et] = c; ++kept;
                }
            n_list = kept;
        };
        auto flush = [&](int m, int piece) {      // write this thread's piece of row m * kPairM + row_in_tile
            compact();
            const int row = m * kPairM + row_in_tile;
            if (row < p.R) {
                if (lost) atomicOr(p.status, kStatusOverflow);
                const int64_t slot = (int64_t)row * p.pieces + piece * kEpiGroups + grp;
                p.out.ref[slot] = cref != kPNoRef ? __float2int_rn(cref) : INT_MIN;
                p.out.sum[slot] = sum;
                p.out.n[slot] = n_list;
                for (int e = 0; e < n_list; ++e) {
                    p.out.val[slot * kListCap + e] = unord32(sm.list_key[e][et]);
                    p.out.col[slot * kListCap + e] = col_first + (int)sm.list_col[e][et];
                }
            }
        };
        // piece of row block m that pair c writes = c - (pair that owns the row block's first tile)
        auto first_cta = [&](int m) {
            const long long t0 = (long long)m * p.tiles_n;
            // largest c with c * n_tiles / grid <= t0
            long long c = ((t0 + 1) * n_pairs - 1) / n_tiles;
            while (c > 0 && c * n_tiles / n_pairs > t0) --c;
            while ((c + 1) * n_tiles / n_pairs <= t0) ++c;
            return (int)c;
        };

#pragma unroll 1
        for (int t = t_begin; t < t_end && ok; ++t, ++tile_no) {
            const int m = t / p.tiles_n, nn = t - m * p.tiles_n;
            if (m != cur_m) {          // (both groups pass here, whoever gets the row block's first tile)
                if (cur_m >= 0) flush(cur_m, pair - first_cta(cur_m));
                cur_m = m; col_first = nn * kBN;
                cref = kPNoRef; sum = 0.f; tau = kTauNone; tau_key = 0; n_list = 0; lost = false;
            }
            if ((tile_no & 1u) != (uint32_t)grp) continue;
            const uint32_t acc = (uint32_t)grp, acc_use = tile_no >> 1;
            // what the row's other pieces have found meanwhile (asked for before the wait, used after it)
            const bool live = m * kPairM + row_in_tile < p.R;            // (the last row block may reach past the last row)
            uint32_t seen = 0;
            if (live) asm volatile("ld.global.cg.u32 %0, [%1];" : "=r"(seen) : "l"(p.row_tau + m * kPairM + row_in_tile));
            // a list that has grown since its bound was last raised is tidied while the tile is still being computed
            if (__any_sync(kFullMask, n_list >= p.K1 + kRefreshSlack)) compact();
            if (!__all_sync(kFullMask, pbar_wait(psmem_u32(&sm.acc_full[acc]), acc_use & 1u, abort_flag))) { ok = false; break; }
            tmem_fence_after();
            if (seen > tau_key) { tau_key = seen; tau = unord32(seen); }
            const int col0 = nn * kBN;
            const bool ragged = col0 + kBN > p.V;           // the vocabulary ends inside this tile
#pragma unroll 1
            for (int ch = 0; ch < kBN / 32; ++ch) {
                float x[32];
                tmem_ld32(tmem_base + lane_base + acc * kBN + ch * 32, x);
                const int cbase = col0 + ch * 32;
                if (ragged) {
#pragma unroll
                    for (int c = 0; c < 32; ++c) if (cbase + c >= p.V) x[c] = neg_inf();
                }
                float cm = neg_inf();
#pragma unroll
                for (int c = 0; c < 32; ++c) cm = fmaxf(cm, x[c]);
                // candidates: the columns at or above the bound (a finite number, so -inf never is), as a bit mask;
                // they go to the list eight columns at a time, and a list that is full is tidied (which raises
                // the bound) before the rest is looked at again
                if (__any_sync(kFullMask, live && cm >= tau)) {
                    uint32_t mk = 0;
#pragma unroll
                    for (int c = 0; c < 32; ++c) mk |= (x[c] >= tau ? 1u : 0u) << c;
                    if (!live) mk = 0;
#pragma unroll 1
                    for (int round = 0; ; ++round) {
                        uint32_t pending = 0;
#pragma unroll
                        for (int g8 = 0; g8 < 4; ++g8) {
                            uint32_t sub = (mk >> (8 * g8)) & 0xffu;
                            while (sub) {
                                if (n_list == kListCap) { pending |= sub << (8 * g8); break; }
                                const int c = __ffs(sub) - 1;
                                sub &= sub - 1;
                                const float a0 = (c & 1) ? x[g8 * 8 + 1] : x[g8 * 8], a1 = (c & 1) ? x[g8 * 8 + 3] : x[g8 * 8 + 2];
                                const float a2 = (c & 1) ? x[g8 * 8 + 5] : x[g8 * 8 + 4], a3 = (c & 1) ? x[g8 * 8 + 7] : x[g8 * 8 + 6];
                                const float b0 = (c & 2) ? a1 : a0, b1 = (c & 2) ? a3 : a2;
                                const float v = (c & 4) ? b1 : b0;
                                sm.list_key[n_list][et] = ord32(v);
                                sm.list_col[n_list][et] = (uint16_t)(cbase + g8 * 8 + c - col_first);
                                ++n_list;
                            }
                        }
                        // (the loop is left by the whole warp together: the votes inside it name every lane)
                        if (!__any_sync(kFullMask, pending != 0)) break;
                        compact();
                        if (pending != 0 && (n_list == kListCap || round >= 8)) { lost = true; pending = 0; }   // more ties than places
                        mk = 0;
#pragma unroll
                        for (int c = 0; c < 32; ++c) mk |= (x[c] >= tau ? 1u : 0u) << c;
                        mk &= pending;
                    }
                }
                // the normaliser
                const float need = cm * kPLog2e;
                if (need > cref + 8.f) {
                    const float cn = ceilf(need);
                    const float dd = cref - cn;
                    sum *= dd < -126.f ? 0.f : ppow2i((int)dd);
                    cref = cn;
                }
                float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
                for (int c = 0; c < 32; c += 4) {
                    s0 += pex2(fmaf(x[c], kPLog2e, -cref)); s1 += pex2(fmaf(x[c + 1], kPLog2e, -cref));
                    s2 += pex2(fmaf(x[c + 2], kPLog2e, -cref)); s3 += pex2(fmaf(x[c + 3], kPLog2e, -cref));
                }
                sum += (s0 + s1) + (s2 + s3);
            }
            // the accumulator may be overwritten
            tmem_fence_before();
            __syncwarp();
            if (lane == 0) pbar_arrive_cluster(cluster_addr(psmem_u32(&sm.acc_empty[acc]), 0));
        }
        if (ok && cur_m >= 0) flush(cur_m, pair - first_cta(cur_m));
    }
    // the pair leaves together: neither CTA's shared memory, barriers or tensor memory may go while the other
    // could still signal or use them
    tmem_fence_before();
    __syncthreads();
    cluster_sync_all();
    tmem_fence_after();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    if (tid == 0 && sm.ctl.abort_flag) atomicOr(p.status, kStatusTimeout);
}

// Orders the pieces of every row exactly: one warp per row adds up the pieces' sums (in the order of the pieces),
// gathers their candidates into shared memory, finds the value of the K1-th largest a byte at a time (a histogram
// of the next byte over the entries that share the bytes found so far) and ranks the entries that reach it
// (value descending, lower column first).  Global memory is read in batches of independent loads: a row costs a
// few round trips to L2, not one per piece.
constexpr int kMergeWarps = 4;
constexpr int kMergeKeys = 1024;         // entries of a row that fit in shared memory (more: they are read in place)
constexpr int kMergeBuf = 128;           // entries at or above the K1-th largest value that are ranked the short way
__global__ void __launch_bounds__(kMergeWarps * 32) project_merge_kernel(ProjParams p, int grid_scan, RowTop top) {
    __shared__ uint64_t s_key[kMergeWarps][kMergeKeys];
    __shared__ uint32_t s_hist[kMergeWarps][256];
    const int row = blockIdx.x * kMergeWarps + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    if (row >= p.R) return;
    // a scan that gave up (a wait that ran out, a list that overflowed) has not written every piece: nothing is
    // read, the row's results stay what they were, and the failure is reported from the status word
    if (*reinterpret_cast<volatile uint32_t*>(p.status) & (kStatusTimeout | kStatusOverflow)) return;
    const long long n_tiles = (long long)p.tiles_m * p.tiles_n;
    const int m = row / kPairM;
    // pairs that own the first and the last tile of this row block
    auto owner = [&](long long t) {
        long long c = ((t + 1) * grid_scan - 1) / n_tiles;
        while (c > 0 && c * n_tiles / grid_scan > t) --c;
        while ((c + 1) * n_tiles / grid_scan <= t) ++c;
        return (int)c;
    };
    const int c0 = owner((long long)m * p.tiles_n), c1 = owner((long long)(m + 1) * p.tiles_n - 1);
    const int n_pieces = (c1 - c0 + 1) * kEpiGroups;
    const int64_t base = (int64_t)row * p.pieces;
    const unsigned lt_mask = (1u << lane) - 1u;
    uint64_t* keys = s_key[wib];
    uint32_t* hist = s_hist[wib];

    // ---- normaliser: highest reference first, then the sums rescaled to it, added in the order of the pieces
    int C = INT_MIN;
    for (int g0 = 0; g0 < n_pieces; g0 += 32) {
        const int g = g0 + lane;
        C = max(C, g < n_pieces ? p.out.ref[base + g] : INT_MIN);
    }
    C = __reduce_max_sync(kFullMask, C);
    float total = 0.f;
    int total_n = 0, n_first = 0;          // n_first: lane g holds the length of piece g (the first 32 pieces)
    for (int g0 = 0; g0 < n_pieces; g0 += 32) {
        const int g = g0 + lane;
        float term = 0.f; int ng = 0;
        if (g < n_pieces) {
            const int ref = p.out.ref[base + g];
            if (ref != INT_MIN) term = p.out.sum[base + g] * ppow2i(ref - C);
            ng = p.out.n[base + g];
        }
        for (int j = 0; j < min(32, n_pieces - g0); ++j) total += __shfl_sync(kFullMask, term, j);
        total_n += __reduce_add_sync(kFullMask, ng);
        if (g0 == 0) n_first = ng;
    }
    if (lane == 0) {
        float lse = neg_inf();
        if (C != INT_MIN && total > 0.f) {
            constexpr float kLn2Hi = 0.693147182464599609375f, kLn2Lo = -1.904654299957767e-9f;
            const float c = (float)C, hi = c * kLn2Hi, lo = fmaf(c, kLn2Hi, -hi) + c * kLn2Lo;
            lse = hi + (logf(total) + lo);
        }
        top.lse[row] = lse;
    }

    // ---- candidates
    float* tv = top.val + (int64_t)row * p.K1;
    int32_t* ti = top.idx + (int64_t)row * p.K1;
    const bool in_smem = total_n <= kMergeKeys;
    if (in_smem) {            // all entries to shared memory, as keys (value above, inverted column below)
        static_assert(kListCap <= 64, "a piece is read in two rounds of 32");
        int at = 0;
#pragma unroll 4
        for (int g = 0; g < n_pieces; ++g) {
            const int ng = g < 32 ? __shfl_sync(kFullMask, n_first, g) : p.out.n[base + g];
            const int64_t pb = (base + g) * kListCap;
            const bool h0 = lane < ng, h1 = lane + 32 < ng;
            float v0 = 0.f, v1 = 0.f; int w0 = 0, w1 = 0;
            if (h0) { v0 = p.out.val[pb + lane]; w0 = p.out.col[pb + lane]; }
            if (h1) { v1 = p.out.val[pb + lane + 32]; w1 = p.out.col[pb + lane + 32]; }
            if (h0) keys[at + lane] = row_key(v0, w0);
            if (h1) keys[at + lane + 32] = row_key(v1, w1);
            at += ng;
        }
        __syncwarp();
    }
    // visits the value (as an ordered integer) of every entry of the row
    auto for_each_value = [&](auto&& f) {
        if (in_smem) {
            for (int i = lane; i < total_n; i += 32) f((uint32_t)(keys[i] >> 32));
        } else {
            for (int g = 0; g < n_pieces; ++g) {
                const int ng = p.out.n[base + g];
                for (int e = lane; e < ng; e += 32) f(ord32(p.out.val[(base + g) * kListCap + e]));
            }
        }
    };
    uint32_t thr = 0;                       // ordered-integer value of the K1-th largest entry (0: there are no more than K1)
    if (total_n > p.K1) {
        uint32_t prefix = 0, prefix_mask = 0;
        int need = p.K1;                    // the entry looked for is the need-th largest of those that share the prefix
        for (int shift = 24; shift >= 0; shift -= 8) {
            for (int i = lane; i < 256; i += 32) hist[i] = 0;
            __syncwarp();
            for_each_value([&](uint32_t k32) {
                if ((k32 & prefix_mask) == prefix) atomicAdd(&hist[(k32 >> shift) & 255u], 1u);
            });
            __syncwarp();
            // lane l holds bytes 8l .. 8l+7; the byte wanted is the highest one with (entries above it) < need
            uint32_t bins[8], mine = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) { bins[j] = hist[lane * 8 + j]; mine += bins[j]; }
            uint32_t above = mine;          // entries in this lane's bytes and all higher ones
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t up = __shfl_down_sync(kFullMask, above, o);
                if (lane + o < 32) above += up;
            }
            above -= mine;                  // entries in higher lanes' bytes only
            const bool here = above < (uint32_t)need && above + mine >= (uint32_t)need;
            int digit = 0; uint32_t over = 0;
            if (here) {
                uint32_t acc = above;
                bool found = false;
#pragma unroll
                for (int j = 7; j >= 0; --j) {
                    if (!found && acc + bins[j] >= (uint32_t)need) { digit = lane * 8 + j; over = acc; found = true; }
                    acc += bins[j];
                }
            }
            const int src = __ffs(__ballot_sync(kFullMask, here)) - 1;      // exactly one lane
            digit = __shfl_sync(kFullMask, digit, src); over = __shfl_sync(kFullMask, over, src);
            need -= (int)over;
            prefix |= (uint32_t)digit << shift; prefix_mask |= 255u << shift;
            __syncwarp();
        }
        thr = prefix;
    }
    // the entries that reach the value, to the front of a short list
    uint64_t* buf = reinterpret_cast<uint64_t*>(hist);         // (the histogram is done with: 256 words = 128 keys)
    static_assert(kMergeBuf * 2 <= 256, "the short list lives where the histogram was");
    int cnt = 0;
    auto take = [&](bool valid, uint64_t key) {
        const bool hit = valid && (uint32_t)(key >> 32) >= thr;
        const unsigned bal = __ballot_sync(kFullMask, hit);
        const int pos = cnt + __popc(bal & lt_mask);
        if (hit && pos < kMergeBuf) buf[pos] = key;
        cnt += __popc(bal);
    };
    if (in_smem) {
        for (int i0 = 0; i0 < total_n; i0 += 32) take(i0 + lane < total_n, i0 + lane < total_n ? keys[i0 + lane] : 0ull);
    } else {
        for (int g = 0; g < n_pieces; ++g) {
            const int ng = p.out.n[base + g];
            for (int e0 = 0; e0 < ng; e0 += 32) {
                const int e = e0 + lane;
                take(e < ng, e < ng ? row_key(p.out.val[(base + g) * kListCap + e], p.out.col[(base + g) * kListCap + e]) : 0ull);
            }
        }
    }
    __syncwarp();
    if (cnt <= kMergeBuf) {
        for (int e = cnt + lane; e < p.K1; e += 32) { tv[e] = neg_inf(); ti[e] = -1; }
        for (int i = lane; i < cnt; i += 32) {
            const uint64_t key = buf[i];
            int rank = 0;
            for (int j = 0; j < cnt; ++j) rank += buf[j] > key;
            if (rank < p.K1) { tv[rank] = row_key_val(key); ti[rank] = (int32_t)(0xffffffffu - (uint32_t)key); }
        }
        return;
    }
    // (more entries tied with the K1-th largest than the short way holds: every entry is ranked among all of them)
    for (int e = total_n + lane; e < p.K1; e += 32) { tv[e] = neg_inf(); ti[e] = -1; }
    for (int g = 0; g < n_pieces; ++g) {
        const int ng = p.out.n[base + g];
        for (int e = lane; e < ng; e += 32) {
            const float x = p.out.val[(base + g) * kListCap + e];
            const int w = p.out.col[(base + g) * kListCap + e];
            const uint64_t key = row_key(x, w);
            int rank = 0;
            for (int g2 = 0; g2 < n_pieces; ++g2) {
                const int n2 = p.out.n[base + g2];
                for (int e2 = 0; e2 < n2; ++e2)
                    rank += row_key(p.out.val[(base + g2) * kListCap + e2], p.out.col[(base + g2) * kListCap + e2]) > key;
            }
            if (rank < p.K1) { tv[rank] = x; ti[rank] = w; }
        }
    }
}

// One CTA per sentence; its warps share out the (row, constraint position) pairs: the inner products
// <hidden[r], embed[token j]>, fp32, lanes striding over D two entries at a time (the sentence's rows and tokens
// stay in L1 while its warps go over them).
constexpr int kGatherWarps = 32;
__global__ void __launch_bounds__(kGatherWarps * 32)
constraint_logits_kernel(const __nv_bfloat16* __restrict__ hidden, int64_t hs, const __nv_bfloat16* __restrict__ embed,
                         int64_t es, int D, int k, const SentCons* __restrict__ cons, float* __restrict__ out) {
    const int b = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const SentCons& sc = cons[b];
    const int C = sc.C;
    for (int item = warp; item < k * C; item += kGatherWarps) {
        const int h = item / C, j = item - h * C;
        const int r = b * k + h;
        const uint32_t* e = reinterpret_cast<const uint32_t*>(embed + (int64_t)sc.ctok[j] * es);
        const uint32_t* x = reinterpret_cast<const uint32_t*>(hidden + (int64_t)r * hs);
        float acc = 0.f;
#pragma unroll 4
        for (int i = lane; i < D / 2; i += 32) {
            const uint32_t xw = __ldg(x + i), ew = __ldg(e + i);
            acc = fmaf(__uint_as_float(xw << 16), __uint_as_float(ew << 16), acc);
            acc = fmaf(__uint_as_float(xw & 0xffff0000u), __uint_as_float(ew & 0xffff0000u), acc);
        }
        acc = warp_sum(acc);
        if (lane == 0) out[(int64_t)r * kMaxC + j] = acc;
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)f;
    }
    return fn;
}

// [rows, D] bf16 row-major, rows `stride` elements apart: boxes of 64 elements x box_rows rows, 128-byte swizzle,
// zero fill beyond the edges
bool make_map(CUtensorMap* map, const void* base, int rows, int D, int64_t stride, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)stride * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

cudaError_t launch_constraint_logits(const void* hidden, int64_t hidden_stride, const void* embed, int64_t embed_stride,
                                     int D, const Dims& d, const SentCons* cons, float* out, cudaStream_t st, int* launches) {
    constraint_logits_kernel<<<d.B, kGatherWarps * 32, 0, st>>>(
        (const __nv_bfloat16*)hidden, hidden_stride, (const __nv_bfloat16*)embed, embed_stride, D, d.k, cons, out);
    ++*launches;
    return cudaGetLastError();
}

// Pairs of CTAs of the scan: as many as can run at once, more when a pair would otherwise get more than
// kMaxRunTiles tiles
static int project_pairs(long long n_tiles, int max_pairs) {
    const long long by_run = (n_tiles + kMaxRunTiles - 1) / kMaxRunTiles;
    const long long g = n_tiles < max_pairs ? n_tiles : max_pairs;
    return (int)(g > by_run ? g : by_run);
}

int project_pieces(int R, int V, int sm_count) {
    const int tiles_m = (R + kPairM - 1) / kPairM, tiles_n = (V + kBN - 1) / kBN;
    const int pairs = project_pairs((long long)tiles_m * tiles_n, sm_count / 2 > 0 ? sm_count / 2 : 1);
    return ((pairs + tiles_m - 1) / tiles_m + 2) * kEpiGroups;
}

int project_list_cap() { return kListCap; }

bool project_scan_usable(const void* hidden, int64_t hidden_stride, const void* embed, int64_t embed_stride, int D, int K1) {
    if (((uintptr_t)hidden & 15u) || ((uintptr_t)embed & 15u) || ((hidden_stride * 2) & 15) || ((embed_stride * 2) & 15)) return false;
    return D >= 8 && D % 8 == 0 && K1 <= 32;
}

static void pair_launch_config(cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr, int pairs, cudaStream_t st) {
    *cfg = cudaLaunchConfig_t{};
    cfg->gridDim = dim3(2 * pairs, 1, 1); cfg->blockDim = dim3(kProjThreads, 1, 1);
    cfg->dynamicSmemBytes = sizeof(ProjSmem) + 1024; cfg->stream = st;
    attr->id = cudaLaunchAttributeClusterDimension;
    attr->val.clusterDim.x = 2; attr->val.clusterDim.y = 1; attr->val.clusterDim.z = 1;
    cfg->attrs = attr; cfg->numAttrs = 1;
}

// *max_pairs: how many pairs of CTAs the device runs at once (a pair needs two SMs of one GPC)
cudaError_t configure_project_scan(int* max_pairs) {
    cudaError_t e = cudaFuncSetAttribute(project_scan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(ProjSmem) + 1024);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg; cudaLaunchAttribute attr;
    pair_launch_config(&cfg, &attr, 1, nullptr);
    int n = 0;
    e = cudaOccupancyMaxActiveClusters(&n, project_scan_kernel, &cfg);
    if (e != cudaSuccess) return e;
    if (n < 1) return cudaErrorInvalidConfiguration;
    *max_pairs = n;
    return cudaSuccess;
}

cudaError_t launch_project_scan(const void* hidden, int64_t hidden_stride, const void* embed, int64_t embed_stride,
                                int R, int V, int D, int K1, const ProjPieces& pieces, int piece_stride,
                                const RowTop& top, uint32_t* status, int max_pairs, const ScanDebug& dbg, cudaStream_t st,
                                int* launches) {
    CUtensorMap map_a, map_b;
    if (!make_map(&map_a, hidden, R, D, hidden_stride, kBM) || !make_map(&map_b, embed, V, D, embed_stride, kHalfN))
        return cudaErrorInvalidValue;
    ProjParams p;
    p.R = R; p.V = V; p.D = D; p.K1 = K1;
    p.tiles_m = (R + kPairM - 1) / kPairM; p.tiles_n = (V + kBN - 1) / kBN;
    p.pieces = piece_stride; p.out = pieces; p.row_tau = pieces.row_tau; p.status = status;
    p.wait_clocks = dbg.wait_clocks > 0 ? dbg.wait_clocks : kProjWaitClocks; p.drop_item = dbg.drop_item;
    cudaError_t e0 = cudaMemsetAsync(pieces.row_tau, 0, sizeof(uint32_t) * (size_t)R, st);
    if (e0 != cudaSuccess) return e0;
    const long long n_tiles = (long long)p.tiles_m * p.tiles_n;
    const int pairs = project_pairs(n_tiles, max_pairs);
    cudaLaunchConfig_t cfg; cudaLaunchAttribute attr;
    pair_launch_config(&cfg, &attr, pairs, st);
    cudaError_t e = cudaLaunchKernelEx(&cfg, project_scan_kernel, map_a, map_b, p);
    ++*launches;
    if (e != cudaSuccess) return e;
    project_merge_kernel<<<(R + kMergeWarps - 1) / kMergeWarps, kMergeWarps * 32, 0, st>>>(p, pairs, top);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace dba
