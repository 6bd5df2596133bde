// Row scan: per row the log-sum-exp and the K1 largest entries.
// This file holds the generic kernel (any alignment, plain loads), the choice between it and the streaming one,
// segment planning, and the stand-alone merge of the streaming kernel's per-segment results.
#include "dba_device.cuh"
#include "dba_internal.h"

namespace dba {

namespace {

constexpr int kScanThreads = 512;

// Deterministic block reductions over kScanThreads threads (fixed tree, result broadcast to all).
__device__ float block_max(float v, float* sm) {
    v = warp_max(v);
    if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = sm[0];
    for (int i = 1; i < kScanThreads / 32; ++i) r = fmaxf(r, sm[i]);
    __syncthreads();
    return r;
}
__device__ float block_sum(float v, float* sm) {
    v = warp_sum(v);
    if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = sm[0];
    for (int i = 1; i < kScanThreads / 32; ++i) r += sm[i];
    __syncthreads();
    return r;
}
__device__ uint64_t block_max_u64(uint64_t v, uint64_t* sm) {
    v = warp_max_u64(v);
    if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = v;
    __syncthreads();
    uint64_t r = sm[0];
    for (int i = 1; i < kScanThreads / 32; ++i) r = sm[i] > r ? sm[i] : r;
    __syncthreads();
    return r;
}

// Generic scan: one CTA per row; K1 + 2 passes over the row (it stays in L2 between them).
template <typename T>
__global__ void __launch_bounds__(kScanThreads)
row_scan_generic_kernel(const T* __restrict__ logits, int64_t stride, int V, int K1, int eos,
                        const float* __restrict__ open_score, const int32_t* __restrict__ open_token,
                        int32_t* __restrict__ zero_count, float* __restrict__ row_lse,
                        float* __restrict__ top_val, int32_t* __restrict__ top_idx) {
    __shared__ float smf[kScanThreads / 32];
    __shared__ uint64_t smu[kScanThreads / 32];
    const int r = blockIdx.x;
    if (zero_count && r == 0 && threadIdx.x == 0) *zero_count = 0;
    if (open_score) {
        if (open_score[r] == neg_inf() || open_token[r] == eos) return;   // empty or finished slot
    }
    const T* row = logits + (int64_t)r * stride;

    float m = neg_inf();
    for (int w = threadIdx.x; w < V; w += kScanThreads) m = fmaxf(m, load_logit<T>(row + w));
    m = block_max(m, smf);
    float s = 0.f;
    if (m != neg_inf())
        for (int w = threadIdx.x; w < V; w += kScanThreads) s += expf(load_logit<T>(row + w) - m);
    s = block_sum(s, smf);
    if (threadIdx.x == 0) row_lse[r] = m == neg_inf() ? neg_inf() : m + logf(s);

    uint64_t prev = ~0ull;
    for (int i = 0; i < K1; ++i) {
        uint64_t best = 0;
        for (int w = threadIdx.x; w < V; w += kScanThreads) {
            uint64_t key = row_key(load_logit<T>(row + w), w);
            if (key < prev && key > best) best = key;
        }
        best = block_max_u64(best, smu);
        if (threadIdx.x == 0) {
            top_val[(int64_t)r * K1 + i] = best ? row_key_val(best) : neg_inf();
            top_idx[(int64_t)r * K1 + i] = best ? row_key_idx(best) : -1;
        }
        prev = best ? best : 0;   // once exhausted, nothing is below key 0
    }
}

// Stand-alone merge of the S segment results of each row: log-sum-exp and the n_top best entries.
// One warp per row.
__global__ void row_merge_kernel(int R, int S, int K1, int n_top, const float* __restrict__ part_m,
                                 const float* __restrict__ part_s, const float* __restrict__ pv,
                                 const int32_t* __restrict__ pi, float* __restrict__ row_lse,
                                 float* __restrict__ top_val, int32_t* __restrict__ top_idx) {
    const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (r >= R) return;
    if (lane == 0) {
        float M = neg_inf();
        for (int g = 0; g < S; ++g) M = fmaxf(M, part_m[r * S + g]);
        float sum = 0.f;
        if (M != neg_inf())
            for (int g = 0; g < S; ++g)
                if (part_m[r * S + g] != neg_inf()) sum += part_s[r * S + g] * expf(part_m[r * S + g] - M);
        row_lse[r] = M == neg_inf() ? neg_inf() : M + logf(sum);
    }
    const int n = S * K1;
    const float* v = pv + (int64_t)r * n;
    const int32_t* ix = pi + (int64_t)r * n;
    for (int e = lane; e < n_top; e += 32) { top_val[(int64_t)r * n_top + e] = neg_inf(); top_idx[(int64_t)r * n_top + e] = -1; }
    __syncwarp();
    for (int e = lane; e < n; e += 32) {
        if (ix[e] < 0) continue;
        uint64_t key = row_key(v[e], ix[e]);
        int rank = 0;
        for (int j = 0; j < n; ++j)
            if (ix[j] >= 0 && row_key(v[j], ix[j]) > key) ++rank;
        if (rank < n_top) { top_val[(int64_t)r * n_top + rank] = v[e]; top_idx[(int64_t)r * n_top + rank] = ix[e]; }
    }
}

// The stand-alone scan has no handle whose later calls could report a failed wait: if the scan recorded one,
// every row's result is replaced by one that cannot be taken for a real one (normaliser NaN, list (-inf, -1)).
__global__ void scan_check_kernel(const uint32_t* __restrict__ status, int R, int n_top, RowTop top) {
    if (!(*status & (kStatusTimeout | kStatusOverflow))) return;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < (int64_t)R * n_top; i += (int64_t)gridDim.x * blockDim.x) {
        top.val[i] = neg_inf(); top.idx[i] = -1;
        if (i < R) top.lse[i] = __int_as_float(0x7fc00000);
    }
}

}  // namespace

cudaError_t launch_scan_check(const uint32_t* status, int R, int n_top, const RowTop& top, cudaStream_t st) {
    scan_check_kernel<<<64, 256, 0, st>>>(status, R, n_top, top);
    return cudaGetLastError();
}

void plan_segments(Dims& d, int sm_count) {
    // Segments are whole 4 KB chunks, at most eleven of them (what one team of the streaming kernel holds);
    // shorter segments when there are few rows, so that every SM has several (row, segment) items to work on,
    // but never more than kMaxSeg segments per row.
    const int es = d.dtype == DBA_F32 ? 4 : 2;
    const int chunk_elems = 4096 / es;
    const int row_chunks = (d.V + chunk_elems - 1) / chunk_elems;
    auto segs = [&](int c) { return (row_chunks + c - 1) / c; };
    int chunks;
    if (segs(11) > kMaxSeg) {                                         // long rows: full-length segments, more of them;
        chunks = 11;                                                  // beyond kMaxSegLong: longer ones (generic kernel)
        while (segs(chunks) > kMaxSegLong) chunks *= 2;
    } else {
        chunks = (row_chunks + segs(11) - 1) / segs(11);             // as few segments as possible, evened out
        while (chunks > 1 && (int64_t)d.R * segs(chunks) < 4LL * sm_count && segs((chunks + 1) / 2) <= kMaxSeg)
            chunks = (chunks + 1) / 2;
    }
    d.seg_len = chunks * chunk_elems;
    d.S = segs(chunks);
    d.K1 = d.k + 2;
}

int max_segments(int V, int dtype) {
    const int chunk_elems = 4096 / (dtype == DBA_F32 ? 4 : 2);
    const int row_chunks = (V + chunk_elems - 1) / chunk_elems;
    const int full = (row_chunks + 10) / 11;
    return full <= kMaxSeg ? kMaxSeg : (full <= kMaxSegLong ? full : kMaxSegLong);
}

cudaError_t launch_row_scan(const void* logits, int64_t stride, const Dims& d, const float* open_score,
                            const int32_t* open_token, const int32_t* open_list, const int32_t* open_count,
                            int32_t* zero_count, const RowTop& out, const ScanScratch& part, uint32_t* status,
                            int sm_count, const ScanDebug& dbg, cudaStream_t st, int* launches, bool* partial) {
    ++*launches;
    *partial = row_scan_tma_usable(logits, stride, d);
    if (*partial)
        return launch_row_scan_tma(logits, stride, d, open_list, open_count, zero_count, part, status, sm_count, dbg, st);
    if (d.dtype == DBA_F32)
        row_scan_generic_kernel<float><<<d.R, kScanThreads, 0, st>>>(
            (const float*)logits, stride, d.V, d.K1, d.eos_id, open_score, open_token, zero_count, out.lse, out.val,
            out.idx);
    else
        row_scan_generic_kernel<__nv_bfloat16><<<d.R, kScanThreads, 0, st>>>(
            (const __nv_bfloat16*)logits, stride, d.V, d.K1, d.eos_id, open_score, open_token, zero_count, out.lse,
            out.val, out.idx);
    return cudaGetLastError();
}

cudaError_t launch_row_merge(const Dims& d, const ScanScratch& part, int n_top, float* row_lse, float* top_val,
                             int32_t* top_idx, cudaStream_t st, int* launches) {
    const int warps = 4;
    row_merge_kernel<<<(d.R + warps - 1) / warps, warps * 32, 0, st>>>(d.R, d.S, d.K1, n_top, part.m, part.s,
                                                                      part.val, part.idx, row_lse,
                                                                      top_val, top_idx);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace dba
