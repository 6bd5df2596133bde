// Host side of the C ABI declared in include/dba.h: argument checks, workspace carving, launch sequence.
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "dba_internal.h"

using namespace dba;

struct dba_handle {
    Dims d;
    int32_t max_steps;
    cudaStream_t stream;
    int device;
    int sm_count;
    int proj_pairs;                // only with DBA_FLAG_FUSED_PROJECTION: pairs of CTAs the device runs at once
    // carved from the caller's workspace
    SentCons* cons;
    Beam beam[2];
    int32_t* hist_bp;
    int32_t* hist_tok;
    RowTop top;                    // the row scan's results (top.lse doubles as the step's row_lse output)
    ScanScratch part;
    ProjPieces proj;               // only with DBA_FLAG_FUSED_PROJECTION: scratch of the fused projection
    int proj_stride;
    float* s2_logit;               // and the logits of the constraint tokens, [R, 64]
    CandLaunch cand;               // block size and shared memory of the candidate kernel on this handle's device
    ScanDebug dbg;
    uint32_t* status;
    int32_t* open_list;            // rows the next step scans, and how many
    int32_t* open_count;           // two counts: step t reads [t & 1], its last kernel fills [(t + 1) & 1]
                                   // ([2], [3]: the row scan's work counters, alternating the same way)
    int32_t* fin_tokens; int32_t* fin_len; float* fin_score; int32_t* fin_flags;
    void* stage_logits;            // only with DBA_FLAG_HOST_STAGING
    dba_step_out stage_out;
    // progress
    int32_t t;
    int cur;
    int launches_tmp;
    uint64_t launches;
    // optional kernel timing
    bool timing;
    std::vector<cudaEvent_t> ev;   // 3 events per recorded step
    int ev_steps;
};

constexpr int kTimingCap = 4096;

// testing aids of the stand-alone row scan (dba_test_hook with a null handle)
static ScanDebug g_scan_debug;

namespace {

struct Carver {   // hands out 256-byte aligned pieces of the workspace; with base == nullptr it only measures
    char* base;
    size_t off = 0;
    explicit Carver(void* b) : base((char*)b) {}
    template <typename T>
    T* take(size_t n) {
        off = (off + 255) / 256 * 256;
        T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
        off += n * sizeof(T);
        return p;
    }
};

struct Shape {
    int32_t max_phrases = 1;   // most phrases in one sentence
};

dba_status check_config(const dba_config* c, Shape* shape, std::vector<SentCons>* cons_out) {
    if (!c) return DBA_ERR_INVALID_ARG;
    if (c->B < 1 || c->k < 1 || c->V < 1 || c->max_steps < 1) return DBA_ERR_INVALID_ARG;
    if (c->logit_dtype != DBA_F32 && c->logit_dtype != DBA_BF16) return DBA_ERR_INVALID_ARG;
    if (c->prune_threshold != c->prune_threshold) return DBA_ERR_INVALID_ARG;      // NaN
    if (c->flags & ~(DBA_FLAG_ADJUST_OFF | DBA_FLAG_LENGTH_NORM | DBA_FLAG_HOST_STAGING | DBA_FLAG_PRUNE_NORMALISED |
                     DBA_FLAG_FUSED_PROJECTION))
        return DBA_ERR_INVALID_ARG;
    const int32_t sp[3] = {c->pad_id, c->bos_id, c->eos_id};
    for (int i = 0; i < 3; ++i)
        if (sp[i] < 0 || sp[i] >= c->V) return DBA_ERR_INVALID_ARG;
    if (c->eos_id == c->pad_id || c->eos_id == c->bos_id) return DBA_ERR_INVALID_ARG;
    if (c->k > kMaxK) return DBA_ERR_UNSUPPORTED;
    if ((int64_t)c->k * c->V >= (int64_t)1 << 31) return DBA_ERR_UNSUPPORTED;
    if ((int64_t)c->B * c->k >= (int64_t)1 << 27) return DBA_ERR_UNSUPPORTED;
    if (!c->sent_phrase_off) return DBA_ERR_INVALID_ARG;
    const int32_t P0 = c->sent_phrase_off[0], P1 = c->sent_phrase_off[c->B];
    if (P0 < 0 || P1 < P0) return DBA_ERR_INVALID_ARG;
    if (P1 > P0 && (!c->phrase_tok_off || !c->tok)) return DBA_ERR_INVALID_ARG;
    if (cons_out) cons_out->assign(c->B, SentCons{});
    for (int b = 0; b < c->B; ++b) {
        const int32_t pa = c->sent_phrase_off[b], pb = c->sent_phrase_off[b + 1];
        if (pb < pa || pa < P0 || pb > P1) return DBA_ERR_INVALID_ARG;
        SentCons sc{};
        int j = 0;
        for (int32_t p = pa; p < pb; ++p) {
            const int32_t ta = c->phrase_tok_off[p], tb = c->phrase_tok_off[p + 1];
            if (ta < 0 || tb <= ta) return DBA_ERR_INVALID_ARG;             // phrases are non-empty
            if (j + (tb - ta) > kMaxC) return DBA_ERR_UNSUPPORTED;
            const int start = j;
            for (int32_t i = ta; i < tb; ++i, ++j) {
                const int32_t w = c->tok[i];
                if (w < 0 || w >= c->V || w == c->pad_id || w == c->bos_id || w == c->eos_id) return DBA_ERR_INVALID_ARG;
                sc.ctok[j] = w;
                sc.pstart[j] = (uint8_t)start;
                if (i == ta) sc.first_mask |= 1ull << j;
                if (i == tb - 1) sc.last_mask |= 1ull << j;
            }
        }
        for (int q = 0; q < j; ++q) {
            sc.prev_same[q] = 255;
            if (!((sc.first_mask >> q) & 1ull)) continue;
            for (int e = q - 1; e >= 0; --e)
                if (((sc.first_mask >> e) & 1ull) && sc.ctok[e] == sc.ctok[q]) { sc.prev_same[q] = (uint8_t)e; break; }
        }
        sc.C = j;
        sc.n_phrases = pb - pa;
        if (shape && sc.n_phrases > shape->max_phrases) shape->max_phrases = sc.n_phrases;
        if (cons_out) (*cons_out)[b] = sc;
    }
    return DBA_OK;
}

void fill_dims(const dba_config* c, const Shape& sh, Dims* d) {
    d->B = c->B; d->k = c->k; d->V = c->V; d->R = c->B * c->k;
    d->pad_id = c->pad_id; d->bos_id = c->bos_id; d->eos_id = c->eos_id;
    d->dtype = c->logit_dtype; d->flags = c->flags;
    d->prune = c->prune_threshold > 0.f ? c->prune_threshold : 0.f;
    d->max_cand = c->k * (sh.max_phrases + 2);
    d->K1 = c->k + 2; d->S = max_segments(c->V, c->logit_dtype); d->seg_len = 0;   // an upper bound until plan_segments runs
}

Beam carve_beam(Carver& cv, int R) {
    Beam b;
    b.score = cv.take<float>(R); b.token = cv.take<int32_t>(R); b.mask = cv.take<uint64_t>(R);
    b.active = cv.take<int32_t>(R); b.len = cv.take<int32_t>(R); b.bank = cv.take<int32_t>(R);
    b.backptr = cv.take<int32_t>(R);
    return b;
}

RowTop carve_top(Carver& cv, size_t R, int K1) {
    RowTop t;
    t.lse = cv.take<float>(R); t.val = cv.take<float>(R * K1); t.idx = cv.take<int32_t>(R * K1);
    return t;
}

ScanScratch carve_scratch(Carver& cv, size_t R, int S, int K1) {
    ScanScratch s;
    s.m = cv.take<float>(R * S); s.s = cv.take<float>(R * S);
    s.val = cv.take<float>(R * S * K1); s.idx = cv.take<int32_t>(R * S * K1);
    return s;
}

ProjPieces carve_pieces(Carver& cv, size_t R, int P) {
    ProjPieces q;
    const size_t cap = (size_t)project_list_cap();
    q.ref = cv.take<int32_t>(R * P); q.sum = cv.take<float>(R * P); q.n = cv.take<int32_t>(R * P);
    q.val = cv.take<float>(R * P * cap); q.col = cv.take<int32_t>(R * P * cap);
    q.row_tau = cv.take<uint32_t>(R);
    return q;
}

// Lays the handle's arrays out in the workspace.
size_t carve(dba_handle* h, void* base, int32_t max_steps) {
    Carver cv(base);
    const Dims& d = h->d;
    const size_t R = d.R;
    h->cons = cv.take<SentCons>(d.B);
    h->beam[0] = carve_beam(cv, d.R);
    h->beam[1] = carve_beam(cv, d.R);
    h->hist_bp = cv.take<int32_t>(R * max_steps);
    h->hist_tok = cv.take<int32_t>(R * max_steps);
    h->top = carve_top(cv, R, d.K1);
    h->part = carve_scratch(cv, R, max_segments(d.V, d.dtype), d.K1);
    h->status = cv.take<uint32_t>(64);
    h->open_list = cv.take<int32_t>(R);
    h->open_count = cv.take<int32_t>(64);
    h->fin_tokens = cv.take<int32_t>((size_t)d.B * max_steps);
    h->fin_len = cv.take<int32_t>(d.B);
    h->fin_score = cv.take<float>(d.B);
    h->fin_flags = cv.take<int32_t>(d.B);
    h->s2_logit = nullptr; h->proj_stride = 0;
    std::memset(&h->proj, 0, sizeof h->proj);
    if (d.flags & DBA_FLAG_FUSED_PROJECTION) {
        h->proj_stride = project_pieces(d.R, d.V, h->sm_count);
        h->proj = carve_pieces(cv, R, h->proj_stride);
        h->s2_logit = cv.take<float>(R * kMaxC);
    }
    h->stage_logits = nullptr;
    std::memset(&h->stage_out, 0, sizeof h->stage_out);
    if (d.flags & DBA_FLAG_HOST_STAGING) {
        h->stage_logits = cv.take<char>(R * (size_t)d.V * (d.dtype == DBA_F32 ? 4 : 2));
        h->stage_out.backptr = cv.take<int32_t>(R); h->stage_out.token = cv.take<int32_t>(R);
        h->stage_out.score = cv.take<float>(R); h->stage_out.bank = cv.take<int32_t>(R);
        h->stage_out.met_mask = cv.take<uint64_t>(R); h->stage_out.active = cv.take<int32_t>(R);
        h->stage_out.row_lse = cv.take<float>(R);
        h->stage_out.stop = cv.take<int32_t>(d.B);
    }
    return (cv.off + 255) / 256 * 256;
}

inline dba_status cuda_fail(cudaError_t e) { return e == cudaSuccess ? DBA_OK : DBA_ERR_CUDA; }

// The three events of a recorded step (null when timing is off or the record is full).  False: event creation failed.
bool step_events(dba_handle* h, cudaEvent_t** ev) {
    *ev = nullptr;
    if (!h->timing || h->ev_steps >= kTimingCap) return true;
    if ((int)h->ev.size() < 3 * (h->ev_steps + 1)) {
        for (int i = 0; i < 3; ++i) {
            cudaEvent_t x;
            if (cudaEventCreate(&x) != cudaSuccess) return false;
            h->ev.push_back(x);
        }
    }
    *ev = &h->ev[3 * h->ev_steps];
    h->ev_steps += 1;
    return true;
}

}  // namespace

extern "C" {

dba_status dba_workspace_bytes(const dba_config* cfg, size_t* bytes) {
    if (!bytes) return DBA_ERR_INVALID_ARG;
    Shape sh;
    dba_status st = check_config(cfg, &sh, nullptr);
    if (st != DBA_OK) return st;
    dba_handle tmp{};
    fill_dims(cfg, sh, &tmp.d);
    int dev = 0;
    tmp.sm_count = 1;
    if (cfg->flags & DBA_FLAG_FUSED_PROJECTION)      // the projection's scratch depends on the current device's SM count
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&tmp.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            return DBA_ERR_CUDA;
    *bytes = carve(&tmp, nullptr, cfg->max_steps);
    return DBA_OK;
}

dba_status dba_init(const dba_config* cfg, void* workspace_dev, size_t workspace_bytes, void* cuda_stream,
                    dba_handle** out) {
    if (!out) return DBA_ERR_INVALID_ARG;
    *out = nullptr;
    Shape sh;
    std::vector<SentCons> cons;
    dba_status st = check_config(cfg, &sh, &cons);
    if (st != DBA_OK) return st;
    if (!workspace_dev || ((uintptr_t)workspace_dev & 255u)) return DBA_ERR_WORKSPACE;
    dba_handle* h = new (std::nothrow) dba_handle{};
    if (!h) return DBA_ERR_INVALID_ARG;
    fill_dims(cfg, sh, &h->d);
    h->max_steps = cfg->max_steps;
    cudaError_t e = cudaGetDevice(&h->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device);
    if (e != cudaSuccess) { delete h; return DBA_ERR_CUDA; }
    if ((cfg->flags & DBA_FLAG_FUSED_PROJECTION) && h->d.K1 > 32) { delete h; return DBA_ERR_UNSUPPORTED; }
    const size_t need = carve(h, workspace_dev, cfg->max_steps);
    if (workspace_bytes < need) { delete h; return DBA_ERR_WORKSPACE; }
    h->stream = (cudaStream_t)cuda_stream;
    plan_segments(h->d, h->sm_count);
    bool fits = false;
    e = configure_candidates(h->d, &h->cand, &fits);
    if (e == cudaSuccess && !fits) { delete h; return DBA_ERR_UNSUPPORTED; }
    if (e == cudaSuccess) e = configure_row_scan_tma();
    if (e == cudaSuccess && (cfg->flags & DBA_FLAG_FUSED_PROJECTION)) e = configure_project_scan(&h->proj_pairs);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(h->cons, cons.data(), sizeof(SentCons) * cons.size(), cudaMemcpyHostToDevice, h->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->status, 0, 256, h->stream);
    h->launches_tmp = 0;
    if (e == cudaSuccess)
        e = launch_reset(h->d, h->beam[0], h->open_list, h->open_count, h->top, h->stream, &h->launches_tmp);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);   // `cons` is a local buffer
    if (e != cudaSuccess) { delete h; return DBA_ERR_CUDA; }
    h->launches = h->launches_tmp;
    h->t = 0; h->cur = 0;
    *out = h;
    return DBA_OK;
}

dba_status dba_reset(dba_handle* h) {
    if (!h) return DBA_ERR_INVALID_ARG;
    h->launches_tmp = 0;
    cudaError_t e = launch_reset(h->d, h->beam[0], h->open_list, h->open_count, h->top, h->stream,
                                 &h->launches_tmp);
    h->launches += h->launches_tmp;
    h->t = 0; h->cur = 0;
    return cuda_fail(e);
}

dba_status dba_step(dba_handle* h, const void* logits_dev, int64_t row_stride_elems,
                    const float* row_lse_in_dev, const dba_step_out* out_dev) {
    if (!h || !logits_dev || row_stride_elems < h->d.V) return DBA_ERR_INVALID_ARG;
    if (h->t >= h->max_steps) return DBA_ERR_STATE;
    dba_step_out out{};
    if (out_dev) out = *out_dev;
    const Beam& cur = h->beam[h->cur];
    const Beam& nxt = h->beam[h->cur ^ 1];
    h->launches_tmp = 0;
    cudaEvent_t* ev = nullptr;
    if (!step_events(h, &ev)) return DBA_ERR_CUDA;
    cudaError_t e = cudaSuccess;
    bool partial = false;
    if (ev) e = cudaEventRecord(ev[0], h->stream);
    if (e == cudaSuccess)
        e = launch_row_scan(logits_dev, row_stride_elems, h->d, cur.score, cur.token, h->open_list,
                            h->open_count + (h->t & 1), h->open_count + ((h->t + 1) & 1), h->top, h->part, h->status,
                            h->sm_count, h->dbg, h->stream, &h->launches_tmp, &partial);
    if (ev && e == cudaSuccess) e = cudaEventRecord(ev[1], h->stream);
    ScanScratch part = h->part;
    if (!partial) part.m = nullptr;           // the plain kernel wrote the rows' finished results
    if (e == cudaSuccess)
        e = launch_candidates(logits_dev, row_stride_elems, h->d, h->cons, cur, nxt, h->top, part, row_lse_in_dev, nullptr, out,
                              h->hist_bp + (size_t)h->t * h->d.R, h->hist_tok + (size_t)h->t * h->d.R, h->status,
                              h->open_list, h->open_count + ((h->t + 1) & 1), h->cand, h->stream, &h->launches_tmp);
    if (ev && e == cudaSuccess) e = cudaEventRecord(ev[2], h->stream);
    h->launches += h->launches_tmp;
    if (e != cudaSuccess) return DBA_ERR_CUDA;
    h->cur ^= 1;
    h->t += 1;
    return DBA_OK;
}

dba_status dba_step_fused(dba_handle* h, const void* hidden_dev, int64_t hidden_stride_elems, const void* embed_dev,
                          int64_t embed_stride_elems, int32_t D, const dba_step_out* out_dev) {
    if (!h || !hidden_dev || !embed_dev || D < 1 || hidden_stride_elems < D || embed_stride_elems < D) return DBA_ERR_INVALID_ARG;
    if (!h->s2_logit) return DBA_ERR_STATE;
    if (h->t >= h->max_steps) return DBA_ERR_STATE;
    if (!project_scan_usable(hidden_dev, hidden_stride_elems, embed_dev, embed_stride_elems, D, h->d.K1)) return DBA_ERR_UNSUPPORTED;
    dba_step_out out{};
    if (out_dev) out = *out_dev;
    const Beam& cur = h->beam[h->cur];
    const Beam& nxt = h->beam[h->cur ^ 1];
    h->launches_tmp = 0;
    cudaEvent_t* ev = nullptr;
    if (!step_events(h, &ev)) return DBA_ERR_CUDA;
    // the list of open rows is not used by this path (every row is projected), but its count is kept in step
    cudaError_t e = cudaMemsetAsync(h->open_count + ((h->t + 1) & 1), 0, sizeof(int32_t), h->stream);
    // (nor does it run the row scan, whose launches clear each other's work counter in turn: both are cleared here)
    if (e == cudaSuccess) e = cudaMemsetAsync(h->open_count + 2, 0, 2 * sizeof(int32_t), h->stream);
    if (ev && e == cudaSuccess) e = cudaEventRecord(ev[0], h->stream);
    if (e == cudaSuccess)
        e = launch_project_scan(hidden_dev, hidden_stride_elems, embed_dev, embed_stride_elems, h->d.R, h->d.V, D, h->d.K1,
                                h->proj, h->proj_stride, h->top, h->status, h->proj_pairs, h->dbg, h->stream, &h->launches_tmp);
    if (ev && e == cudaSuccess) e = cudaEventRecord(ev[1], h->stream);
    if (e == cudaSuccess)
        e = launch_constraint_logits(hidden_dev, hidden_stride_elems, embed_dev, embed_stride_elems, D, h->d, h->cons,
                                     h->s2_logit, h->stream, &h->launches_tmp);
    if (e == cudaSuccess)
        e = launch_candidates(nullptr, 0, h->d, h->cons, cur, nxt, h->top, ScanScratch{}, nullptr, h->s2_logit, out,
                              h->hist_bp + (size_t)h->t * h->d.R, h->hist_tok + (size_t)h->t * h->d.R, h->status,
                              h->open_list, h->open_count + ((h->t + 1) & 1), h->cand, h->stream, &h->launches_tmp);
    if (ev && e == cudaSuccess) e = cudaEventRecord(ev[2], h->stream);
    h->launches += h->launches_tmp;
    if (e != cudaSuccess) return DBA_ERR_CUDA;
    h->cur ^= 1;
    h->t += 1;
    return DBA_OK;
}

dba_status dba_step_host(dba_handle* h, const void* logits_host, int64_t row_stride_elems,
                         const dba_step_out* out_host) {
    if (!h || !logits_host || row_stride_elems < h->d.V) return DBA_ERR_INVALID_ARG;
    if (!h->stage_logits) return DBA_ERR_STATE;
    if (h->t >= h->max_steps) return DBA_ERR_STATE;
    const size_t es = h->d.dtype == DBA_F32 ? 4 : 2;
    const size_t R = h->d.R;
    cudaError_t e;
    if (row_stride_elems == h->d.V)
        e = cudaMemcpyAsync(h->stage_logits, logits_host, R * h->d.V * es, cudaMemcpyHostToDevice, h->stream);
    else
        e = cudaMemcpy2DAsync(h->stage_logits, h->d.V * es, logits_host, row_stride_elems * es, h->d.V * es, R,
                              cudaMemcpyHostToDevice, h->stream);
    if (e != cudaSuccess) return DBA_ERR_CUDA;
    dba_status st = dba_step(h, h->stage_logits, h->d.V, nullptr, &h->stage_out);
    if (st != DBA_OK) return st;
    if (out_host) {
        const dba_step_out& s = h->stage_out;
        const cudaMemcpyKind k = cudaMemcpyDeviceToHost;
        if (out_host->backptr && e == cudaSuccess) e = cudaMemcpyAsync(out_host->backptr, s.backptr, R * 4, k, h->stream);
        if (out_host->token && e == cudaSuccess) e = cudaMemcpyAsync(out_host->token, s.token, R * 4, k, h->stream);
        if (out_host->score && e == cudaSuccess) e = cudaMemcpyAsync(out_host->score, s.score, R * 4, k, h->stream);
        if (out_host->bank && e == cudaSuccess) e = cudaMemcpyAsync(out_host->bank, s.bank, R * 4, k, h->stream);
        if (out_host->met_mask && e == cudaSuccess) e = cudaMemcpyAsync(out_host->met_mask, s.met_mask, R * 8, k, h->stream);
        if (out_host->active && e == cudaSuccess) e = cudaMemcpyAsync(out_host->active, s.active, R * 4, k, h->stream);
        if (out_host->row_lse && e == cudaSuccess) e = cudaMemcpyAsync(out_host->row_lse, s.row_lse, R * 4, k, h->stream);
        if (out_host->stop && e == cudaSuccess) e = cudaMemcpyAsync(out_host->stop, s.stop, (size_t)h->d.B * 4, k, h->stream);
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
    return cuda_fail(e);
}

dba_status dba_finalize(dba_handle* h, int32_t* tokens_host, int32_t* len_host, float* score_host,
                        int32_t* flags_host) {
    if (!h) return DBA_ERR_INVALID_ARG;
    h->launches_tmp = 0;
    cudaError_t e = launch_finalize(h->d, h->beam[h->cur], h->hist_bp, h->hist_tok, h->t, h->max_steps,
                                    h->fin_tokens, h->fin_len, h->fin_score, h->fin_flags, h->stream,
                                    &h->launches_tmp);
    h->launches += h->launches_tmp;
    const cudaMemcpyKind k = cudaMemcpyDeviceToHost;
    const size_t B = h->d.B;
    uint32_t status = 0;
    if (tokens_host && e == cudaSuccess)
        e = cudaMemcpyAsync(tokens_host, h->fin_tokens, B * h->max_steps * 4, k, h->stream);
    if (len_host && e == cudaSuccess) e = cudaMemcpyAsync(len_host, h->fin_len, B * 4, k, h->stream);
    if (score_host && e == cudaSuccess) e = cudaMemcpyAsync(score_host, h->fin_score, B * 4, k, h->stream);
    if (flags_host && e == cudaSuccess) e = cudaMemcpyAsync(flags_host, h->fin_flags, B * 4, k, h->stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(&status, h->status, 4, k, h->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
    if (e != cudaSuccess) return DBA_ERR_CUDA;
    if (status & kStatusTimeout) return DBA_ERR_TIMEOUT;
    if (status & kStatusOverflow) return DBA_ERR_CUDA;
    return DBA_OK;
}

dba_status dba_timing_enable(dba_handle* h, int32_t on) {
    if (!h) return DBA_ERR_INVALID_ARG;
    h->timing = on != 0;
    return DBA_OK;
}

dba_status dba_timing_read(dba_handle* h, double ms_total[3], int64_t* steps) {
    if (!h || !ms_total || !steps) return DBA_ERR_INVALID_ARG;
    if (cudaStreamSynchronize(h->stream) != cudaSuccess) return DBA_ERR_CUDA;
    ms_total[0] = ms_total[1] = ms_total[2] = 0.0;
    for (int i = 0; i < h->ev_steps; ++i)
        for (int j = 0; j < 2; ++j) {
            float ms = 0.f;
            if (cudaEventElapsedTime(&ms, h->ev[3 * i + j], h->ev[3 * i + j + 1]) != cudaSuccess) return DBA_ERR_CUDA;
            ms_total[j] += ms;
        }
    *steps = h->ev_steps;
    h->ev_steps = 0;
    return DBA_OK;
}

dba_status dba_counters(dba_handle* h, uint32_t counters[4]) {
    if (!h || !counters) return DBA_ERR_INVALID_ARG;
    uint32_t words[4] = {};
    cudaError_t e = cudaMemcpyAsync(words, h->status, sizeof words, cudaMemcpyDeviceToHost, h->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
    if (e != cudaSuccess) return DBA_ERR_CUDA;
    counters[0] = words[kStatusWordRescans]; counters[1] = words[kStatusWordUnresolved]; counters[2] = counters[3] = 0;
    return DBA_OK;
}

uint64_t dba_launch_count(const dba_handle* h) { return h ? h->launches : 0; }

dba_status dba_test_hook(dba_handle* h, int64_t wait_clocks, int32_t drop_item) {
    ScanDebug& dbg = h ? h->dbg : g_scan_debug;
    dbg.wait_clocks = wait_clocks > 0 ? (long long)wait_clocks : 0;
    dbg.drop_item = drop_item >= 0 ? drop_item : -1;
    return DBA_OK;
}

void dba_destroy(dba_handle* h) {
    if (!h) return;
    for (cudaEvent_t e : h->ev) cudaEventDestroy(e);
    delete h;
}

const char* dba_status_string(dba_status s) {
    switch (s) {
        case DBA_OK: return "ok";
        case DBA_ERR_INVALID_ARG: return "invalid argument";
        case DBA_ERR_UNSUPPORTED: return "over a supported limit";
        case DBA_ERR_STATE: return "call not allowed in this state";
        case DBA_ERR_CUDA: return "CUDA error";
        case DBA_ERR_TIMEOUT: return "device-side wait timed out";
        case DBA_ERR_WORKSPACE: return "workspace too small or misaligned";
    }
    return "unknown status";
}

dba_status dba_row_scan_scratch_bytes(int32_t R, int32_t V, int32_t n_top, int32_t logit_dtype, size_t* bytes) {
    if (!bytes || R < 1 || V < 1 || n_top < 1) return DBA_ERR_INVALID_ARG;
    if (logit_dtype != DBA_F32 && logit_dtype != DBA_BF16) return DBA_ERR_INVALID_ARG;
    if (n_top > kMaxTop) return DBA_ERR_UNSUPPORTED;
    Carver cv(nullptr);
    carve_scratch(cv, (size_t)R, max_segments(V, logit_dtype), n_top);
    cv.take<uint32_t>(64);
    *bytes = (cv.off + 255) / 256 * 256;
    return DBA_OK;
}

dba_status dba_row_scan(const void* logits_dev, int32_t logit_dtype, int32_t R, int32_t V, int64_t row_stride_elems,
                        int32_t n_top, void* scratch_dev, size_t scratch_bytes, float* row_lse_dev,
                        float* top_val_dev, int32_t* top_idx_dev, void* cuda_stream) {
    size_t need = 0;
    dba_status st = dba_row_scan_scratch_bytes(R, V, n_top, logit_dtype, &need);
    if (st != DBA_OK) return st;
    if (!logits_dev || !row_lse_dev || !top_val_dev || !top_idx_dev || row_stride_elems < V) return DBA_ERR_INVALID_ARG;
    if (!scratch_dev || ((uintptr_t)scratch_dev & 255u) || scratch_bytes < need) return DBA_ERR_WORKSPACE;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return DBA_ERR_CUDA;
    Dims d{};
    d.B = R; d.k = 1; d.V = V; d.R = R; d.dtype = logit_dtype; d.eos_id = -1; d.pad_id = 0; d.bos_id = 0;
    plan_segments(d, sms);
    d.K1 = n_top;
    Carver cv(scratch_dev);
    ScanScratch part = carve_scratch(cv, (size_t)R, max_segments(V, logit_dtype), n_top);
    uint32_t* status = cv.take<uint32_t>(64);
    RowTop top;
    top.lse = row_lse_dev; top.val = top_val_dev; top.idx = top_idx_dev;
    int launches = 0;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    // the scratch may hold anything (it may be shared with earlier calls): the status word starts at zero, everything
    // else is written before it is read
    bool partial = false;
    e = cudaMemsetAsync(status, 0, 256, stream);
    if (e == cudaSuccess) e = configure_row_scan_tma();
    if (e == cudaSuccess)
        e = launch_row_scan(logits_dev, row_stride_elems, d, nullptr, nullptr, nullptr, nullptr, nullptr, top, part, status,
                            sms, g_scan_debug, stream, &launches, &partial);
    if (e == cudaSuccess && partial) e = launch_row_merge(d, part, n_top, row_lse_dev, top_val_dev, top_idx_dev, stream, &launches);
    if (e == cudaSuccess) e = launch_scan_check(status, R, n_top, top, stream);
    return cuda_fail(e);
}

dba_status dba_project_scan_scratch_bytes(int32_t R, int32_t V, int32_t n_top, size_t* bytes) {
    if (!bytes || R < 1 || V < 1 || n_top < 1) return DBA_ERR_INVALID_ARG;
    if (n_top > 32) return DBA_ERR_UNSUPPORTED;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return DBA_ERR_CUDA;
    Carver cv(nullptr);
    carve_pieces(cv, (size_t)R, project_pieces(R, V, sms));
    cv.take<uint32_t>(64);
    *bytes = (cv.off + 255) / 256 * 256;
    return DBA_OK;
}

dba_status dba_project_scan(const void* hidden_dev, int64_t hidden_stride_elems, const void* embed_dev,
                            int64_t embed_stride_elems, int32_t R, int32_t V, int32_t D, int32_t n_top,
                            void* scratch_dev, size_t scratch_bytes, float* row_lse_dev, float* top_val_dev,
                            int32_t* top_idx_dev, void* cuda_stream) {
    size_t need = 0;
    dba_status st = dba_project_scan_scratch_bytes(R, V, n_top, &need);
    if (st != DBA_OK) return st;
    if (!hidden_dev || !embed_dev || !row_lse_dev || !top_val_dev || !top_idx_dev || D < 1 || hidden_stride_elems < D ||
        embed_stride_elems < D)
        return DBA_ERR_INVALID_ARG;
    if (!project_scan_usable(hidden_dev, hidden_stride_elems, embed_dev, embed_stride_elems, D, n_top)) return DBA_ERR_UNSUPPORTED;
    if (!scratch_dev || ((uintptr_t)scratch_dev & 255u) || scratch_bytes < need) return DBA_ERR_WORKSPACE;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return DBA_ERR_CUDA;
    Carver cv(scratch_dev);
    const int stride = project_pieces(R, V, sms);
    ProjPieces pieces = carve_pieces(cv, (size_t)R, stride);
    uint32_t* status = cv.take<uint32_t>(64);
    RowTop top;
    top.lse = row_lse_dev; top.val = top_val_dev; top.idx = top_idx_dev;
    int launches = 0;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    e = cudaMemsetAsync(status, 0, 256, stream);
    int max_pairs = 0;
    if (e == cudaSuccess) e = configure_project_scan(&max_pairs);
    if (e == cudaSuccess)
        e = launch_project_scan(hidden_dev, hidden_stride_elems, embed_dev, embed_stride_elems, R, V, D, n_top, pieces, stride,
                                top, status, max_pairs, g_scan_debug, stream, &launches);
    if (e == cudaSuccess) e = launch_scan_check(status, R, n_top, top, stream);
    return cuda_fail(e);
}

}  // extern "C"
