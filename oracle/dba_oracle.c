/*
 * dba_oracle.c -- plain, slow, single-threaded CPU statement of one sentence's
 * Dynamic Beam Allocation step (Post & Vilar 2018, Algorithm 2 with Sections
 * 3.1-3.3), the log-softmax in front of it (Section 2) and the final pick of
 * the best completed hypothesis (Section 3.3).
 *
 * THIS IS TEST INFRASTRUCTURE.  It exists so that the CUDA library can be checked
 * against something written straight from the paper.  It shares no code, header,
 * table or helper with the CUDA path, is never called by the library, and must
 * not be tuned: every function takes the steps in the paper's order on plain
 * arrays, in double precision where the paper leaves precision open.
 *
 * Where the paper is silent the reading taken is marked "READING" below.  Pin
 * status (what the CPU tests tie each function to, other than itself):
 *   orc_row_lse        pinned   closed forms (constant, two-value, geometric rows), shift invariance
 *   orc_row_top        pinned   equals a stable descending sort of the row
 *   orc_project        pinned   one-hot hidden state returns a row of the embedding; constant hidden state
 *                               returns scaled row sums; small integers give exact integer inner products
 *   step at C = 0      pinned   equals Algorithm 1's ARGMAX_K over the k x V matrix (full sort)
 *   candidate set      pinned   brute force by predicate over every (h, w) cell on small V, k
 *   orc_add            pinned   hand traces of Section 3.1's unwinding text; substring semantics on
 *                               non-overlapping phrases; exhaustive search regime;
 *                               parity unpinned: continuation before opening, first matching constraint
 *                               (conventions; tests/golden/add_masks.txt holds them as such)
 *   orc_allocate       pinned   Fig. 1 / Fig. 2 captions (k = 5, four constraints), sum = min(k, #cand),
 *                               alloc <= count, C >= k; nearest-bank-first and moving outward (Section 3.2's
 *                               adjustment sentence) by hand-derived allocations without ties;
 *                               parity unpinned: which of two equally near banks is served first and the
 *                               order in which overfilled banks act (the paper only outlines the procedure
 *                               and the figure that shows one is lost)
 *   finishing          pinned   every completed output holds all constraints; exhaustive regime
 *                               equals brute force over all sequences
 *   pruning, stopping  pinned   closed form on a two-word vocabulary (two scores exactly theta' apart: kept iff
 *                               theta' <= threshold), the best completed hypothesis is never removed, an
 *                               infinite threshold changes nothing, stop bits on hand-built beams;
 *                               the other reading (normalised completed scores, ORC_FLAG_PRUNE_NORM) by a
 *                               hand-built beam on which the two readings remove different hypotheses;
 *                               parity unpinned: which of the two readings the paper means
 *   conventions        parity unpinned: finished hypotheses staying on the beam with a frozen
 *                               score, empty slots, global order of the new beam, length counted
 *                               with the end token (READINGS below)
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_MAX_C 64

enum { ORC_F32 = 0, ORC_BF16 = 1 };
enum { ORC_FLAG_ADJUST_OFF = 1u, ORC_FLAG_LENGTH_NORM = 2u, ORC_FLAG_PRUNE_NORM = 8u };

typedef struct {
    int h, w;          /* coordinates in the k x V matrix (Section 3.1 names a candidate by its cell) */
    float score;
    uint64_t mask;     /* constraint marks after generating w */
    int active;        /* position of the last met token of a begun, unfinished phrase, else -1 */
    int bank;          /* number of constraint tokens met */
    int len;
} orc_cand;

typedef struct orc_sentence {
    int k, V, max_steps, pad, bos, eos;
    unsigned flags;
    float prune;       /* Section 4's pruning threshold; <= 0: no pruning */
    /* constraints flattened to positions 0..C-1 (Section 3: C = total tokens over all words and phrases) */
    int C;
    int ctok[ORC_MAX_C];
    int first[ORC_MAX_C];   /* position opens its phrase */
    int last[ORC_MAX_C];    /* position closes its phrase */
    int pstart[ORC_MAX_C];  /* first position of the phrase this position belongs to */
    int pend[ORC_MAX_C];    /* last position of that phrase */
    /* beam: k slots */
    float *score; int *tok; int *backptr; int *bank; uint64_t *mask; int *active; int *len;
    /* history of (back-pointer, token) per step, for the final trace */
    int t; int *hist_bp; int *hist_tok;
    /* last step's candidate list, kept for inspection by tests */
    orc_cand *cand; int ncand; int cand_cap;
    int alloc[ORC_MAX_C + 1]; int count[ORC_MAX_C + 1];
} orc_sentence;

static int popcount64(uint64_t v) { int c = 0; while (v) { c += (int)(v & 1u); v >>= 1; } return c; }

static float widen(const void *row, int dtype, long i)
{
    if (dtype == ORC_F32) return ((const float *)row)[i];
    uint32_t bits = ((uint32_t)((const uint16_t *)row)[i]) << 16;   /* bf16 is the top half of an fp32 */
    float f; memcpy(&f, &bits, 4); return f;
}

/* ------------------------------------------------------------------------------------------
 * Section 2: each row of the k x |V_T| matrix is a distribution over the vocabulary; Section 4
 * scores a hypothesis by its summed log-probability, so the entry is a log-probability.
 * log-sum-exp of one row, in double: lse = m + log(sum_w exp(x_w - m)), m = max_w x_w.
 * A row with no finite entry has lse = -inf.
 * ------------------------------------------------------------------------------------------ */
double orc_row_lse(const void *row, int dtype, int V)
{
    double m = -INFINITY;
    for (int w = 0; w < V; ++w) { double x = widen(row, dtype, w); if (x > m) m = x; }
    if (m == -INFINITY) return -INFINITY;
    double s = 0.0;
    for (int w = 0; w < V; ++w) s += exp((double)widen(row, dtype, w) - m);
    return m + log(s);
}

/* ------------------------------------------------------------------------------------------
 * Section 2, DECODER-STEP's last stage (the step of Algorithm 1 that produces the k x |V_T| matrix): the model output
 * for hypothesis r and word w is the inner product of the decoder's final hidden state h_r with the
 * output embedding E_w.  Plain triple loop, bf16 inputs widened exactly, accumulation in double in
 * index order, one rounding to fp32 at the end.
 *   hidden: [R, d] bf16 bits;  embed: [V, d] bf16 bits;  logits_out: [R, V] fp32.
 * ------------------------------------------------------------------------------------------ */
void orc_project(const uint16_t *hidden, const uint16_t *embed, int R, int V, int d, float *logits_out)
{
    for (int r = 0; r < R; ++r)
        for (int w = 0; w < V; ++w) {
            double acc = 0.0;
            for (int j = 0; j < d; ++j)
                acc += (double)widen(hidden + (size_t)r * d, ORC_BF16, j) * (double)widen(embed + (size_t)w * d, ORC_BF16, j);
            logits_out[(size_t)r * V + w] = (float)acc;
        }
}

/* ------------------------------------------------------------------------------------------
 * Algorithm 1, ARGMAX_K restricted to one row: the n largest entries in order, by taking the best
 * remaining entry n times (value descending; READING: the lower index first among equal values).
 * Fewer than n entries: the tail is (-inf, -1).
 * ------------------------------------------------------------------------------------------ */
void orc_row_top(const void *row, int dtype, int V, int n, float *val_out, int *idx_out)
{
    unsigned char *taken = (unsigned char *)calloc((size_t)V, 1);
    for (int i = 0; i < n; ++i) {
        int best = -1;
        for (int w = 0; w < V; ++w) {
            if (taken[w]) continue;
            if (best < 0 || widen(row, dtype, w) > widen(row, dtype, best)) best = w;
        }
        if (best < 0) { val_out[i] = -INFINITY; idx_out[i] = -1; continue; }
        taken[best] = 1;
        val_out[i] = widen(row, dtype, best); idx_out[i] = best;
    }
    free(taken);
}

/* ------------------------------------------------------------------------------------------
 * Section 3.1, last paragraph, and Algorithm 2's constraints[i].add(j).
 * State: bit j of mask = token position j is marked met; active = position of the last met token of
 * a phrase that has been begun but not finished (-1 if none).  Phrases are completed in order
 * (Fig. 1 caption).  Generating w:
 *   1. inside a begun phrase: if w is its next token, mark it; otherwise the tokens of that phrase
 *      marked so far are reset to unmet ("unwind") and rule 2 is applied to w
 *      (READING: the token that broke a phrase may itself start a constraint);
 *   2. not inside a phrase: the first position, in order, that opens a wholly unmet word/phrase and
 *      carries token w is marked (READING: lowest position when several match; continuation of the
 *      open phrase, rule 1, wins over starting another one).
 * ------------------------------------------------------------------------------------------ */
void orc_add(const orc_sentence *s, uint64_t mask, int active, int w, uint64_t *mask_out, int *active_out)
{
    if (active >= 0) {
        int n = active + 1;
        if (w == s->ctok[n]) {
            mask |= (uint64_t)1 << n;
            *mask_out = mask; *active_out = s->last[n] ? -1 : n;
            return;
        }
        for (int j = s->pstart[active]; j <= active; ++j) mask &= ~((uint64_t)1 << j);
        active = -1;
    }
    for (int j = 0; j < s->C; ++j) {
        if (s->first[j] && !((mask >> j) & 1u) && s->ctok[j] == w) {
            mask |= (uint64_t)1 << j;
            active = s->last[j] ? -1 : j;
            break;
        }
    }
    *mask_out = mask; *active_out = active;
}

/* ------------------------------------------------------------------------------------------
 * Algorithm 2's loop over the unmet constraints of hypothesis h; Section 3.1 item 2 says what they
 * are for: to make hypotheses advance through their constraints.
 * READING: the tokens taken are those whose generation raises the number of met tokens by one:
 * the next token of the begun phrase if there is one, otherwise the opening token of every wholly
 * unmet word/phrase.  Duplicate token ids are merged.  Returns the number written to out[].
 * ------------------------------------------------------------------------------------------ */
int orc_progress_set(const orc_sentence *s, uint64_t mask, int active, int *out)
{
    int n = 0;
    if (active >= 0) { out[n++] = s->ctok[active + 1]; return n; }
    for (int j = 0; j < s->C; ++j) {
        if (!s->first[j] || ((mask >> j) & 1u)) continue;
        int seen = 0;
        for (int i = 0; i < n; ++i) if (out[i] == s->ctok[j]) seen = 1;
        if (!seen) out[n++] = s->ctok[j];
    }
    return n;
}

/* ------------------------------------------------------------------------------------------
 * Section 3.2.  C + 1 banks (bank b = b constraint tokens met, bank 0 included).
 * Base: every bank gets the same share, what is left goes to the topmost bank C.
 * READING: the share is floor(k / (C + 1)); the printed floor(k / C) over C + 1 banks would hand out
 * more than k slots whenever C divides k and is undefined at C = 0, while Fig. 1 and Fig. 2
 * (k = 5, four constraints, every bank one slot) fit floor(k / (C + 1)).
 * Adjustment (the paper outlines it without giving every detail): a bank holding more slots than candidates gives the
 * surplus away, nearest banks first, moving outward, to banks with more candidates than slots, until
 * the beam holds min(k, #candidates).
 * READING: overfilled banks act in ascending order; at equal distance the higher (more constrained)
 * bank is served first; a receiver takes as much as it can use.
 * n[b] = candidates in bank b.  alloc[b] = slots of the new beam given to bank b.
 * ------------------------------------------------------------------------------------------ */
void orc_allocate(int k, int C, const int *n, unsigned flags, int *alloc)
{
    int share = k / (C + 1);
    for (int b = 0; b <= C; ++b) alloc[b] = share;
    alloc[C] += k - share * (C + 1);

    if (flags & ORC_FLAG_ADJUST_OFF) {          /* Section 5 runs its grid-beam-search simulation without adjustment */
        for (int b = 0; b <= C; ++b) if (alloc[b] > n[b]) alloc[b] = n[b];
        return;
    }
    for (int b = 0; b <= C; ++b) {
        int surplus = alloc[b] - n[b];
        if (surplus <= 0) continue;
        alloc[b] = n[b];
        for (int d = 1; d <= C && surplus > 0; ++d) {
            int nb[2] = { b + d, b - d };
            for (int q = 0; q < 2 && surplus > 0; ++q) {
                int r = nb[q];
                if (r < 0 || r > C) continue;
                int room = n[r] - alloc[r];
                if (room <= 0) continue;
                int g = surplus < room ? surplus : room;
                alloc[r] += g; surplus -= g;
            }
        }
        /* whatever is left cannot be placed: fewer than k candidates exist */
    }
}

/* ------------------------------------------------------------------------------------------ */

orc_sentence *orc_create(int k, int V, int max_steps, int pad, int bos, int eos, unsigned flags,
                         int n_phrases, const int *phrase_off, const int *tok)
{
    if (k < 1 || V < 1 || max_steps < 1 || n_phrases < 0) return NULL;
    int C = n_phrases ? phrase_off[n_phrases] - phrase_off[0] : 0;
    if (C > ORC_MAX_C) return NULL;
    orc_sentence *s = (orc_sentence *)calloc(1, sizeof *s);
    s->k = k; s->V = V; s->max_steps = max_steps; s->pad = pad; s->bos = bos; s->eos = eos; s->flags = flags;
    s->C = C;
    int j = 0;
    for (int p = 0; p < n_phrases; ++p) {
        int a = phrase_off[p], b = phrase_off[p + 1];
        if (b <= a) { free(s); return NULL; }
        int start = j;
        for (int i = a; i < b; ++i, ++j) {
            int w = tok[i];
            if (w < 0 || w >= V || w == pad || w == bos || w == eos) { free(s); return NULL; }
            s->ctok[j] = w; s->first[j] = (i == a); s->last[j] = (i == b - 1);
            s->pstart[j] = start; s->pend[j] = start + (b - a) - 1;
        }
    }
    s->score = (float *)malloc(sizeof(float) * k);   s->tok = (int *)malloc(sizeof(int) * k);
    s->backptr = (int *)malloc(sizeof(int) * k);     s->bank = (int *)malloc(sizeof(int) * k);
    s->mask = (uint64_t *)malloc(sizeof(uint64_t) * k); s->active = (int *)malloc(sizeof(int) * k);
    s->len = (int *)malloc(sizeof(int) * k);
    s->hist_bp = (int *)malloc(sizeof(int) * (size_t)k * max_steps);
    s->hist_tok = (int *)malloc(sizeof(int) * (size_t)k * max_steps);
    s->cand_cap = k * (C + 2) + k;
    s->cand = (orc_cand *)malloc(sizeof(orc_cand) * s->cand_cap);
    /* Algorithm 1, DECODER-INIT: READING: one live hypothesis holding the start symbol with score 0;
       the other k-1 slots are empty (score -inf) and produce nothing until they are filled. */
    for (int h = 0; h < k; ++h) {
        s->score[h] = -INFINITY; s->tok[h] = pad; s->backptr[h] = 0; s->bank[h] = -1;
        s->mask[h] = 0; s->active[h] = -1; s->len[h] = 0;
    }
    s->score[0] = 0.0f; s->tok[0] = bos; s->bank[0] = 0;
    s->t = 0; s->ncand = 0;
    return s;
}

void orc_destroy(orc_sentence *s)
{
    if (!s) return;
    free(s->score); free(s->tok); free(s->backptr); free(s->bank); free(s->mask); free(s->active);
    free(s->len); free(s->hist_bp); free(s->hist_tok); free(s->cand); free(s);
}

int orc_num_constraints(const orc_sentence *s) { return s->C; }
int orc_steps_done(const orc_sentence *s) { return s->t; }

void orc_get_beam(const orc_sentence *s, float *score, int *tok, int *backptr, int *bank,
                  uint64_t *mask, int *active, int *len)
{
    for (int h = 0; h < s->k; ++h) {
        if (score) score[h] = s->score[h];
        if (tok) tok[h] = s->tok[h];
        if (backptr) backptr[h] = s->backptr[h];
        if (bank) bank[h] = s->bank[h];
        if (mask) mask[h] = s->mask[h];
        if (active) active[h] = s->active[h];
        if (len) len[h] = s->len[h];
    }
}

/* Overwrites the beam (tests use it to start a step from a hand-made state). */
void orc_set_beam(orc_sentence *s, const float *score, const int *tok, const uint64_t *mask,
                  const int *active, const int *len)
{
    for (int h = 0; h < s->k; ++h) {
        s->score[h] = score[h]; s->tok[h] = tok[h]; s->mask[h] = mask[h]; s->active[h] = active[h];
        s->len[h] = len ? len[h] : 0; s->bank[h] = isinf(score[h]) ? -1 : popcount64(mask[h]);
        s->backptr[h] = 0;
    }
}

int orc_last_candidates(const orc_sentence *s, int cap, int *h, int *w, float *score, int *bank,
                        uint64_t *mask, int *active)
{
    int n = s->ncand < cap ? s->ncand : cap;
    for (int i = 0; i < n; ++i) {
        h[i] = s->cand[i].h; w[i] = s->cand[i].w; score[i] = s->cand[i].score; bank[i] = s->cand[i].bank;
        if (mask) mask[i] = s->cand[i].mask;
        if (active) active[i] = s->cand[i].active;
    }
    return s->ncand;
}

void orc_last_allocation(const orc_sentence *s, int *count, int *alloc)
{
    for (int b = 0; b <= s->C; ++b) { count[b] = s->count[b]; alloc[b] = s->alloc[b]; }
}

/* order used everywhere two cells compete: higher score first, then lower flat index h*V + w
   (READING: the paper does not say how equal scores are ordered) */
static int better(float sa, long fa, float sb, long fb)
{
    if (sa != sb) return sa > sb;
    return fa < fb;
}

/* insertion sort by (score desc, flat asc): the arrays are tiny */
static void sort_cands(orc_cand *c, int n, int V)
{
    for (int i = 1; i < n; ++i) {
        orc_cand x = c[i]; long fx = (long)x.h * V + x.w; int j = i - 1;
        while (j >= 0 && better(x.score, fx, c[j].score, (long)c[j].h * V + c[j].w)) { c[j + 1] = c[j]; --j; }
        c[j + 1] = x;
    }
}

static void push_cand(orc_sentence *s, int h, int w, float score)
{
    for (int i = 0; i < s->ncand; ++i)                   /* a set: each (h, w) once */
        if (s->cand[i].h == h && s->cand[i].w == w) return;
    orc_cand *c = &s->cand[s->ncand++];
    c->h = h; c->w = w; c->score = score;
    if (s->tok[h] == s->eos) {                           /* finished hypothesis carried forward unchanged */
        c->mask = s->mask[h]; c->active = s->active[h]; c->len = s->len[h];
    } else {
        orc_add(s, s->mask[h], s->active[h], w, &c->mask, &c->active);
        c->len = s->len[h] + 1;
    }
    c->bank = popcount64(c->mask);
}

/* ------------------------------------------------------------------------------------------
 * One call of KBEST-DBA (Algorithm 2) for this sentence.
 * logits: k rows of V entries, row h belongs to beam slot h, rows row_stride entries apart.
 * lse_out (optional): the k row normalisers as used (fp32; 0 for rows that are not open).
 * Returns 0, or -1 if max_steps calls have been made already.
 * ------------------------------------------------------------------------------------------ */
int orc_step(orc_sentence *s, const void *logits, int dtype, long row_stride, float *lse_out)
{
    const int k = s->k, V = s->V, C = s->C;
    if (s->t >= s->max_steps) return -1;
    const size_t esz = dtype == ORC_F32 ? 4 : 2;

    /* --- the k x V score matrix (Section 2; Section 3.1: rows are distributions) ------------------
       slot kinds (READING): empty = score -inf; finished = last token is the end token; open = the rest.
       open row:     score(h, w) = fl32(fl32(x - lse_h) + parent_h), lse_h = fl32(double log-sum-exp)
       finished row: only the end token again, at the parent's score (stays on the beam, frozen)
       empty row:    nothing
       Section 3.3: an open hypothesis that has not met all C tokens may not generate the end token:
       its entry is -inf (READING: applied after normalisation, no renormalisation). */
    float *S = (float *)malloc(sizeof(float) * (size_t)k * V);
    float *lse = (float *)calloc(k, sizeof(float));
    for (int h = 0; h < k; ++h) {
        float *Sh = S + (size_t)h * V;
        const char *row = (const char *)logits + (size_t)h * row_stride * esz;
        for (int w = 0; w < V; ++w) Sh[w] = -INFINITY;
        if (isinf(s->score[h])) continue;                               /* empty */
        if (s->tok[h] == s->eos) { Sh[s->eos] = s->score[h]; continue; } /* finished */
        lse[h] = (float)orc_row_lse(row, dtype, V);
        if (isinf(lse[h])) continue;
        for (int w = 0; w < V; ++w) {
            float x = widen(row, dtype, w);
            if (x == -INFINITY) continue;
            volatile float d = x - lse[h];
            volatile float sc = d + s->score[h];
            Sh[w] = sc;
        }
        if (popcount64(s->mask[h]) < C) Sh[s->eos] = -INFINITY;
    }
    if (lse_out) memcpy(lse_out, lse, sizeof(float) * k);

    s->ncand = 0;
    /* --- Algorithm 2, top overall k (Section 3.1 item 1): the k best cells of the whole matrix ------ */
    {
        unsigned char *taken = (unsigned char *)calloc((size_t)k * V, 1);
        for (int i = 0; i < k; ++i) {
            long best = -1;
            for (long f = 0; f < (long)k * V; ++f) {
                if (taken[f] || S[f] == -INFINITY) continue;
                if (best < 0 || better(S[f], f, S[best], best)) best = f;
            }
            if (best < 0) break;
            taken[best] = 1;
            push_cand(s, (int)(best / V), (int)(best % V), S[best]);
        }
        free(taken);
    }
    /* --- for each hypothesis: its unmet constraints, then its single best word -------------------- */
    for (int h = 0; h < k; ++h) {
        const float *Sh = S + (size_t)h * V;
        if (isinf(s->score[h])) continue;
        if (s->tok[h] != s->eos) {
            int prog[ORC_MAX_C];
            int np = orc_progress_set(s, s->mask[h], s->active[h], prog);
            for (int i = 0; i < np; ++i)
                if (Sh[prog[i]] != -INFINITY) push_cand(s, h, prog[i], Sh[prog[i]]);
        }
        int wbest = -1;
        for (int w = 0; w < V; ++w)
            if (Sh[w] != -INFINITY && (wbest < 0 || Sh[w] > Sh[wbest])) wbest = w;   /* lowest w on ties */
        if (wbest >= 0) push_cand(s, h, wbest, Sh[wbest]);
    }

    /* --- ALLOCATE (Section 3.2) --------------------------------------------------------------------- */
    for (int b = 0; b <= C; ++b) s->count[b] = 0;
    for (int i = 0; i < s->ncand; ++i) s->count[s->cand[i].bank]++;
    orc_allocate(k, C, s->count, s->flags, s->alloc);

    /* Section 3.1: the candidates are split by bank and ordered inside each bank;
       bank b keeps its alloc[b] best. */
    orc_cand *kept = (orc_cand *)malloc(sizeof(orc_cand) * (k + 1));
    orc_cand *tmp = (orc_cand *)malloc(sizeof(orc_cand) * (s->ncand + 1));
    int nkept = 0;
    for (int b = 0; b <= C; ++b) {
        int nb = 0;
        for (int i = 0; i < s->ncand; ++i) if (s->cand[i].bank == b) tmp[nb++] = s->cand[i];
        sort_cands(tmp, nb, V);
        for (int i = 0; i < s->alloc[b] && i < nb; ++i) kept[nkept++] = tmp[i];
    }
    /* Section 3.1: a beam is held in decreasing score order, best hypothesis first
       (READING: one global order, not bank by bank). */
    sort_cands(kept, nkept, V);

    /* Section 4 (and Section 6.3): threshold pruning of the beam.  A hypothesis whose log-probability is not
       within the threshold of the best completed hypothesis is removed, whether it is itself complete or not.
       READING: both sides of the comparison are cumulative log-probabilities (the scores the beam is ordered
       by); a removed hypothesis leaves an empty slot and the hypotheses behind it move up.
       OTHER READING (ORC_FLAG_PRUNE_NORM): Section 4 first says that completed hypotheses are normalised
       (cumulative score divided by the number of words) and then states the pruning rule, so the value a
       completed hypothesis enters the comparison with is its normalised score (on both sides: as the
       reference, and when it is itself tested); a hypothesis that is not completed enters with its cumulative
       score.  The beam stays ordered by cumulative score. */
    if (s->prune > 0) {
        float *val = (float *)malloc(sizeof(float) * (nkept + 1));
        for (int i = 0; i < nkept; ++i) {
            val[i] = kept[i].score;
            if ((s->flags & ORC_FLAG_PRUNE_NORM) && kept[i].w == s->eos && kept[i].len > 0)
                val[i] = kept[i].score / (float)kept[i].len;
        }
        float best = -INFINITY;
        for (int i = 0; i < nkept; ++i)
            if (kept[i].w == s->eos && val[i] > best) best = val[i];
        if (best != -INFINITY) {
            volatile float cut = best - s->prune;
            int n = 0;
            for (int i = 0; i < nkept; ++i)
                if (!(val[i] < cut)) kept[n++] = kept[i];
            nkept = n;
        }
        free(val);
    }

    int *hb = s->hist_bp + (size_t)s->t * k, *ht = s->hist_tok + (size_t)s->t * k;
    for (int i = 0; i < k; ++i) {
        if (i < nkept) {
            s->score[i] = kept[i].score; s->tok[i] = kept[i].w; s->backptr[i] = kept[i].h;
            s->bank[i] = kept[i].bank; s->mask[i] = kept[i].mask; s->active[i] = kept[i].active;
            s->len[i] = kept[i].len;
        } else {
            s->score[i] = -INFINITY; s->tok[i] = s->pad; s->backptr[i] = 0; s->bank[i] = -1;
            s->mask[i] = 0; s->active[i] = -1; s->len[i] = 0;
        }
        hb[i] = s->backptr[i]; ht[i] = s->tok[i];
    }
    s->t++;
    free(kept); free(tmp); free(S); free(lse);
    return 0;
}

/* Section 4's pruning threshold ("within 20" in the paper's experiments); <= 0 switches pruning off. */
void orc_set_prune(orc_sentence *s, float threshold) { s->prune = threshold; }

/* ------------------------------------------------------------------------------------------
 * Section 4: "Decoding stops when either all hypotheses still on the beam are completed or the maximum
 * length is reached"; Section 6.4's alternative, early stopping, stops at the first completed hypothesis.
 * Bit 0: the beam is not empty and every hypothesis on it is completed.  Bit 1: some hypothesis on the
 * beam is completed.  The caller owns the loop and decides which to act on.
 * ------------------------------------------------------------------------------------------ */
int orc_stop_flags(const orc_sentence *s)
{
    int live = 0, done = 0;
    for (int h = 0; h < s->k; ++h) {
        if (isinf(s->score[h])) continue;
        ++live;
        if (s->tok[h] == s->eos) ++done;
    }
    return (live > 0 && done == live ? 1 : 0) | (done > 0 ? 2 : 0);
}

/* ------------------------------------------------------------------------------------------
 * Section 3.3: the result is the completed hypothesis with the highest score; Section 4: completed hypotheses may
 * be normalised by the number of words (READING: generated tokens, end token included; only with
 * ORC_FLAG_LENGTH_NORM).  If nothing is completed (READING, by analogy with grid beam search returning
 * from the topmost bank): the best live slot of the highest occupied bank, flagged not completed.
 * tokens_out: the generated tokens (start symbol excluded) up to and including the first end token.
 * ------------------------------------------------------------------------------------------ */
void orc_finalize(const orc_sentence *s, int *tokens_out, int *len_out, float *score_out, int *completed_out)
{
    const int k = s->k;
    int pick = -1; float pickval = 0;
    for (int h = 0; h < k; ++h) {
        if (isinf(s->score[h]) || s->tok[h] != s->eos) continue;
        float v = s->score[h];
        if ((s->flags & ORC_FLAG_LENGTH_NORM) && s->len[h] > 0) v = s->score[h] / (float)s->len[h];
        if (pick < 0 || v > pickval) { pick = h; pickval = v; }
    }
    int completed = pick >= 0;
    if (!completed) {
        int bestbank = -1;
        for (int h = 0; h < k; ++h) {
            if (isinf(s->score[h])) continue;
            int b = popcount64(s->mask[h]);
            if (b > bestbank || (b == bestbank && s->score[h] > pickval)) { bestbank = b; pick = h; pickval = s->score[h]; }
        }
    }
    *completed_out = completed;
    if (pick < 0 || s->t == 0) { *len_out = 0; *score_out = pick < 0 ? -INFINITY : pickval; return; }
    *score_out = pickval;
    int *rev = (int *)malloc(sizeof(int) * s->t);
    int slot = pick;
    for (int t = s->t - 1; t >= 0; --t) {
        rev[t] = s->hist_tok[(size_t)t * k + slot];
        slot = s->hist_bp[(size_t)t * k + slot];
    }
    int n = 0;
    for (int t = 0; t < s->t; ++t) { tokens_out[n++] = rev[t]; if (rev[t] == s->eos) break; }
    *len_out = n;
    free(rev);
}
