"""CPU tests that tie the oracle to things other than itself: closed forms, the paper's captions,
hand traces, textbook beam search, brute force.  No GPU."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import dba_oracle as O

NEG = -np.inf


# ----------------------------------------------------------------------------- row log-sum-exp
def test_lse_constant_row():
    for V, c in [(1, 0.5), (7, -3.25), (1000, 2.0), (32000, -11.5)]:
        x = np.full(V, c, np.float32)
        assert abs(O.row_lse(x) - (c + math.log(V))) < 1e-12


def test_lse_two_values():
    x = np.array([1.5] * 3 + [-2.0] * 5, np.float32)
    assert abs(O.row_lse(x) - math.log(3 * math.exp(1.5) + 5 * math.exp(-2.0))) < 1e-12


def test_lse_geometric_row():
    a, V = 0.125, 400
    x = (-a * np.arange(V)).astype(np.float32)          # multiples of 1/8: exact in fp32
    closed = math.log((1 - math.exp(-a * V)) / (1 - math.exp(-a)))
    assert abs(O.row_lse(x) - closed) < 1e-12


def test_lse_shift_invariance_and_distribution():
    rng = np.random.default_rng(1)
    x = (rng.integers(-4000, 4000, 513) / 256.0).astype(np.float32)    # exact dyadic values
    l0 = O.row_lse(x)
    assert abs(O.row_lse((x + np.float32(64.0)).astype(np.float32)) - (l0 + 64.0)) < 1e-11
    assert abs(np.exp(x.astype(np.float64) - l0).sum() - 1.0) < 1e-12
    big = (x + np.float32(3000.0)).astype(np.float32)                  # exp would overflow without the max
    assert abs(O.row_lse(big) - (l0 + 3000.0)) < 1e-9


def test_lse_minus_inf_entries_and_bf16():
    x = np.array([NEG, 0.0, NEG, 0.0], np.float32)
    assert abs(O.row_lse(x) - math.log(2.0)) < 1e-15
    assert O.row_lse(np.full(5, NEG, np.float32)) == NEG
    vals = np.array([1.0, -2.5, 0.15625, 3.0], np.float32)            # exactly representable in bf16
    bits = (vals.view(np.uint32) >> 16).astype(np.uint16)
    assert abs(O.row_lse(bits) - O.row_lse(vals)) == 0.0


# ----------------------------------------------------------------------------- constraint tracker
def _parse_traces(path):
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        ph, toks, met = [f.strip() for f in line.split(";")]
        yield ([[int(t) for t in p.split()] for p in ph.split("|")],
               [int(t) for t in toks.split()], [int(t) for t in met.split()])


def test_add_hand_traces(golden_dir):
    n = 0
    for phrases, toks, met in _parse_traces(os.path.join(golden_dir, "add_traces.txt")):
        s = O.Sentence(2, 64, 4, phrases)
        mask, active = 0, -1
        got = []
        for w in toks:
            mask, active = s.add(mask, active, w)
            got.append(bin(mask).count("1"))
        assert got == met, (phrases, toks, got, met)
        n += 1
    assert n >= 10


def test_add_marks_the_positions_the_conventions_name(golden_dir):
    """Which positions are marked (tests/golden/add_masks.txt): continuation of the begun phrase wins over opening
    another constraint; of several unmet constraints opening with the token the first in order is marked."""
    n = 0
    for line in open(os.path.join(golden_dir, "add_masks.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        ph, toks, want = [f.strip() for f in line.split(";")]
        phrases = [[int(t) for t in p.split()] for p in ph.split("|")]
        s = O.Sentence(2, 64, 4, phrases)
        mask, active = 0, -1
        for w in toks.split():
            mask, active = s.add(mask, active, int(w))
        want_mask = 0 if want == "-" else sum(1 << int(t) for t in want.split())
        assert mask == want_mask, (line, bin(mask))
        n += 1
    assert n >= 8


def _phrase_bits(phrases):
    pos, out = 0, []
    for p in phrases:
        out.append(list(range(pos, pos + len(p)))); pos += len(p)
    return out


def test_add_invariants_random_walk():
    rng = np.random.default_rng(7)
    for trial in range(200):
        nph = int(rng.integers(1, 5))
        phrases = [rng.integers(4, 9, int(rng.integers(1, 4))).tolist() for _ in range(nph)]  # ids repeat a lot
        s = O.Sentence(1, 16, 4, phrases)
        bits = _phrase_bits(phrases)
        mask, active = 0, -1
        for _ in range(40):
            w = int(rng.integers(3, 10))
            before = bin(mask).count("1")
            open_len = 0
            if active >= 0:
                open_len = [active - b[0] + 1 for b in bits if b[0] <= active <= b[-1]][0]
            mask, active = s.add(mask, active, w)
            after = bin(mask).count("1")
            assert after - before in (1, 0, -open_len, -open_len + 1)
            partial = []
            for b in bits:
                marks = [(mask >> j) & 1 for j in b]
                assert marks == sorted(marks, reverse=True)        # met tokens of a phrase form a prefix
                if 0 < sum(marks) < len(b):
                    partial.append(b[0] + sum(marks) - 1)
            assert len(partial) <= 1                               # at most one phrase is open
            assert (active >= 0) == (len(partial) == 1)
            if partial:
                assert active == partial[0]


def _contains(seq, phrase):
    n = len(phrase)
    return any(seq[i:i + n] == phrase for i in range(len(seq) - n + 1))


def test_add_equals_substring_semantics_for_distinct_tokens():
    """With all constraint tokens distinct, a phrase is met exactly when it has occurred contiguously."""
    rng = np.random.default_rng(11)
    for trial in range(300):
        ids = rng.permutation(np.arange(4, 12)).tolist()
        lens = [int(rng.integers(1, 4)) for _ in range(int(rng.integers(1, 4)))]
        phrases, i = [], 0
        for L in lens:
            phrases.append(ids[i:i + L]); i += L
        s = O.Sentence(1, 16, 4, phrases)
        bits = _phrase_bits(phrases)
        seq, mask, active = [], 0, -1
        for _ in range(30):
            w = int(rng.choice(ids[:i] + [3]))
            seq.append(w)
            mask, active = s.add(mask, active, w)
            for p, b in zip(phrases, bits):
                done = all((mask >> j) & 1 for j in b)
                assert done == _contains(seq, p), (phrases, seq)


def test_progress_set_is_the_set_of_tokens_that_raise_the_met_count():
    rng = np.random.default_rng(5)
    for trial in range(200):
        phrases = [rng.integers(4, 10, int(rng.integers(1, 4))).tolist() for _ in range(int(rng.integers(1, 5)))]
        s = O.Sentence(1, 16, 4, phrases)
        mask, active = 0, -1
        for _ in range(25):
            base = bin(mask).count("1")
            brute = sorted(w for w in range(16) if bin(s.add(mask, active, w)[0]).count("1") == base + 1)
            assert sorted(s.progress_set(mask, active)) == brute
            mask, active = s.add(mask, active, int(rng.integers(3, 11)))


# ----------------------------------------------------------------------------- allocation
def test_allocation_figure_captions(golden_dir):
    rows = 0
    for line in open(os.path.join(golden_dir, "allocation_figures.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, n, exp = [f.strip() for f in line.split(";")]
        n = [int(t) for t in n.split()]
        alloc = O.allocate(int(k), n).tolist()
        assert sum(alloc) == min(int(k), sum(n))
        for a, e in zip(alloc, exp.split()):
            if e == "+":
                assert a >= 1
            elif e != "*":
                assert a == int(e)
        rows += 1
    assert rows >= 13


def test_allocation_base_share_when_every_bank_is_full():
    for k in range(1, 41):
        for C in range(0, 64):
            alloc = O.allocate(k, [k] * (C + 1))
            share = k // (C + 1)
            assert alloc.sum() == k
            assert all(alloc[:C] == share) and alloc[C] == k - share * C


def test_allocation_invariants_random():
    rng = np.random.default_rng(3)
    for trial in range(3000):
        k = int(rng.integers(1, 65)); C = int(rng.integers(0, 65))
        n = rng.integers(0, 4, C + 1) * (rng.random(C + 1) < 0.5)
        if trial % 3 == 0:
            n = rng.integers(0, 2 * k, C + 1)
        alloc = O.allocate(k, n)
        assert alloc.sum() == min(k, n.sum())            # beam filled up to min(k, #candidates)
        assert (alloc <= n).all() and (alloc >= 0).all()
        off = O.allocate(k, n, O.FLAG_ADJUST_OFF)
        share = k // (C + 1); base = np.full(C + 1, share); base[C] += k - share * (C + 1)
        assert (off == np.minimum(base, n)).all()
        assert (alloc >= off).all()                      # adjustment only ever adds to a bank's base


def test_allocation_more_constraints_than_beam():
    # C >= k: the base share is zero everywhere but the top bank, adjustment must still fill the beam
    alloc = O.allocate(5, [3, 4, 0, 0, 0, 0, 0, 0, 0, 0, 0])
    assert alloc.sum() == 5 and alloc[2:].sum() == 0
    alloc = O.allocate(3, [0] * 9 + [2, 1])
    assert alloc.tolist() == [0] * 9 + [2, 1]


# ----------------------------------------------------------------------------- whole step
def _np_lse32(row):
    return np.float32(np.logaddexp.reduce(row.astype(np.float64)))


def _np_scores(x, parent, lse):
    return ((x - lse[:, None]).astype(np.float32) + parent[:, None]).astype(np.float32)


def test_unconstrained_step_is_textbook_beam_search():
    """No constraints: one bank, so the new beam is ARGMAX_K over the k x V matrix (Algorithm 1)."""
    rng = np.random.default_rng(0)
    k, V, T = 4, 50, 8
    s = O.Sentence(k, V, T, [])
    score = np.full(k, NEG, np.float32); score[0] = 0.0
    tok = np.zeros(k, np.int32); tok[0] = 1
    for t in range(T):
        x = rng.normal(0, 2, (k, V)).astype(np.float32)
        x[:, 2] = -60.0 if t < 5 else 3.0                 # end token unlikely, then likely
        lse = np.array([_np_lse32(r) for r in x])
        S = _np_scores(x, score, lse)
        S[np.isinf(score)] = NEG
        for h in range(k):                                # finished hypotheses repeat the end token
            if np.isfinite(score[h]) and tok[h] == 2:
                S[h] = NEG; S[h, 2] = score[h]
        flat = S.ravel()
        order = np.argsort(-flat, kind="stable")[:k]
        order = [f for f in order if np.isfinite(flat[f])]
        got_lse = s.step(x)
        bm = s.beam()
        n = len(order)
        assert bm["backptr"][:n].tolist() == [f // V for f in order]
        assert bm["token"][:n].tolist() == [f % V for f in order]
        assert np.array_equal(bm["score"][:n], flat[order])
        assert np.isinf(bm["score"][n:]).all()
        live = np.isfinite(score) & (tok != 2)
        assert np.array_equal(got_lse[live], lse[live])
        score, tok = bm["score"].copy(), bm["token"].copy()


def _random_closed_loop(rng, k, V, T, phrases, eos_after=None, flags=0, quantised=False):
    s = O.Sentence(k, V, T, phrases, flags=flags)
    for t in range(T):
        before = s.beam()
        x = rng.normal(0, 2, (k, V)).astype(np.float32)
        if quantised:                                  # few distinct values: ties in every row
            x = np.round(x).astype(np.float32)
        if eos_after is not None:
            x[:, 2] = -30.0 if t < eos_after else 4.0
        s.step(x)
        yield s, before, x, s.beam()


@pytest.mark.parametrize("quantised", [False, True])
def test_candidate_set_matches_brute_force_predicate(quantised):
    rng = np.random.default_rng(42)
    for trial in range(30):
        k, V, T = int(rng.integers(1, 5)), 14, 7
        ids = rng.permutation(np.arange(4, V)).tolist()
        phrases = [ids[0:2], ids[2:3], ids[3:6]][:int(rng.integers(1, 4))]
        C = sum(len(p) for p in phrases)
        for s, b, x, after in _random_closed_loop(rng, k, V, T, phrases, eos_after=4, quantised=quantised):
            live = np.isfinite(b["score"])
            fin = live & (b["token"] == 2)
            lse = np.array([_np_lse32(r) for r in x])
            S = _np_scores(x, b["score"], lse)
            S[~live] = NEG
            for h in np.nonzero(fin)[0]:
                S[h] = NEG; S[h, 2] = b["score"][h]
            for h in np.nonzero(live & ~fin)[0]:
                if bin(int(b["met_mask"][h])).count("1") < C:
                    S[h, 2] = NEG
            order = np.argsort(-S.ravel(), kind="stable")
            rank = np.empty(k * V, np.int64); rank[order] = np.arange(k * V)
            want = set()
            for h in range(k):
                if not live[h]:
                    continue
                base = bin(int(b["met_mask"][h])).count("1")
                wbest = int(np.argmax(S[h]))
                for w in range(V):
                    if not np.isfinite(S[h, w]):
                        continue
                    progress = (not fin[h]) and \
                        bin(s.add(int(b["met_mask"][h]), int(b["active"][h]), w)[0]).count("1") == base + 1
                    if rank[h * V + w] < k or progress or w == wbest:
                        want.add((h, w))
            c = s.candidates()
            got = set(zip(c["h"].tolist(), c["w"].tolist()))
            assert len(got) == len(c["h"])                                   # no duplicates
            assert got == want
            for h, w, sc, bank, m in zip(c["h"], c["w"], c["score"], c["bank"], c["met_mask"]):
                assert sc == S[h, w] and bank == bin(int(m)).count("1")
            # bookkeeping is bounded by k * (unmet + 2) whatever C is (Table 1: constant in C)
            assert len(got) <= k * (C + 2)
            cnt, alloc = s.allocation()
            assert alloc.sum() == min(k, len(got)) == np.isfinite(after["score"]).sum()


def test_no_end_token_before_all_constraints_and_outputs_hold_them():
    rng = np.random.default_rng(9)
    completed = 0
    for trial in range(40):
        k, V, T = int(rng.integers(2, 7)), 24, 14
        ids = rng.permutation(np.arange(4, V)).tolist()
        phrases = [ids[0:2], ids[2:3], ids[3:6], ids[6:7]][:int(rng.integers(1, 5))]
        C = sum(len(p) for p in phrases)
        s = None
        for s, b, x, after in _random_closed_loop(rng, k, V, T, phrases, eos_after=3):
            for h in range(k):
                if np.isfinite(after["score"][h]) and after["token"][h] == 2:
                    assert bin(int(after["met_mask"][h])).count("1") == C
            sc = after["score"][np.isfinite(after["score"])]
            assert (np.diff(sc) <= 0).all()                                   # beam in decreasing order
        toks, score, done = s.finalize()
        if done:
            completed += 1
            assert toks[-1] == 2 and 2 not in toks[:-1]
            for p in phrases:
                assert _contains(toks, p)
    assert completed >= 30          # a beam of >= 2 always gets the constraints in (Section 5)


def _history_rows(rng_seed, hist, V):
    out = np.empty((len(hist), V), np.float32)
    for i, h in enumerate(hist):
        out[i] = np.random.default_rng([rng_seed] + list(h)).normal(0, 1.5, V).astype(np.float32)
    return out


@pytest.mark.parametrize("phrases", [[[3]], [[4, 5]], [[3], [5, 4]], []])
def test_exhaustive_regime_equals_brute_force_over_all_sequences(phrases):
    """Beam large enough that nothing is ever cut: the result is the best complete, all-constraints
    sequence of the whole search space."""
    V, N, seed = 6, 4, 123
    k = V ** N + 8
    s = O.Sentence(k, V, N, phrases)
    hist = [(1,)] + [()] * (k - 1)
    for t in range(N):
        b = s.beam()
        x = _history_rows(seed, [h if h else (0,) for h in hist], V)
        s.step(x)
        a = s.beam()
        hist = [hist[a["backptr"][i]] + (int(a["token"][i]),) if np.isfinite(a["score"][i]) else ()
                for i in range(k)]
        assert np.isfinite(a["score"]).sum() < k          # never full: nothing was cut
    toks, score, done = s.finalize()

    best, best_seq = -np.inf, None
    for L in range(1, N + 1):
        for body in itertools.product([0, 1, 3, 4, 5], repeat=L - 1):
            seq = list(body) + [2]
            if not all(_contains(seq, p) for p in phrases):
                continue
            sc, h = np.float32(0.0), (1,)
            for w in seq:
                row = _history_rows(seed, [h], V)[0]
                sc = np.float32(np.float32(row[w] - _np_lse32(row)) + sc)
                h = h + (w,)
            if sc > best:
                best, best_seq = sc, seq
    assert done and toks == best_seq and score == best


def test_ties_go_to_the_lowest_flat_index():
    """Quantised logits make equal scores common; the textbook stable sort keeps the lowest h*V + w."""
    rng = np.random.default_rng(21)
    k, V, T = 3, 12, 6
    for trial in range(20):
        s = O.Sentence(k, V, T, [])
        score = np.full(k, NEG, np.float32); score[0] = 0.0
        for t in range(T):
            x = rng.integers(0, 2, (k, V)).astype(np.float32)       # only two distinct values per row
            x[:, 2] = -40.0
            if t > 0:
                x[1] = x[0]                                         # identical rows as well
            lse = np.array([_np_lse32(r) for r in x])
            S = _np_scores(x, score, lse); S[np.isinf(score)] = NEG
            order = [f for f in np.argsort(-S.ravel(), kind="stable")[:k] if np.isfinite(S.ravel()[f])]
            s.step(x)
            bm = s.beam()
            assert bm["backptr"][:len(order)].tolist() == [f // V for f in order]
            assert bm["token"][:len(order)].tolist() == [f % V for f in order]
            score = bm["score"].copy()
    # a constant row: the k lowest token ids, in order
    s = O.Sentence(4, 9, 2, [])
    s.step(np.zeros((4, 9), np.float32))
    assert s.beam()["token"].tolist() == [0, 1, 2, 3]


def test_length_normalisation_divides_completed_scores_by_their_length():
    k, V = 2, 6
    for flags, want in [(0, np.float32(-4.0)), (O.FLAG_LENGTH_NORM, np.float32(-1.0))]:
        s = O.Sentence(k, V, 3, [], flags=flags)
        s.set_beam([-4.0, -5.0], [2, 2], [0, 0], [-1, -1], [2, 5])    # two finished hypotheses
        s.step(np.zeros((k, V), np.float32))
        bm = s.beam()
        assert bm["len"].tolist() == [2, 5] and bm["token"].tolist() == [2, 2]
        toks, score, done = s.finalize()
        assert done and score == want
    # lengths count generated tokens, end token included
    rng = np.random.default_rng(2)
    s = O.Sentence(3, 10, 9, [[5]], flags=O.FLAG_LENGTH_NORM)
    for t in range(9):
        x = rng.normal(0, 1, (3, 10)).astype(np.float32); x[:, 2] = -20.0 if t < 4 else 5.0
        s.step(x)
    toks, score, done = s.finalize()
    bm = s.beam()
    fin = [h for h in range(3) if np.isfinite(bm["score"][h]) and bm["token"][h] == 2]
    assert done and any(bm["len"][h] == len(toks) and np.float32(bm["score"][h] / np.float32(len(toks))) == score
                        for h in fin)


def test_row_top_is_a_stable_descending_sort():
    rng = np.random.default_rng(17)
    for V, n in [(1, 3), (5, 5), (40, 7), (300, 22)]:
        for quant in (False, True):
            x = rng.normal(0, 2, V).astype(np.float32)
            if quant:
                x = np.round(x)
                x[rng.integers(0, V)] = NEG
            val, idx = O.row_top(x, n)
            order = np.argsort(-x, kind="stable")[:n]
            m = min(n, V)
            assert idx[:m].tolist() == order.tolist() and np.array_equal(val[:m], x[order])
            assert (idx[m:] == -1).all() and np.isinf(val[m:]).all()


# ------------------------------------------------------------------------------------------ pruning, stopping
def test_pruning_keeps_exactly_the_hypotheses_within_the_threshold_of_the_best_completed_one():
    """Section 4: a hypothesis is removed when its log-probability is not within the threshold of the best
    completed hypothesis.  Vocabulary {pad, bos, eos, a}: the first step offers the end token with logit 0 and
    `a` with logit -d, so the two continuations score -log(1+e^-d) and -d - log(1+e^-d): exactly d apart."""
    for d, theta, kept in [(5.0, 20.0, True), (19.5, 20.0, True), (20.5, 20.0, False), (25.0, 20.0, False),
                           (2.5, 3.0, True), (3.5, 3.0, False), (25.0, 0.0, True)]:
        s = O.Sentence(3, 4, 2, [], prune=theta)
        x = np.full((3, 4), NEG, np.float32); x[0, 2] = 0.0; x[0, 3] = -d
        s.step(x)
        bm = s.beam()
        lse = np.log1p(np.exp(-d))
        assert bm["token"][0] == 2 and abs(bm["score"][0] + lse) < 1e-6
        if kept:
            assert bm["token"][1] == 3 and abs(bm["score"][1] + d + lse) < 1e-5 and s.stop_flags() == 2
        else:       # the slot is empty, and then everything on the beam is completed
            assert np.isinf(bm["score"][1]) and bm["token"][1] == 0 and bm["bank"][1] == -1 and s.stop_flags() == 3
        assert np.isinf(bm["score"][2])


def test_pruning_removes_completed_hypotheses_too_and_never_the_best_completed_one():
    k, V = 4, 4
    s = O.Sentence(k, V, 3, [], prune=20.0)
    assert s.stop_flags() == 0                       # nothing completed at the start
    s.set_beam([-1.0, -30.0, -5.0, NEG], [2, 2, 3, 0], [0] * 4, [-1] * 4, [1, 1, 1, 0])
    x = np.full((k, V), NEG, np.float32); x[2, 2] = 0.0; x[2, 3] = 0.0        # the open one: two equal choices
    s.step(x)
    bm = s.beam()
    half = np.float32(-5.0) + np.float32(-np.log(2.0))
    assert bm["score"][0] == np.float32(-1.0) and bm["token"][0] == 2 and bm["backptr"][0] == 0
    assert bm["backptr"][1:3].tolist() == [2, 2] and bm["token"][1:3].tolist() == [2, 3]
    assert np.allclose(bm["score"][1:3], half, atol=1e-6)
    assert np.isinf(bm["score"][3])                  # the completed hypothesis at -30 is gone
    assert s.stop_flags() == 2
    # without pruning it stays
    u = O.Sentence(k, V, 3, [])
    u.set_beam([-1.0, -30.0, -5.0, NEG], [2, 2, 3, 0], [0] * 4, [-1] * 4, [1, 1, 1, 0])
    u.step(x)
    assert u.beam()["score"][3] == np.float32(-30.0) and u.beam()["token"][3] == 2


def test_pruning_by_normalised_completed_scores_removes_what_the_hand_calculation_says():
    """Section 4 normalises completed hypotheses (score / number of words) before it states the pruning rule.
    Under that reading (ORC_FLAG_PRUNE_NORM) a beam of two completed hypotheses, A (-6 over 3 words: -2 per word)
    and B (-5 over 1 word), and two open ones whose only continuation has probability 1 (C at -3.5, D at -4.5)
    with threshold 2 keeps what is within 2 of A's -2: A (-2) and C (-3.5); B (-5) and D (-4.5) go.  Under the
    default reading the reference is B's -5 and all four stay (all >= -7)."""
    k, V = 4, 4
    x = np.full((k, V), NEG, np.float32); x[2, 3] = 0.0; x[3, 3] = 0.0       # open rows: one word, probability 1
    beam = ([-5.0, -6.0, -3.5, -4.5], [2, 2, 3, 3], [0] * 4, [-1] * 4, [1, 3, 2, 2])
    s = O.Sentence(k, V, 3, [], flags=O.FLAG_PRUNE_NORM, prune=2.0)
    s.set_beam(*beam)
    s.step(x)
    bm = s.beam()
    # the beam stays in order of cumulative score: C (-3.5, from slot 2) before A (-6, from slot 1)
    assert bm["score"][:2].tolist() == [-3.5, -6.0] and bm["backptr"][:2].tolist() == [2, 1]
    assert bm["token"][:2].tolist() == [3, 2] and np.isinf(bm["score"][2:]).all()
    u = O.Sentence(k, V, 3, [], prune=2.0)
    u.set_beam(*beam)
    u.step(x)
    bu = u.beam()
    assert bu["score"].tolist() == [-3.5, -4.5, -5.0, -6.0] and bu["backptr"].tolist() == [2, 3, 0, 1]
    # a threshold that reaches everything: the two readings agree again
    w = O.Sentence(k, V, 3, [], flags=O.FLAG_PRUNE_NORM, prune=10.0)
    w.set_beam(*beam)
    w.step(x)
    assert np.array_equal(w.beam()["score"], bu["score"])


def test_stop_bit_zero_needs_every_hypothesis_on_the_beam_completed():
    s = O.Sentence(3, 5, 4, [])
    s.set_beam([-1.0, -2.0, NEG], [2, 2, 0], [0] * 3, [-1] * 3, [2, 2, 0])
    assert s.stop_flags() == 3
    s.step(np.zeros((3, 5), np.float32))             # completed hypotheses repeat the end token, frozen
    assert s.stop_flags() == 3 and s.beam()["score"][:2].tolist() == [-1.0, -2.0]
    s.set_beam([-1.0, -2.0, -3.0], [2, 4, 2], [0] * 3, [-1] * 3, [2, 2, 2])
    assert s.stop_flags() == 2


def test_a_huge_threshold_changes_nothing_and_survivors_are_always_within_the_threshold():
    rng = np.random.default_rng(5)
    k, V, T = 6, 40, 14
    phrases = [[7, 8], [9]]
    a, b, c = O.Sentence(k, V, T, phrases), O.Sentence(k, V, T, phrases, prune=1e30), O.Sentence(k, V, T, phrases, prune=2.0)
    pruned_something = False
    for t in range(T):
        x = rng.normal(0, 2, (k, V)).astype(np.float32)
        x[:, 2] += 2.0 if t > 3 else -5.0
        x[:, 7:10] += 3.0
        for s in (a, b, c):
            s.step(x)
        ba, bb, bc = a.beam(), b.beam(), c.beam()
        for f in ("score", "token", "backptr", "bank", "met_mask", "active"):
            assert np.array_equal(ba[f], bb[f])
        live = np.isfinite(bc["score"])
        done = live & (bc["token"] == 2)
        if done.any():
            best = bc["score"][done].max()
            assert (bc["score"][live] >= np.float32(best - np.float32(2.0))).all()
            pruned_something |= live.sum() < np.isfinite(ba["score"]).sum()
        assert (np.diff(live.astype(int)) <= 0).all()
    assert pruned_something


# ------------------------------------------------------------------------------------------ output projection
def _bf16(x):
    from synth_inputs.logits import to_bf16_bits
    return to_bf16_bits(np.ascontiguousarray(x, np.float32))


def test_projection_closed_forms():
    """Section 2: the score matrix is the hidden states times the output embedding.  A one-hot hidden state
    picks a column of the embedding; a constant one gives scaled row sums; small integers multiply exactly; a
    transposed operand or a dropped term fails one of these."""
    from synth_inputs.logits import bf16_bits_to_f32
    rng = np.random.default_rng(11)
    V, d = 37, 24
    E = rng.normal(0, 1, (V, d)).astype(np.float32)
    Eb = _bf16(E); Ef = bf16_bits_to_f32(Eb).astype(np.float64)
    H = np.zeros((d, d), np.float32); H[np.arange(d), np.arange(d)] = 1.0          # row j is the j-th unit vector
    got = O.project(_bf16(H), Eb)
    assert got.shape == (d, V) and np.array_equal(got, Ef.T.astype(np.float32))
    H = np.full((2, d), 0.5, np.float32); H[1] = -2.0
    got = O.project(_bf16(H), Eb)
    assert np.array_equal(got[0], (0.5 * Ef.sum(1)).astype(np.float32))
    assert np.array_equal(got[1], (-2.0 * Ef.sum(1)).astype(np.float32))
    Hi = rng.integers(-8, 9, (5, d)).astype(np.float32); Ei = rng.integers(-8, 9, (V, d)).astype(np.float32)
    got = O.project(_bf16(Hi), _bf16(Ei))
    assert np.array_equal(got, (Hi.astype(np.int64) @ Ei.astype(np.int64).T).astype(np.float32))
    # not symmetric in its operands: the shapes alone catch a transposition
    assert O.project(_bf16(Hi[:3]), _bf16(Ei)).shape == (3, V)
