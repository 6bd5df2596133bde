"""The input generators: determinism, shapes and the distributions the workloads promise.  No GPU."""
import numpy as np

from synth_inputs import CONFIGS, LogitStream, make_workload
from synth_inputs.logits import bf16_bits_to_f32, mix, normal_table, to_bf16_bits


def test_mix_is_splitmix64():
    # first outputs of splitmix64 seeded with 0 (state advances by the golden-ratio constant)
    golden = np.uint64(0x9E3779B97F4A7C15)
    with np.errstate(over="ignore"):
        got = [int(mix(np.uint64(i) * golden)) for i in range(3)]
    assert got == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


def test_normal_table_is_standard_normal():
    q = normal_table().astype(np.float64)
    assert abs(q.mean()) < 1e-6 and abs(q.std() - 1.0) < 1e-3
    assert np.all(np.diff(q) > 0) and q[32768] > 0 > q[32767]


def test_bf16_round_trip_is_nearest_even():
    x = np.array([1.0, 1.00390625, 1.01171875, -3.0078125], np.float32)   # ties at the bf16 half-way point
    b = to_bf16_bits(x)
    assert bf16_bits_to_f32(b).tolist() == [1.0, 1.0, 1.015625, -3.0]


def test_constraint_shapes_follow_the_workloads():
    for name, p in CONFIGS.items():
        for C in ([1, 5, 10, 20, 50] if name == "scaling" else [None]):
            wl = make_workload(name, C=C)
            assert len(wl.constraints) == wl.B
            for c in wl.constraints:
                flat = [w for ph in c for w in ph]
                assert len(set(flat)) == len(flat) and all(4 <= w < wl.V for w in flat)
                if name == "tiny":
                    assert [len(ph) for ph in c] == [1, 1]
                if name == "phrasal":
                    assert len(c) == 4 and all(1 <= len(ph) <= 3 for ph in c)
                if name == "ragged":
                    assert len(flat) <= 8 and len(c) <= 4 and all(1 <= len(ph) <= 3 for ph in c)
                if name == "scaling":
                    assert len(flat) == C and all(len(ph) == 1 for ph in c)
                if name == "serving":
                    assert len(flat) == 10 and all(1 <= len(ph) <= 4 for ph in c)
    rag = make_workload("ragged")
    totals = {sum(len(p) for p in c) for c in rag.constraints}
    assert 0 in totals and max(totals) == 8
    so, po, tok = rag.csr()
    assert so[-1] == len(po) - 1 and po[-1] == len(tok)


def test_rows_depend_only_on_step_sentence_and_last_token():
    wl = make_workload("ragged", B=3, V=2000)
    ls = LogitStream(wl)
    tok = np.array([7, 9, 7] + [5] * (wl.R - 3), np.int32)
    mask = np.zeros(wl.R, np.uint64)
    a = ls.step_logits(4, tok, mask)
    b = ls.step_logits(4, tok, mask)
    assert a.dtype == np.uint16 and np.array_equal(a, b)
    assert np.array_equal(a[0], a[2]) and not np.array_equal(a[0], a[1])
    assert not np.array_equal(a[0], a[wl.k])                       # another sentence, another row
    assert not np.array_equal(a, ls.step_logits(5, tok, mask))
    sub = wl.subset([2])
    c = LogitStream(sub).step_logits(4, tok[2 * wl.k:3 * wl.k], mask[:wl.k])
    assert np.array_equal(c, a[2 * wl.k:3 * wl.k])                 # a subset keeps its streams


def test_zipf_rows_have_the_stated_shape():
    wl = make_workload("phrasal", V=8000)
    ls = LogitStream(wl)
    x = ls.step_logits(0, np.full(wl.R, 1, np.int32), np.full(wl.R, np.uint64(2**63 - 1) * 2 + 1, np.uint64))
    resid = x - ls.mu[None, :]
    resid = np.delete(resid, [2], axis=1)
    assert abs(resid.mean()) < 0.02 and abs(resid.std() - 1.0) < 0.02
    ranks = np.exp(-ls.mu[4:].astype(np.float64) / 1.1)
    assert np.allclose(np.sort(ranks), np.arange(1, wl.V - 3), rtol=1e-5)
    assert 0.5 * wl.steps <= ls.end_step[0] <= 0.9 * wl.steps
    late = ls.step_logits(int(ls.end_step[0]), np.full(wl.R, 1, np.int32), np.zeros(wl.R, np.uint64))
    assert late[:, 2].mean() > 0 > x[:, 2].mean()


def test_boost_hits_the_first_unmet_constraint_token_about_30_percent_of_the_time():
    wl = make_workload("serving", B=40, V=4000)
    ls = LogitStream(wl)
    tok = np.arange(wl.R, dtype=np.int32) % 97 + 4
    mask = np.zeros(wl.R, np.uint64); mask[::2] = 1                # odd rows: nothing met; even rows: first met
    keys = ls.row_keys(3, tok)
    bt = ls.boost_tokens(keys, mask)
    frac = (bt >= 0).mean()
    assert 0.2 < frac < 0.4
    ct, _ = wl.flat_tokens()
    for r in np.nonzero(bt >= 0)[0]:
        assert bt[r] == ct[r // wl.k, 1 if r % 2 == 0 else 0]
    full = np.full(wl.R, np.uint64(1023), np.uint64)               # everything met: nothing to boost
    assert (ls.boost_tokens(keys, full) == -1).all()
