"""GPU parity tests: the CUDA library (through its C ABI) against the CPU oracle, element by element."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from oracle import dba_oracle as O                                    # noqa: E402
from synth_inputs import LogitStream, make_workload                   # noqa: E402
from tests.parity import (assert_beam_equal, assert_finalize_equal, gpu_beam, lockstep, to_device_logits,  # noqa: E402
                          to_host_logits)


@pytest.fixture(scope="module")
def dba():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_1804_06609_b200 as pkg
    pkg.lib()                    # raises if libdba.so is missing: no fallback
    return pkg


def _stepper(dba, wl, steps=None, flags=0):
    return dba.DbaStepper(wl.B, wl.k, wl.V, steps or wl.steps, constraints=wl.constraints,
                          dtype=dba.BF16 if wl.dtype == "bf16" else dba.F32, flags=flags)


# ------------------------------------------------------------------------------------------ generators
@pytest.mark.parametrize("name,kw", [("tiny", {}), ("phrasal", dict(V=5003)), ("ragged", dict(B=5, V=4096)),
                                     ("serving", dict(B=3, V=6001))])
def test_gpu_generator_writes_the_same_bits_as_numpy(dba, name, kw):
    from synth_inputs.gpu import GpuLogitStream
    wl = make_workload(name, **kw)
    host, dev = LogitStream(wl), GpuLogitStream(wl)
    rng = np.random.default_rng(0)
    for step in (0, 3, wl.steps - 1):
        tok = rng.integers(0, wl.V, wl.R).astype(np.int32)
        mask = rng.integers(0, 1 << 10, wl.R).astype(np.uint64)
        a = host.step_logits(step, tok, mask)
        b = to_host_logits(dev.step_logits(step, torch.from_numpy(tok).cuda(),
                                           torch.from_numpy(mask.view(np.int64)).cuda()))
        assert a.dtype == b.dtype and np.array_equal(a, b)


# ------------------------------------------------------------------------------------------ row scan
def _rows(kind, R, V, rng):
    if kind == "normal":
        return rng.normal(0, 3, (R, V)).astype(np.float32)
    if kind == "ascending":
        return np.tile(np.linspace(-8, 8, V, dtype=np.float32), (R, 1))
    if kind == "descending":
        return np.tile(np.linspace(8, -8, V, dtype=np.float32), (R, 1))
    if kind == "constant":
        return np.full((R, V), 1.25, np.float32)
    if kind == "quantised":
        return np.round(rng.normal(0, 2, (R, V))).astype(np.float32) + np.float32(0.0)
    if kind == "holes":
        x = rng.normal(0, 3, (R, V)).astype(np.float32)
        x[rng.random((R, V)) < 0.3] = -np.inf
        x[0, :] = -np.inf
        if V > 3:
            x[0, 3] = 0.5
        return x
    if kind == "signed_zero":
        x = np.zeros((R, V), np.float32)
        x[:, ::2] = -0.0
        return x
    raise ValueError(kind)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("kind", ["normal", "ascending", "descending", "constant", "quantised", "holes", "signed_zero"])
@pytest.mark.parametrize("V,n_top", [(1, 3), (7, 7), (1000, 7), (4099, 22), (32000, 12), (64000, 22), (20011, 66),
                                      (24576, 12), (150000, 22), (262144, 7), (1000003, 22), (1048576, 12)])
def test_row_scan_matches_oracle(dba, dtype, kind, V, n_top):
    from synth_inputs.logits import to_bf16_bits
    rng = np.random.default_rng(V + n_top)
    R = 3
    x = _rows(kind, R, V, rng)
    if dtype == "bf16":
        bits = to_bf16_bits(np.where(np.isinf(x), np.float32(0), x))
        bits[np.isinf(x)] = 0xFF80
        x_np, x_dev = bits, torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    else:
        x_np, x_dev = x, torch.from_numpy(x).cuda()
    lse, val, idx = dba.row_scan(x_dev, n_top)
    lse, val, idx = lse.cpu().numpy(), val.cpu().numpy(), idx.cpu().numpy()
    for r in range(R):
        want = O.row_lse(x_np[r])
        if np.isinf(want):
            assert np.isinf(lse[r]) and lse[r] < 0
        else:
            assert abs(float(lse[r]) - want) <= 1e-5, (r, lse[r], want)
        wv, wi = O.row_top(x_np[r], n_top)
        assert np.array_equal(idx[r], wi), (r, idx[r], wi)
        assert np.array_equal(val[r], wv)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_repeated_scans_of_the_same_rows_agree(dba, dtype):
    """The streaming scan's warps hand work to one another through barriers; a mistake in that hand-over shows
    as a result that changes from launch to launch.  30 launches over the same 3000 benchmark-shaped rows must
    give the same bits, and sampled rows must match the oracle."""
    from synth_inputs.logits import to_bf16_bits
    R, V, n_top = 3000, 64000, 22
    g = torch.Generator(device="cuda"); g.manual_seed(5)
    mu = -1.1 * torch.log(torch.randperm(V, device="cuda", generator=g).float() + 1)
    x = torch.randn(R, V, device="cuda", generator=g) + mu
    if dtype == "bf16":
        x = x.to(torch.bfloat16)
    first = None
    for it in range(30):
        lse, val, idx = dba.row_scan(x, n_top)
        got = (lse.clone(), val.clone(), idx.clone())
        if first is None:
            first = got
        else:
            for a, b, what in zip(got, first, ("lse", "values", "indices")):
                assert torch.equal(a, b), f"launch {it}: {what} differ from the first launch in {int((a != b).any(-1).sum() if a.dim() > 1 else (a != b).sum())} rows"
    lse, val, idx = (t.cpu().numpy() for t in first)
    for r in (0, 1, 1499, 2998, 2999):
        row = x[r].float().cpu().numpy()
        row_in = to_bf16_bits(row) if dtype == "bf16" else row
        wv, wi = O.row_top(row_in, n_top)
        assert np.array_equal(idx[r], wi) and np.array_equal(val[r], wv)
        assert abs(float(lse[r]) - O.row_lse(row_in)) <= 1e-5


# ------------------------------------------------------------------------------------------ fused projection
@pytest.mark.parametrize("R,V,D,n_top", [(5, 1000, 64, 7), (128, 4096, 256, 22), (300, 20011, 128, 22), (20, 64000, 1024, 22),
                                          (131, 5000, 72, 32), (260, 33000, 64, 12)])
def test_fused_projection_and_row_scan_match_the_oracle(dba, R, V, D, n_top):
    """Section 2's output projection on the tensor cores with the row scan in its epilogue, against the oracle's
    double-precision inner products.  The kernel accumulates bf16 products in fp32, so a logit may differ from
    the oracle's by the rounding of D additions: normalisers within 1e-4, listed values within 1e-4 rank by rank,
    and where the listed word differs from the oracle's it must be one whose exact logit ties with the oracle's
    choice within that bound."""
    from synth_inputs.logits import to_bf16_bits
    rng = np.random.default_rng(R + V + D)
    h = rng.normal(0, 1, (R, D)).astype(np.float32)
    mu = (-1.1 * np.log(rng.permutation(V) + 1.0)).astype(np.float32)          # Zipf-shaped word offsets
    e = rng.normal(0, 1, (V, D)).astype(np.float32) / np.float32(np.sqrt(D))
    e[:, 0] = mu; h[:, 0] = 1.0                                                  # logits = offset + noise
    hb, eb = to_bf16_bits(h), to_bf16_bits(e)
    X = O.project(hb, eb)
    hd = torch.from_numpy(hb.view(np.int16)).cuda().view(torch.bfloat16)
    ed = torch.from_numpy(eb.view(np.int16)).cuda().view(torch.bfloat16)
    lse, val, idx = dba.project_scan(hd, ed, n_top)
    lse, val, idx = lse.cpu().numpy(), val.cpu().numpy(), idx.cpu().numpy()
    tol = 1e-4
    for r in range(R):
        assert abs(float(lse[r]) - O.row_lse(X[r])) <= tol, (r, lse[r], O.row_lse(X[r]))
        wv, wi = O.row_top(X[r], n_top)
        assert np.abs(val[r] - wv).max() <= tol, (r, val[r], wv)
        assert ((idx[r] >= 0) & (idx[r] < V)).all() and len(set(idx[r].tolist())) == n_top
        assert np.abs(X[r][idx[r]] - wv).max() <= tol, (r, idx[r], wi)


def _bf16_pair(h, e):
    from synth_inputs.logits import to_bf16_bits
    hb, eb = to_bf16_bits(h), to_bf16_bits(e)
    hd = torch.from_numpy(hb.view(np.int16)).cuda().view(torch.bfloat16)
    ed = torch.from_numpy(eb.view(np.int16)).cuda().view(torch.bfloat16)
    return hb, eb, hd, ed


def test_fused_projection_long_runs_of_tiles(dba):
    """Many row blocks and few CTAs per row block: a pair of CTAs works through a whole row block's vocabulary
    (253 tiles), so the columns it keeps, counted from its first one, use all 16 bits.  Sampled rows against the
    oracle (first and last rows, and rows on both sides of the boundaries between CTAs and between row blocks)."""
    R, V, D, n_top = 19200, 64768, 16, 8
    rng = np.random.default_rng(11)
    h = rng.normal(0, 1, (R, D)).astype(np.float32)
    e = rng.normal(0, 1, (V, D)).astype(np.float32)
    e[-3:, :] = 3.0 * np.sign(h[R - 1])[None, :]              # the last row's best words are the vocabulary's last
    hb, eb, hd, ed = _bf16_pair(h, e)
    lse, val, idx = dba.project_scan(hd, ed, n_top)
    lse, val, idx = lse.cpu().numpy(), val.cpu().numpy(), idx.cpu().numpy()
    assert not np.isnan(lse).any()
    rows = [0, 1, 127, 128, 255, 256, 9999, R - 129, R - 128, R - 1]
    X = O.project(hb[rows], eb)
    for i, r in enumerate(rows):
        assert abs(float(lse[r]) - O.row_lse(X[i])) <= 1e-4
        wv, wi = O.row_top(X[i], n_top)
        assert np.abs(val[r] - wv).max() <= 1e-4
        assert np.abs(X[i][idx[r]] - wv).max() <= 1e-4 and len(set(idx[r].tolist())) == n_top
    assert set(idx[R - 1][:3].tolist()) == {V - 3, V - 2, V - 1}


def test_fused_projection_ties_across_the_vocabulary(dba):
    """Two hundred words spread over the vocabulary share a row's largest logit exactly: each thread meets only
    a few of them, the merge of the row's pieces meets them all (more than its short list holds, and more
    entries in all than it keeps in shared memory) and must list the lowest-numbered ones."""
    R, V, D, n_top = 3, 64000, 8, 8
    rng = np.random.default_rng(12)
    h = np.zeros((R, D), np.float32); h[:, 0] = 1.0           # logits = embed[:, 0], exactly
    e = np.zeros((V, D), np.float32)
    e[:, 0] = np.clip(np.round(rng.normal(0, 1, V) * 8) / 16, -1.5, 1.5)      # (bf16-exact values below 2)
    ties = 300 * np.arange(200) + 7
    e[ties, 0] = 2.0
    hb, eb, hd, ed = _bf16_pair(h, e)
    lse, val, idx = dba.project_scan(hd, ed, n_top)
    lse, val, idx = lse.cpu().numpy(), val.cpu().numpy(), idx.cpu().numpy()
    X = O.project(hb, eb)
    for r in range(R):
        wv, wi = O.row_top(X[r], n_top)
        assert np.array_equal(wi, ties[:n_top]) and np.array_equal(idx[r], wi) and np.array_equal(val[r], wv)
        assert abs(float(lse[r]) - O.row_lse(X[r])) <= 1e-4


def test_fused_projection_reports_a_plateau_it_cannot_hold(dba):
    """Every logit of a row equal: a thread's list cannot hold the ties at the n_top-th largest value, and the
    call reports it the documented way (every row NaN with an empty list) instead of listing a wrong choice."""
    R, V, D, n_top = 4, 1000, 8, 5
    h = np.zeros((R, D), np.float32)
    e = np.ones((V, D), np.float32)
    _, _, hd, ed = _bf16_pair(h, e)
    lse, val, idx = dba.project_scan(hd, ed, n_top)
    assert torch.isnan(lse).all() and (idx == -1).all() and torch.isinf(val).all()


def test_fused_step_follows_the_oracle_on_the_projected_logits(dba):
    """dba_step_fused against the oracle stepping on the exactly projected logits.  Sentences must match field by
    field; where one first differs the two beams must hold the same scores rank by rank within the accumulated
    tolerance of the fp32 accumulation (a near-tie decided the other way), and it leaves the comparison."""
    from synth_inputs.logits import to_bf16_bits
    from tests.parity import BEAM_FIELDS
    B, k, V, D, steps = 6, 5, 3000, 64, 16
    cons = [[[5, 6]], [[7], [8, 9]], [], [[10]], [[11, 12, 13]], [[14], [15]]]
    rng = np.random.default_rng(42)
    mu = (-1.1 * np.log(rng.permutation(V) + 1.0)).astype(np.float32)
    e = rng.normal(0, 1, (V, D)).astype(np.float32) / np.float32(np.sqrt(D))
    e[:, 0] = mu
    e[:, 1] = 0.0; e[2, 1] = 1.0                     # the end token's logit follows hidden[:, 1]
    for c in cons:                                   # constraint tokens are among the likeliest words
        for ph in c:
            for w in ph:
                e[w, 0] = 1.5
    eb = to_bf16_bits(e)
    ed = torch.from_numpy(eb.view(np.int16)).cuda().view(torch.bfloat16)
    st = dba.DbaStepper(B, k, V, steps, constraints=cons, dtype=dba.F32, flags=dba.FLAG_FUSED_PROJECTION)
    orc = O.Batch(k, V, steps, cons, threads=1)
    alive = [True] * B
    compared = 0
    for t in range(steps):
        h = rng.normal(0, 1, (B * k, D)).astype(np.float32)
        h[:, 0] = 1.0
        h[:, 1] = -6.0 if t < 8 else 12.0            # the end token becomes by far the likeliest in the second half
        hb = to_bf16_bits(h)
        X = O.project(hb, eb)
        orc.step(X)
        out = st.step_fused(torch.from_numpy(hb.view(np.int16)).cuda().view(torch.bfloat16), ed)
        g, ob = gpu_beam(out), orc.beam()
        tol = 1e-4 * (t + 1)
        for b in range(B):
            if not alive[b]:
                continue
            sl = slice(b * k, (b + 1) * k)
            fin = np.isfinite(ob["score"][sl])
            assert (np.isfinite(g["score"][sl]) == fin).all()
            assert np.abs(g["score"][sl][fin] - ob["score"][sl][fin]).max(initial=0) <= tol, (t, b)
            if all((g[f][sl] == ob[f][sl]).all() for f in BEAM_FIELDS):
                compared += 1
            else:
                alive[b] = False
        if t > 0 and not any(alive):
            break
        # both sides go on from the oracle's beam only while they agree; a sentence that left is not looked at again
    assert sum(alive) >= B - 2 and compared >= (B - 2) * steps
    assert st.counters()[1] == 0
    tokens, length, score, flags = st.finalize()
    done = [d for _, _, d in orc.finalize()]
    for b in range(B):
        if alive[b]:
            assert bool(flags[b] & 1) == done[b]
    assert sum(done) >= 3
    st.close()


# ------------------------------------------------------------------------------------------ whole step
def test_step_parity_tiny(dba):
    wl = make_workload("tiny")
    st = _stepper(dba, wl)
    orc, worst = lockstep(wl, st)
    assert_finalize_equal(st, orc)


def test_step_parity_phrasal(dba):
    wl = make_workload("phrasal")
    st = _stepper(dba, wl)
    orc, worst = lockstep(wl, st)
    assert_finalize_equal(st, orc)


def test_step_parity_ragged(dba):
    from synth_inputs.gpu import GpuLogitStream
    wl = make_workload("ragged")
    st = _stepper(dba, wl)
    orc, worst = lockstep(wl, st, gpu_gen=GpuLogitStream(wl))
    assert_finalize_equal(st, orc)


@pytest.mark.parametrize("C", [1, 5, 10, 20, 50])
def test_step_parity_scaling(dba, C):
    from synth_inputs.gpu import GpuLogitStream
    wl = make_workload("scaling", C=C)
    st = _stepper(dba, wl)
    orc, worst = lockstep(wl, st, gpu_gen=GpuLogitStream(wl))        # all 100 steps
    assert_finalize_equal(st, orc)


def test_step_parity_serving_sampled_sentences(dba):
    """Eight of the 256 sentences of the serving workload, all 120 steps, as a batch of their own."""
    from synth_inputs.gpu import GpuLogitStream
    wl = make_workload("serving").subset([0, 31, 64, 100, 129, 177, 200, 255])
    st = _stepper(dba, wl)
    orc, worst = lockstep(wl, st, gpu_gen=GpuLogitStream(wl))
    assert_finalize_equal(st, orc)
    assert sum(done for _, _, done in orc.finalize()) >= 6        # the stream lets most sentences finish


def test_serving_full_size_free_run_against_sampled_oracle(dba):
    """The launch configuration the benchmark times (B=256, k=20, V=64000, bf16), free-running."""
    from synth_inputs.gpu import GpuLogitStream
    from tests.parity import free_run
    wl = make_workload("serving")
    st = _stepper(dba, wl)
    steps = wl.steps           # all 120: finished rows, the shrinking list of open rows and the last waves included
    sample = [3, 40, 77, 111, 140, 201, 230, 254]
    compared, left = free_run(wl, st, sample, steps, GpuLogitStream(wl))
    assert len(left) <= 1 and compared >= (len(sample) - 1) * steps, left     # a departure is a verified near-tie
    assert st.counters()[0] == 0
    tokens, length, score, flags = st.finalize()
    assert (flags & 1).sum() >= 200                       # the stream lets most sentences finish


@pytest.mark.parametrize("name,kw", [("tiny", {}), ("phrasal", {}), ("ragged", {}), ("scaling", dict(C=1)),
                                     ("scaling", dict(C=50))])
def test_small_workloads_free_running_on_the_gpus_own_normalisers(dba, name, kw):
    """The four small configurations, every sentence, every step, with the library ranking by the normalisers it
    computes itself (the lock-step tests hand it the oracle's)."""
    from synth_inputs.gpu import GpuLogitStream
    from tests.parity import free_run
    wl = make_workload(name, **kw)
    st = _stepper(dba, wl)
    compared, left = free_run(wl, st, list(range(wl.B)), wl.steps, GpuLogitStream(wl))
    assert len(left) <= max(1, wl.B // 16) and compared >= (wl.B - len(left) - 1) * wl.steps, left
    st.close()


@pytest.mark.parametrize("dtype,B,V", [("f32", 210, 262144), ("bf16", 212, 524288)])
def test_logit_matrices_beyond_four_gigabytes(dba, dtype, B, V):
    """Rows of 1 MiB, more than 4096 of them: the byte offsets of the last sentences' rows do not fit 32 bits
    (f32: 4.4 GB; bf16: 4.4 GB as well, 2.2e9 elements, more than 2^31).  Free-running; the oracle follows the first, a middle and the last sentences."""
    from synth_inputs.gpu import GpuLogitStream
    from tests.parity import free_run
    wl = make_workload("scaling", C=5, B=B, V=V, dtype=dtype)
    assert wl.R * wl.V * (4 if dtype == "f32" else 2) > 2**32
    st = _stepper(dba, wl)
    steps = 5
    sample = [0, B // 2, B - 5, B - 1]
    compared, left = free_run(wl, st, sample, steps, GpuLogitStream(wl))
    assert len(left) <= 1 and compared >= 3 * steps


# ------------------------------------------------------------------------------------------ edge cases
def _custom(name, B, k, V, steps, constraints, dtype="f32", zipf=True):
    from synth_inputs.configs import Workload
    return Workload(name=name, cfg_id=9, B=B, k=k, V=V, steps=steps, dtype=dtype, zipf=zipf, boost=True,
                    constraints=constraints, seed=0, sent_ids=np.arange(B, dtype=np.int64))


EDGE = {
    "beam_of_one":            dict(B=2, k=1, V=300, steps=12, constraints=[[[5], [6, 7]], []]),
    "no_constraints":         dict(B=3, k=4, V=517, steps=10, constraints=[[], [], []]),
    "more_constraints_than_beam": dict(B=2, k=3, V=400, steps=16, constraints=[[[w] for w in range(10, 20)], [[30, 31, 32, 33], [40], [41]]]),
    "sixty_four_constraints": dict(B=1, k=4, V=700, steps=20, constraints=[[[w] for w in range(100, 164)]]),
    "sixty_four_in_phrases":  dict(B=1, k=6, V=700, steps=20, constraints=[[list(range(100 + 4 * i, 104 + 4 * i)) for i in range(16)]]),
    "odd_vocab_f32":          dict(B=2, k=5, V=1003, steps=10, constraints=[[[5, 6]], [[7]]]),
    "odd_vocab_bf16":         dict(B=2, k=5, V=1001, steps=10, constraints=[[[5, 6]], [[7]]], dtype="bf16"),
    "duplicate_tokens":       dict(B=1, k=5, V=200, steps=12, constraints=[[[9], [9], [9, 10], [10, 9, 11]]]),
    "self_overlapping_phrase": dict(B=1, k=6, V=120, steps=14, constraints=[[[8, 8, 9], [8, 9]]]),
    "big_beam":               dict(B=2, k=64, V=2048, steps=8, constraints=[[[5, 6], [7]], [[9]]], dtype="bf16"),
    "plain_normal_rows":      dict(B=2, k=7, V=900, steps=10, constraints=[[[5]], [[6, 7, 8]]], zipf=False),
    # k + 2 = 32 entries per row is the widest list the candidate kernel merges in registers; 33 takes the other way
    "beam_of_thirty":         dict(B=2, k=30, V=30000, steps=8, constraints=[[[5, 6], [7]], [[9], [10], [11, 12, 13]]], dtype="bf16"),
    "beam_of_thirty_one":     dict(B=2, k=31, V=30000, steps=8, constraints=[[[5, 6], [7]], [[9], [10], [11, 12, 13]]], dtype="bf16"),
    "widest_beam_long_rows":  dict(B=2, k=64, V=64000, steps=6, constraints=[[[5, 6], [7]], [[9]]], dtype="bf16"),
    # fewer words than beam slots: rows shorter than the k+2 entries the scan keeps, beams that cannot fill
    "vocab_smaller_than_beam": dict(B=2, k=8, V=8, steps=8, constraints=[[[3]], [[4, 5]]]),
    "vocab_smaller_than_beam_bf16": dict(B=2, k=12, V=9, steps=8, constraints=[[[3]], [[4, 5], [6]]], dtype="bf16"),
    # more sentences than the GPU holds blocks of the candidate kernel at once; constraint sets of 0-3 phrases
    "many_sentences":         dict(B=1200, k=3, V=260, steps=6,
                                   constraints=[[[10 + (i + j) % 50 + q for q in range(1 + (i + j) % 2)] for j in range(i % 4)]
                                                for i in range(1200)]),
    "eighty_thousand_rows":   dict(B=4096, k=20, V=256, steps=3, constraints=[[[10 + i % 100]] * (i % 3) for i in range(4096)]),
    # steps go on long after every hypothesis has ended (no open row is left to scan)
    "steps_after_the_end":    dict(B=1, k=3, V=100, steps=40, constraints=[[[5]]]),
    "steps_after_one_sentence_ended": dict(B=2, k=3, V=100, steps=40, constraints=[[[5]], [[6, 7]]]),
    # the widest beam with as many one-word constraints as its candidates leave room for in shared memory
    "widest_beam_forty_constraints": dict(B=1, k=64, V=3000, steps=10, constraints=[[[w] for w in range(100, 140)]]),
    "beam_of_forty_most_constraints": dict(B=1, k=40, V=3000, steps=10, constraints=[[[w] for w in range(100, 164)]]),
}


@pytest.mark.parametrize("case", sorted(EDGE))
def test_step_parity_edge_cases(dba, case):
    p = dict(EDGE[case])
    wl = _custom(case, **p)
    st = _stepper(dba, wl)
    orc, worst = lockstep(wl, st)
    assert_finalize_equal(st, orc)


@pytest.mark.parametrize("dtype,V,pad", [("f32", 4096, 64), ("bf16", 24576, 8), ("f32", 1003, 5), ("bf16", 4096, 3)])
def test_rows_further_apart_than_their_length(dba, dtype, V, pad):
    """row_stride_elems > V, with the gaps holding values above every logit: aligned strides take the streaming
    scan, the others the plain one; neither the scan nor the progress-token look-ups may read a gap."""
    wl = _custom("padded", B=3, k=5, V=V, steps=10, constraints=[[[5, 6]], [[7], [8, 9, 10]], []], dtype=dtype)
    st = _stepper(dba, wl)
    orc, worst = lockstep(wl, st, row_pad=pad)
    assert_finalize_equal(st, orc)


def test_handles_of_different_shapes_alive_together(dba):
    """A handle that needs nearly all the shared memory of a block keeps working after a small one was made
    (what a launch may ask for is a property of the kernel, shared by all handles), steps interleaved."""
    big = _custom("big", **EDGE["widest_beam_forty_constraints"])
    small = _custom("small", **EDGE["beam_of_one"])
    st_big = _stepper(dba, big)
    st_small = _stepper(dba, small)                 # initialised second: must not lower the first one's limit
    orcs = {n: O.Batch(w.k, w.V, w.steps, w.constraints, threads=1) for n, w in (("big", big), ("small", small))}
    gens = {"big": LogitStream(big), "small": LogitStream(small)}
    for t in range(8):
        for n, w, st in (("big", big, st_big), ("small", small, st_small)):
            ob = orcs[n].beam()
            x = gens[n].step_logits(t, ob["token"], ob["met_mask"])
            lse_o = orcs[n].step(x)
            out = st.step(to_device_logits(x, w), row_lse_in=torch.from_numpy(lse_o).cuda())
            assert_beam_equal(gpu_beam(out), orcs[n].beam(), f"{n} step {t}")


def test_steps_on_a_stream_of_the_callers(dba):
    """Everything the library enqueues goes to the stream given at initialisation (here not the default one):
    inputs are made ready before, outputs read after a synchronisation of that stream alone."""
    wl = make_workload("ragged", B=5, V=4096, steps=20)
    s = torch.cuda.Stream()
    st = dba.DbaStepper(wl.B, wl.k, wl.V, wl.steps, constraints=wl.constraints, dtype=dba.BF16, stream=s)
    orc = O.Batch(wl.k, wl.V, wl.steps, wl.constraints, threads=1)
    gen = LogitStream(wl)
    for t in range(wl.steps):
        ob = orc.beam()
        x = gen.step_logits(t, ob["token"], ob["met_mask"])
        lse_o = orc.step(x)
        x_dev, lse_dev = to_device_logits(x, wl), torch.from_numpy(lse_o).cuda()
        torch.cuda.current_stream().synchronize()
        out = st.step(x_dev, row_lse_in=lse_dev)
        s.synchronize()
        assert_beam_equal(gpu_beam(out), orc.beam(), f"step {t}")
    assert_finalize_equal(st, orc)


def test_special_symbols_elsewhere_in_the_vocabulary(dba):
    """pad, bos and eos are configuration, not 0, 1, 2: here they sit at the end and in the middle of the
    vocabulary (the stream's columns 0, 1, 2 are moved there) and 0, 1, 2 are ordinary, constrained words."""
    V, k, B, steps = 1200, 6, 3, 16
    pad, bos, eos = 1199, 640, 77
    wl = _custom("ids", B=B, k=k, V=V, steps=steps, constraints=[[[5, 6]], [[0], [2, 1]], []], dtype="bf16")
    perm = np.arange(V); perm[[0, pad]] = [pad, 0]; perm[[1, bos]] = [bos, 1]; perm[[2, eos]] = [eos, 2]
    st = dba.DbaStepper(B, k, V, steps, constraints=wl.constraints, dtype=dba.BF16, pad=pad, bos=bos, eos=eos)
    orc = O.Batch(k, V, steps, wl.constraints, pad=pad, bos=bos, eos=eos, threads=1)
    gen = LogitStream(wl)
    for t in range(steps):
        ob = orc.beam()
        x = np.ascontiguousarray(gen.step_logits(t, ob["token"], ob["met_mask"])[:, perm])
        lse_o = orc.step(x)
        out = st.step(to_device_logits(x, wl), row_lse_in=torch.from_numpy(lse_o).cuda())
        assert_beam_equal(gpu_beam(out), orc.beam(), f"step {t}")
    tokens, length, score, flags = st.finalize()
    want = orc.finalize()
    assert all(done for _, _, done in want)
    for b, (toks, sc, done) in enumerate(want):
        assert tokens[b, :length[b]].tolist() == toks and toks[-1] == eos and (tokens[b, length[b]:] == pad).all()
        assert score[b] == np.float32(sc) and flags[b] & 1


@pytest.mark.parametrize("name,kw,theta", [("tiny", {}, 3.0), ("ragged", dict(B=6, V=4096, steps=40), 20.0),
                                           ("ragged", dict(B=6, V=4096, steps=40), 2.0),
                                           ("serving", dict(B=3, V=8192, steps=60), 5.0)])
def test_threshold_pruning_and_stop_bits_match_the_oracle(dba, name, kw, theta):
    wl = make_workload(name, **kw)
    st = dba.DbaStepper(wl.B, wl.k, wl.V, wl.steps, constraints=wl.constraints,
                        dtype=dba.BF16 if wl.dtype == "bf16" else dba.F32, prune=theta)
    orc, worst = lockstep(wl, st, prune=theta)
    assert_finalize_equal(st, orc)
    flags = orc.stop_flags()
    assert name == "tiny" or (flags & 2).any()      # the stream does complete hypotheses: the pruning had work to do
    st.close()


@pytest.mark.parametrize("name,kw,theta", [("ragged", dict(B=6, V=4096, steps=40), 2.0), ("ragged", dict(B=6, V=4096, steps=40), 0.5),
                                           ("serving", dict(B=3, V=8192, steps=60), 1.0)])
def test_pruning_by_normalised_completed_scores_matches_the_oracle(dba, name, kw, theta):
    """Section 4's other reading: completed hypotheses enter the threshold comparison with score / length.  The
    hypotheses removed are then not always the tail of the beam."""
    wl = make_workload(name, **kw)
    st = dba.DbaStepper(wl.B, wl.k, wl.V, wl.steps, constraints=wl.constraints,
                        dtype=dba.BF16 if wl.dtype == "bf16" else dba.F32, prune=theta, flags=dba.FLAG_PRUNE_NORMALISED)
    orc, worst = lockstep(wl, st, prune=theta, flags=dba.FLAG_PRUNE_NORMALISED)
    assert_finalize_equal(st, orc)
    assert (orc.stop_flags() & 2).any()
    st.close()


@pytest.mark.parametrize("flags", [1, 2, 3])
def test_flags_adjust_off_and_length_norm(dba, flags):
    wl = make_workload("ragged", B=6, V=3000, steps=50)
    st = _stepper(dba, wl, flags=flags)
    orc, worst = lockstep(wl, st, flags=flags)
    assert_finalize_equal(st, orc)


def test_rows_with_minus_inf_and_quantised_logits(dba):
    """Heavy ties (a few distinct values per row) and -inf holes, for both dtypes."""
    rng = np.random.default_rng(5)
    for dtype in ("f32", "bf16"):
        wl = _custom("holes", 3, 5, 260, 9, [[[5, 6], [7]], [[8]], []], dtype=dtype)
        st = _stepper(dba, wl)
        orc = O.Batch(wl.k, wl.V, wl.steps, wl.constraints)
        for t in range(wl.steps):
            x = np.round(rng.normal(0, 1.5, (wl.R, wl.V))).astype(np.float32) + np.float32(0.0)
            x[rng.random(x.shape) < 0.4] = -np.inf
            x[:, 2] = -30.0 if t < 5 else 3.0
            if dtype == "bf16":
                x_np = (x.view(np.uint32) >> 16).astype(np.uint16)       # small integers are exact in bf16
            else:
                x_np = x
            lse_o = orc.step(x_np)
            out = st.step(to_device_logits(x_np, wl), row_lse_in=torch.from_numpy(lse_o).cuda())
            assert_beam_equal(gpu_beam(out), orc.beam(), f"holes {dtype} step {t}")
        assert_finalize_equal(st, orc)


def test_scores_that_round_together_across_the_row_cut(dba):
    """Logits one ulp apart collapse onto a few fp32 scores; the cells kept must then be the lowest token ids
    among the equal scores, also beyond the k+2 entries the row scan keeps."""
    k, V = 4, 96
    wl = _custom("collapse", 1, k, V, 3, [[]])
    st = _stepper(dba, wl)
    orc = O.Batch(k, V, 3, wl.constraints)
    for t in range(3):
        base = np.float32(1.0)
        ulps = np.arange(V, dtype=np.int32)[::-1].copy()             # higher logits at lower... reversed below
        x = (base.view(np.int32) + ulps).view(np.float32)           # descending by index, 1 ulp steps
        x = x[::-1].copy()                                           # ascending: best raw logits have the HIGHEST ids
        x = np.tile(x, (k, 1)).astype(np.float32)
        x[:, 2] = -50.0
        lse_o = orc.step(x)
        out = st.step(torch.from_numpy(x).cuda(), row_lse_in=torch.from_numpy(lse_o).cuda())
        assert_beam_equal(gpu_beam(out), orc.beam(), f"collapse step {t}")
    sc = orc.beam()["score"]
    assert len(np.unique(sc)) < k                                   # the case really had equal scores


def test_step_parity_on_rows_of_more_than_eight_segments(dba):
    """Rows longer than eight full segments (Transformer-sized vocabularies in fp32): up to 24 segments per row."""
    wl = _custom("long_rows", B=2, k=4, V=150000, steps=5, constraints=[[[5, 6], [70000]], [[149999]]])
    st = _stepper(dba, wl)
    orc, worst = lockstep(wl, st, threads=2)
    assert_finalize_equal(st, orc)
    assert st.counters()[0] == 0
    st.close()


@pytest.mark.parametrize("B,k", [(8, 20), (30, 20), (6, 60)])
def test_the_row_scan_needs_no_second_pass_on_benchmark_shaped_rows(dba, B, k):
    """A performance guard: the scan's selection bound must be tight enough on Zipf-shaped bf16 rows that no
    row segment is ranked again from global memory (that pass costs about as much as scanning 150 rows), also
    for the short segments a small batch gets (few warps per segment, hence few reports) and for a wide beam
    (three times as many entries wanted per segment)."""
    from synth_inputs.gpu import GpuLogitStream
    wl = make_workload("serving", B=B, k=k, steps=12)
    st = _stepper(dba, wl)
    gen = GpuLogitStream(wl)
    tok = torch.zeros(wl.R, dtype=torch.int32, device="cuda"); tok[::wl.k] = 1
    mask = torch.zeros(wl.R, dtype=torch.int64, device="cuda")
    for t in range(wl.steps):
        out = st.step(gen.step_logits(t, tok, mask))
        tok, mask = out["token"].clone(), out["met_mask"].clone()
    assert st.counters()[0] == 0
    st.close()


def test_long_runs_of_equal_logits_take_the_second_pass_and_stay_exact(dba):
    wl = _custom("flat", B=2, k=20, V=64000, steps=2, dtype="bf16", constraints=[[[5, 6]], [[7]]])
    st = _stepper(dba, wl)
    orc = O.Batch(wl.k, wl.V, wl.steps, wl.constraints)
    for t in range(wl.steps):
        x = np.full((wl.R, wl.V), 0x3F80, np.uint16)          # every logit 1.0: everything ties at the bound
        lse_o = orc.step(x)
        out = st.step(to_device_logits(x, wl), row_lse_in=torch.from_numpy(lse_o).cuda())
        assert_beam_equal(gpu_beam(out), orc.beam(), f"flat step {t}")
    assert st.counters()[0] > 0
    st.close()


def test_step_host_equals_step_and_reset_replays(dba):
    wl = make_workload("ragged", B=4, V=2000, steps=12)
    gen = LogitStream(wl)
    a = _stepper(dba, wl)
    b = _stepper(dba, wl, flags=dba.FLAG_HOST_STAGING)
    host_out = b.new_outputs(host=True)
    tok = np.zeros(wl.R, np.int32); tok[::wl.k] = 1
    mask = np.zeros(wl.R, np.uint64)
    trace = []
    for t in range(wl.steps):
        x = gen.step_logits(t, tok, mask)
        ga = gpu_beam(a.step(to_device_logits(x, wl)))
        xh = torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).pin_memory()
        if t % 2:                      # host rows further apart than their length, the gaps above every logit
            wide = torch.full((wl.R, wl.V + 24), 3.0e4, dtype=torch.bfloat16).pin_memory()
            wide[:, :wl.V] = xh
            xh = wide[:, :wl.V]
        b.step_host(xh, host_out)
        gb = {f: host_out[f].numpy().copy() for f in host_out}
        gb["met_mask"] = gb["met_mask"].view(np.uint64)
        assert_beam_equal(gb, ga, f"host step {t}", fields=("backptr", "token", "bank", "met_mask", "active", "score", "row_lse"))
        trace.append((x, ga))
        tok, mask = ga["token"], ga["met_mask"]
    fa = a.finalize()
    a.reset()
    for t, (x, want) in enumerate(trace):
        assert_beam_equal(gpu_beam(a.step(to_device_logits(x, wl))), want, f"replay step {t}",
                          fields=("backptr", "token", "bank", "met_mask", "active", "score", "row_lse"))
    for u, v in zip(fa, a.finalize()):
        assert np.array_equal(u, v)
    with pytest.raises(dba.DbaError) as e:
        a.step(to_device_logits(trace[0][0], wl))
    assert e.value.code == 3                                        # DBA_ERR_STATE: past max_steps


def test_a_device_wait_that_runs_out_is_reported_and_the_device_stays_usable(dba):
    """Failure detection without a fault: the row scan's waits are bounded.  The testing aid makes every warp
    announce its first copy without issuing it and shortens the limit to about a millisecond: the waits run out,
    the kernel records that and returns, dba_finalize reports DBA_ERR_TIMEOUT.  A fresh handle on the same
    device and stream then steps in parity with the oracle.  The stand-alone scan reports the same failure in
    its results (NaN normalisers, empty lists)."""
    wl = make_workload("ragged", B=4, V=8192, steps=6)
    gen = LogitStream(wl)
    tok = np.zeros(wl.R, np.int32); tok[::wl.k] = 1
    x = to_device_logits(gen.step_logits(0, tok, np.zeros(wl.R, np.uint64)), wl)
    st = _stepper(dba, wl)
    st.test_hook(wait_clocks=2_000_000, drop_item=0)
    st.step(x)                                   # enqueued; the failure is on the device
    with pytest.raises(dba.DbaError) as e:
        st.finalize()
    assert e.value.code == 5                     # DBA_ERR_TIMEOUT
    st.close()
    L = dba.lib()
    try:
        assert L.dba_test_hook(None, 2_000_000, 0) == 0
        lse, val, idx = dba.row_scan(x, 5)
        assert torch.isnan(lse).all() and (idx == -1).all() and torch.isinf(val).all()
    finally:
        assert L.dba_test_hook(None, 0, -1) == 0
    lse, val, idx = dba.row_scan(x, 5)
    assert torch.isfinite(lse).all() and (idx >= 0).all()
    st2 = _stepper(dba, wl)
    orc, worst = lockstep(wl, st2)
    assert_finalize_equal(st2, orc)
    st2.close()


def test_a_wait_that_runs_out_in_the_fused_projection_is_reported(dba):
    """The same for the projection kernel, whose pairs of CTAs wait on each other's copies: the first CTA of every
    pair announces its first slice of the operands without fetching it, the limit is about a millisecond, every
    role of both CTAs gives up at its next wait and the pair leaves together.  The stand-alone call reports NaN
    rows; the fused step's dba_finalize reports DBA_ERR_TIMEOUT; afterwards the same calls work."""
    R, V, D, n_top = 300, 5000, 128, 7
    rng = np.random.default_rng(5)
    h = rng.normal(0, 1, (R, D)).astype(np.float32)
    e = rng.normal(0, 1, (V, D)).astype(np.float32)
    _, _, hd, ed = _bf16_pair(h, e)
    L = dba.lib()
    try:
        assert L.dba_test_hook(None, 2_000_000, 0) == 0
        lse, val, idx = dba.project_scan(hd, ed, n_top)
        assert torch.isnan(lse).all() and (idx == -1).all() and torch.isinf(val).all()
    finally:
        assert L.dba_test_hook(None, 0, -1) == 0
    lse, val, idx = dba.project_scan(hd, ed, n_top)
    assert torch.isfinite(lse).all() and (idx >= 0).all()
    B, k = 3, 4
    st = dba.DbaStepper(B, k, V, 4, constraints=[[[5]], [], [[6, 7]]], dtype=dba.F32, flags=dba.FLAG_FUSED_PROJECTION)
    st.test_hook(wait_clocks=2_000_000, drop_item=0)
    st.step_fused(hd[:B * k].contiguous(), ed)
    with pytest.raises(dba.DbaError) as err:
        st.finalize()
    assert err.value.code == 5                   # DBA_ERR_TIMEOUT
    st.close()
    st2 = dba.DbaStepper(B, k, V, 4, constraints=[[[5]], [], [[6, 7]]], dtype=dba.F32, flags=dba.FLAG_FUSED_PROJECTION)
    st2.step_fused(hd[:B * k].contiguous(), ed)
    st2.finalize()
    st2.close()


def test_argument_errors_are_reported_not_launched(dba):
    mk = lambda **kw: dba.DbaStepper(**{**dict(B=1, k=2, V=50, max_steps=3, constraints=[[[5]]]), **kw})
    for kw, code in [(dict(k=65), 2), (dict(constraints=[[[w] for w in range(4, 69)]], V=100), 2),
                     (dict(constraints=[[[2]]]), 1), (dict(constraints=[[[50]]]), 1), (dict(constraints=[[[]]]), 1),
                     (dict(k=0), 1), (dict(V=2**31 // 2, k=2), 2),
                     (dict(k=64, V=3000, constraints=[[[w] for w in range(100, 164)]]), 2),    # candidates beyond shared memory
                     (dict(dtype=7), 1), (dict(eos=99), 1)]:
        with pytest.raises(dba.DbaError) as e:
            mk(**kw)
        assert e.value.code == code, kw
    ones = lambda n: [[[w] for w in range(100, 100 + n)]]
    for kw in [dict(k=64, V=88000, constraints=ones(36)), dict(k=64, V=40000, constraints=ones(36)),
               dict(k=64, V=262144, constraints=ones(12)), dict(k=40, V=262144, constraints=ones(64))]:          # the corners the header promises
        mk(**kw).close()
    st = mk()
    with pytest.raises(dba.DbaError) as e:
        st.step_host(torch.zeros(2, 50), st.new_outputs(host=True))
    assert e.value.code == 3                                        # no staging area was requested
