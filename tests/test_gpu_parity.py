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
@pytest.mark.parametrize("V,n_top", [(1, 3), (7, 7), (1000, 7), (4099, 22), (32000, 12), (64000, 22), (20011, 66)])
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
