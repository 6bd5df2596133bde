"""dba_row_scan_static, the entry point for callers that cannot allocate device memory (a process with a
frozen memory pool, a plug-in without an allocator, a latency path that must not synchronise the device):
called through the C ABI twice in a row, it must give what dba_row_scan gives with caller-owned scratch.
This file is collected last on purpose, so a run that stops at the first failure has run everything else."""
import ctypes as C

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def test_static_scratch_row_scan_matches_row_scan_on_two_calls_in_a_row():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_1804_06609_b200 as pkg
    from paper_1804_06609_b200 import binding
    L = pkg.lib()
    assert L.dba_row_scan_static_max_bytes() == 4 << 20
    rng = np.random.default_rng(0)
    # two different problems back to back: the second is smaller, so stale partial results of the first
    # would still sit in the shared scratch if they were read
    for R, V, n_top, dtype in [(24, 20011, 22, torch.float32), (5, 4099, 7, torch.bfloat16), (24, 20011, 22, torch.float32)]:
        x = torch.from_numpy(rng.normal(0, 3, (R, V)).astype(np.float32)).cuda().to(dtype)
        want_lse, want_val, want_idx = pkg.row_scan(x, n_top)
        lse = torch.full((R,), 7.0, dtype=torch.float32, device="cuda")
        val = torch.zeros(R, n_top, dtype=torch.float32, device="cuda")
        idx = torch.zeros(R, n_top, dtype=torch.int32, device="cuda")
        binding.row_scan_static(x, n_top, lse, val, idx)
        torch.cuda.synchronize()
        assert torch.equal(idx, want_idx) and torch.equal(val, want_val)
        assert (lse - want_lse).abs().max().item() <= 1e-5
    # a problem whose partial results do not fit the fixed scratch is refused, nothing is launched
    big = torch.zeros(1, 8, dtype=torch.float32, device="cuda")
    need = C.c_size_t()
    assert L.dba_row_scan_scratch_bytes(100000, 8, 22, 0, C.byref(need)) == 0 and need.value > (4 << 20)
    rc = L.dba_row_scan_static(big.data_ptr(), 0, 100000, 8, 8, 22, lse.data_ptr(), val.data_ptr(), idx.data_ptr(), None)
    assert rc == 2
