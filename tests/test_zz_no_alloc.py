"""dba_row_scan_static, the entry point for callers that cannot allocate device memory (a process with a
frozen memory pool, a plug-in without an allocator, a latency path that must not synchronise the device):
called through the C ABI several times in a row, it must give what dba_row_scan gives with caller-owned
scratch, and what the CPU oracle gives.
This file is collected last on purpose, so a run that stops at the first failure has run everything else."""
import ctypes as C

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def test_static_scratch_row_scan_matches_row_scan_on_calls_in_a_row():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_1804_06609_b200 as pkg
    from oracle import dba_oracle as O
    from synth_inputs.logits import to_bf16_bits
    L = pkg.lib()
    assert L.dba_row_scan_static_max_bytes() == 4 << 20
    rng = np.random.default_rng(0)
    # Different problems back to back on one stream, no synchronisation in between: the later ones are smaller,
    # so stale partial results of the earlier ones would still sit in the shared scratch if they were read.
    # 16-byte aligned rows take the streaming scan, whose warps share rows through the scratch (partial results
    # and ticket counters); the odd shapes take the plain kernel.
    shapes = [(24, 20000, 22, torch.float32), (5, 4096, 7, torch.bfloat16), (24, 20000, 22, torch.float32),
              (7, 20011, 22, torch.float32), (40, 64000, 12, torch.bfloat16)]
    xs = [torch.from_numpy(rng.normal(0, 3, (R, V)).astype(np.float32)).cuda().to(dt) for R, V, _, dt in shapes]
    want = [pkg.row_scan(x, n_top) for x, (_, _, n_top, _) in zip(xs, shapes)]
    outs = [(torch.full((R,), 7.0, dtype=torch.float32, device="cuda"), torch.zeros(R, n, dtype=torch.float32, device="cuda"),
             torch.zeros(R, n, dtype=torch.int32, device="cuda")) for R, _, n, _ in shapes]
    torch.cuda.synchronize()
    pkg.row_scan_static(xs[0], shapes[0][2], *outs[0])              # the first call on the device looks the scratch up
    torch.cuda.synchronize()
    free0, held0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
    for x, (R, V, n_top, _), o in zip(xs, shapes, outs):
        pkg.row_scan_static(x, n_top, *o)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == held0   # nothing was allocated
    for x, (R, V, n_top, dt), (lse, val, idx), (want_lse, want_val, want_idx) in zip(xs, shapes, outs, want):
        assert torch.equal(idx, want_idx) and torch.equal(val, want_val)
        assert (lse - want_lse).abs().max().item() <= 1e-5
        # and against the CPU oracle, row by row
        xn = x.float().cpu().numpy()
        for r in range(0, R, max(1, R // 4)):
            row = to_bf16_bits(xn[r]) if dt == torch.bfloat16 else xn[r]
            wv, wi = O.row_top(row, n_top)
            assert np.array_equal(idx[r].cpu().numpy(), wi) and np.array_equal(val[r].cpu().numpy(), wv)
            assert abs(float(lse[r]) - O.row_lse(row)) <= 1e-5
    # a problem whose partial results do not fit the fixed scratch is refused, nothing is launched
    big = torch.zeros(1, 8, dtype=torch.float32, device="cuda")
    need = C.c_size_t()
    lse, val, idx = outs[0]
    assert L.dba_row_scan_scratch_bytes(100000, 8, 22, 0, C.byref(need)) == 0 and need.value > (4 << 20)
    rc = L.dba_row_scan_static(big.data_ptr(), 0, 100000, 8, 8, 22, lse.data_ptr(), val.data_ptr(), idx.data_ptr(), None)
    assert rc == 2
