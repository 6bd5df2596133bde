"""ctypes binding of the C ABI in include/dba.h.  Argument marshalling only: every step of the method runs
in the CUDA kernels of libdba.so.  torch is used for device memory and streams.  There is no fallback: if the
library has not been built, importing `lib()` raises."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libdba.so")

F32, BF16 = 0, 1
FLAG_ADJUST_OFF, FLAG_LENGTH_NORM, FLAG_HOST_STAGING, FLAG_PRUNE_NORMALISED, FLAG_FUSED_PROJECTION = 1, 2, 4, 8, 16

EXPORTS = ["dba_workspace_bytes", "dba_init", "dba_reset", "dba_step", "dba_step_fused", "dba_step_host", "dba_finalize",
           "dba_timing_enable", "dba_timing_read", "dba_counters", "dba_launch_count", "dba_test_hook", "dba_destroy", "dba_status_string", "dba_row_scan_scratch_bytes", "dba_row_scan",
           "dba_row_scan_static", "dba_row_scan_static_max_bytes", "dba_project_scan_scratch_bytes", "dba_project_scan"]


class DbaError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {lib().dba_status_string(code).decode()} (status {code})")


class Config(C.Structure):
    _fields_ = [("B", C.c_int32), ("k", C.c_int32), ("V", C.c_int32), ("max_steps", C.c_int32),
                ("pad_id", C.c_int32), ("bos_id", C.c_int32), ("eos_id", C.c_int32), ("logit_dtype", C.c_int32),
                ("flags", C.c_uint32), ("sent_phrase_off", C.c_void_p), ("phrase_tok_off", C.c_void_p),
                ("tok", C.c_void_p), ("prune_threshold", C.c_float)]


class StepOut(C.Structure):
    _fields_ = [("backptr", C.c_void_p), ("token", C.c_void_p), ("score", C.c_void_p), ("bank", C.c_void_p),
                ("met_mask", C.c_void_p), ("active", C.c_void_p), ("row_lse", C.c_void_p), ("stop", C.c_void_p)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_1804_06609_b200.build` "
                              "(there is no CPU fallback)")
        L = C.CDLL(_LIB_PATH)
        vp = C.c_void_p
        L.dba_workspace_bytes.argtypes = [C.POINTER(Config), C.POINTER(C.c_size_t)]
        L.dba_init.argtypes = [C.POINTER(Config), vp, C.c_size_t, vp, C.POINTER(vp)]
        L.dba_reset.argtypes = [vp]
        L.dba_step.argtypes = [vp, vp, C.c_int64, vp, C.POINTER(StepOut)]
        L.dba_step_host.argtypes = [vp, vp, C.c_int64, C.POINTER(StepOut)]
        L.dba_step_fused.argtypes = [vp, vp, C.c_int64, vp, C.c_int64, C.c_int32, C.POINTER(StepOut)]
        L.dba_finalize.argtypes = [vp, vp, vp, vp, vp]
        L.dba_timing_enable.argtypes = [vp, C.c_int32]
        L.dba_timing_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
        L.dba_counters.argtypes = [vp, C.POINTER(C.c_uint32)]
        L.dba_launch_count.argtypes = [vp]
        L.dba_launch_count.restype = C.c_uint64
        L.dba_test_hook.argtypes = [vp, C.c_int64, C.c_int32]
        L.dba_destroy.argtypes = [vp]
        L.dba_destroy.restype = None
        L.dba_status_string.argtypes = [C.c_int]
        L.dba_status_string.restype = C.c_char_p
        L.dba_row_scan_scratch_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_size_t)]
        L.dba_row_scan.argtypes = [vp, C.c_int32, C.c_int32, C.c_int32, C.c_int64, C.c_int32, vp, C.c_size_t,
                                   vp, vp, vp, vp]
        L.dba_row_scan_static.argtypes = [vp, C.c_int32, C.c_int32, C.c_int32, C.c_int64, C.c_int32, vp, vp, vp, vp]
        L.dba_row_scan_static_max_bytes.restype = C.c_size_t
        L.dba_project_scan_scratch_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_size_t)]
        L.dba_project_scan.argtypes = [vp, C.c_int64, vp, C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_int32, vp, C.c_size_t,
                                       vp, vp, vp, vp]
        _lib = L
    return _lib


def _check(code, where):
    if code != 0:
        raise DbaError(code, where)


def _dtype_code(t):
    import torch
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"logits must be float32 or bfloat16, got {t.dtype}")


class DbaStepper:
    """Owns a dba_handle and its workspace.  Constraints: per sentence a list of phrases (lists of token ids),
    or the three CSR arrays (sent_phrase_off, phrase_tok_off, tok)."""

    OUT_FIELDS = ("backptr", "token", "score", "bank", "met_mask", "active", "row_lse", "stop")

    def __init__(self, B, k, V, max_steps, constraints=None, csr=None, dtype=F32, pad=0, bos=1, eos=2, flags=0,
                 device="cuda:0", stream=None, prune=0.0):
        import torch
        self.torch = torch
        self.B, self.k, self.V, self.R, self.max_steps, self.dtype = B, k, V, B * k, max_steps, dtype
        self.device = torch.device(device)
        if csr is None:
            so, po, tk = [0], [0], []
            for c in constraints:
                for p in c:
                    tk.extend(p); po.append(len(tk))
                so.append(len(po) - 1)
            csr = (so, po, tk)
        self._so = np.ascontiguousarray(csr[0], np.int32)
        self._po = np.ascontiguousarray(csr[1], np.int32)
        self._tk = np.ascontiguousarray(csr[2] if len(csr[2]) else [0], np.int32)
        self.cfg = Config(B, k, V, max_steps, pad, bos, eos, dtype, flags, self._so.ctypes.data, self._po.ctypes.data,
                          self._tk.ctypes.data, prune)
        n = C.c_size_t()
        _check(lib().dba_workspace_bytes(C.byref(self.cfg), C.byref(n)), "dba_workspace_bytes")
        self.workspace_bytes = n.value
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(n.value + 256, dtype=torch.uint8, device=self.device)
            base = (self.workspace.data_ptr() + 255) // 256 * 256
            self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
            h = C.c_void_p()
            _check(lib().dba_init(C.byref(self.cfg), base, n.value, self.stream.cuda_stream, C.byref(h)), "dba_init")
        self._h = h
        self.out = self.new_outputs()

    def new_outputs(self, host=False):
        torch = self.torch
        kw = dict(device="cpu", pin_memory=True) if host else dict(device=self.device)
        R = self.R
        return dict(backptr=torch.zeros(R, dtype=torch.int32, **kw), token=torch.zeros(R, dtype=torch.int32, **kw),
                    score=torch.zeros(R, dtype=torch.float32, **kw), bank=torch.zeros(R, dtype=torch.int32, **kw),
                    met_mask=torch.zeros(R, dtype=torch.int64, **kw), active=torch.zeros(R, dtype=torch.int32, **kw),
                    row_lse=torch.zeros(R, dtype=torch.float32, **kw),
                    stop=torch.zeros(self.B, dtype=torch.int32, **kw))

    @staticmethod
    def _out_struct(out):
        return StepOut(*[(out[f].data_ptr() if out is not None and out.get(f) is not None else None)
                         for f in DbaStepper.OUT_FIELDS])

    def reset(self):
        _check(lib().dba_reset(self._h), "dba_reset")

    def step(self, logits, row_lse_in=None, out=None):
        """logits: CUDA tensor [B*k, V] (float32 or bfloat16, unit inner stride).  Returns the output dict."""
        assert logits.is_cuda and logits.dim() == 2 and logits.shape == (self.R, self.V) and logits.stride(1) == 1
        assert _dtype_code(logits) == self.dtype
        out = self.out if out is None else out
        so = self._out_struct(out)
        lse_ptr = None
        if row_lse_in is not None:
            assert row_lse_in.is_cuda and row_lse_in.dtype == self.torch.float32 and row_lse_in.numel() == self.R
            lse_ptr = row_lse_in.data_ptr()
        _check(lib().dba_step(self._h, logits.data_ptr(), logits.stride(0), lse_ptr, C.byref(so)), "dba_step")
        return out

    def step_fused(self, hidden, embed, out=None):
        """hidden: CUDA bfloat16 [B*k, D]; embed: CUDA bfloat16 [V, D].  The step on logits = hidden @ embed.T, which are
        never materialised.  The stepper must have been made with FLAG_FUSED_PROJECTION."""
        torch = self.torch
        assert hidden.is_cuda and embed.is_cuda and hidden.dtype == torch.bfloat16 and embed.dtype == torch.bfloat16
        assert hidden.shape[0] == self.R and embed.shape[0] == self.V and hidden.shape[1] == embed.shape[1]
        assert hidden.stride(1) == 1 and embed.stride(1) == 1
        out = self.out if out is None else out
        so = self._out_struct(out)
        _check(lib().dba_step_fused(self._h, hidden.data_ptr(), hidden.stride(0), embed.data_ptr(), embed.stride(0),
                                    hidden.shape[1], C.byref(so)), "dba_step_fused")
        return out

    def step_host(self, logits_host, out_host):
        """logits_host: CPU tensor [B*k, V] (pinned for asynchronous copies); out_host: dict of CPU tensors."""
        assert not logits_host.is_cuda and logits_host.shape == (self.R, self.V) and logits_host.stride(1) == 1
        so = self._out_struct(out_host)
        _check(lib().dba_step_host(self._h, logits_host.data_ptr(), logits_host.stride(0), C.byref(so)), "dba_step_host")
        return out_host

    def finalize(self):
        tokens = np.zeros((self.B, self.max_steps), np.int32)
        length = np.zeros(self.B, np.int32); score = np.zeros(self.B, np.float32); flags = np.zeros(self.B, np.int32)
        _check(lib().dba_finalize(self._h, tokens.ctypes.data, length.ctypes.data, score.ctypes.data, flags.ctypes.data),
               "dba_finalize")
        return tokens, length, score, flags

    def timing_enable(self, on=True):
        _check(lib().dba_timing_enable(self._h, int(on)), "dba_timing_enable")

    def timing_read(self):
        """(ms of [row scan, candidates + allocation, 0] summed over the recorded steps, number of steps)."""
        ms = (C.c_double * 3)(); n = C.c_int64()
        _check(lib().dba_timing_read(self._h, ms, C.byref(n)), "dba_timing_read")
        return list(ms), n.value

    def counters(self):
        """Diagnostic counters: [row segments ranked by the slow second pass, 0, 0, 0]."""
        out = (C.c_uint32 * 4)()
        _check(lib().dba_counters(self._h, out), "dba_counters")
        return list(out)

    def test_hook(self, wait_clocks=0, drop_item=-1):
        """Testing aid: shortens the row scan's bounded waits and can make one run out (see dba_test_hook)."""
        _check(lib().dba_test_hook(self._h, wait_clocks, drop_item), "dba_test_hook")

    def launch_count(self):
        return int(lib().dba_launch_count(self._h))

    def close(self):
        if getattr(self, "_h", None):
            lib().dba_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()


def row_scan(logits, n_top, stream=None):
    """Per row: log-sum-exp and the n_top largest entries (value desc, lower index first)."""
    import torch
    assert logits.is_cuda and logits.dim() == 2 and logits.stride(1) == 1
    R, V = logits.shape
    n = C.c_size_t()
    dt = _dtype_code(logits)
    _check(lib().dba_row_scan_scratch_bytes(R, V, n_top, dt, C.byref(n)), "dba_row_scan_scratch_bytes")
    scratch = torch.empty(n.value + 256, dtype=torch.uint8, device=logits.device)
    base = (scratch.data_ptr() + 255) // 256 * 256
    lse = torch.empty(R, dtype=torch.float32, device=logits.device)
    val = torch.empty(R, n_top, dtype=torch.float32, device=logits.device)
    idx = torch.empty(R, n_top, dtype=torch.int32, device=logits.device)
    st = stream if stream is not None else torch.cuda.current_stream(logits.device)
    _check(lib().dba_row_scan(logits.data_ptr(), dt, R, V, logits.stride(0), n_top, base, n.value, lse.data_ptr(),
                              val.data_ptr(), idx.data_ptr(), st.cuda_stream), "dba_row_scan")
    st.synchronize()          # the scratch tensor must outlive the kernels
    return lse, val, idx


def project_scan(hidden, embed, n_top, stream=None):
    """Fused output projection + row scan: hidden [R, D] and embed [V, D] (CUDA, bfloat16, unit inner stride).  Per
    row of hidden @ embed.T: log-sum-exp and the n_top largest logits, as row_scan returns them."""
    import torch
    assert hidden.is_cuda and embed.is_cuda and hidden.dtype == torch.bfloat16 and embed.dtype == torch.bfloat16
    assert hidden.dim() == 2 and embed.dim() == 2 and hidden.shape[1] == embed.shape[1]
    assert hidden.stride(1) == 1 and embed.stride(1) == 1 and hidden.device == embed.device
    R, D = hidden.shape
    V = embed.shape[0]
    with torch.cuda.device(hidden.device):
        n = C.c_size_t()
        _check(lib().dba_project_scan_scratch_bytes(R, V, n_top, C.byref(n)), "dba_project_scan_scratch_bytes")
        scratch = torch.empty(n.value + 256, dtype=torch.uint8, device=hidden.device)
        base = (scratch.data_ptr() + 255) // 256 * 256
        lse = torch.empty(R, dtype=torch.float32, device=hidden.device)
        val = torch.empty(R, n_top, dtype=torch.float32, device=hidden.device)
        idx = torch.empty(R, n_top, dtype=torch.int32, device=hidden.device)
        st = stream if stream is not None else torch.cuda.current_stream(hidden.device)
        _check(lib().dba_project_scan(hidden.data_ptr(), hidden.stride(0), embed.data_ptr(), embed.stride(0), R, V, D, n_top,
                                      base, n.value, lse.data_ptr(), val.data_ptr(), idx.data_ptr(), st.cuda_stream),
               "dba_project_scan")
        st.synchronize()          # the scratch tensor must outlive the kernels
    return lse, val, idx


def row_scan_static(logits, n_top, lse, val, idx, stream=None):
    """dba_row_scan_static: like row_scan, but the library's built-in scratch is used and the caller brings the
    output tensors (lse [R] f32, val [R, n_top] f32, idx [R, n_top] i32).  Nothing is allocated here."""
    import torch
    assert logits.is_cuda and logits.dim() == 2 and logits.stride(1) == 1
    R, V = logits.shape
    for t, shape, dt in ((lse, (R,), torch.float32), (val, (R, n_top), torch.float32), (idx, (R, n_top), torch.int32)):
        assert t.is_cuda and t.device == logits.device and t.dtype == dt and tuple(t.shape) == shape and t.is_contiguous()
    with torch.cuda.device(logits.device):         # the library looks its scratch up on the current device
        st = stream if stream is not None else torch.cuda.current_stream(logits.device)
        _check(lib().dba_row_scan_static(logits.data_ptr(), _dtype_code(logits), R, V, logits.stride(0), n_top,
                                         lse.data_ptr(), val.data_ptr(), idx.data_ptr(), st.cuda_stream),
               "dba_row_scan_static")
