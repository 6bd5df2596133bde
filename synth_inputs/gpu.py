"""GPU version of LogitStream (same bits as the numpy one), for workloads too large to generate on the host."""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

from .logits import LogitStream

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.cu")
_LIB = os.path.join(_HERE, "libdba_synth.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
                               "--fmad=false", "-Xcompiler", "-fPIC", "-shared", "-o", _LIB, _SRC])
    return _LIB


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB):
            raise ImportError(f"{_LIB} is missing: build it with synth_inputs.gpu.build()")
        _lib = C.CDLL(_LIB)
        vp = C.c_void_p
        _lib.synth_gen_logits.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int64, C.c_uint64, C.c_int,
                                          vp, vp, vp, vp, vp, vp, vp, C.c_float, C.c_int, C.c_int, vp, C.c_float, vp]
    return _lib


class GpuLogitStream:
    def __init__(self, wl, device="cuda:0"):
        import torch
        self.torch, self.wl, self.device = torch, wl, torch.device(device)
        host = LogitStream(wl)
        self.host = host
        dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(self.device)
        self.table, self.mu = dev(host.table), dev(host.mu)
        self.ctok, self.ncon = dev(host.ctok), dev(host.ncon)
        self.end_step = dev(host.end_step)
        self.sent_ids = dev(wl.sent_ids.astype(np.int64))
        self.base_key = int(host.base_key)
        self.tdtype = torch.bfloat16 if wl.dtype == "bf16" else torch.float32

    def step_logits(self, step, last_token, met_mask, out=None):
        """last_token int32 [R], met_mask int64 [R] (CUDA tensors).  Returns [R, V] logits on the device."""
        torch, wl = self.torch, self.wl
        if out is None:
            out = torch.empty(wl.R, wl.V, dtype=self.tdtype, device=self.device)
        assert out.shape == (wl.R, wl.V) and out.stride(1) == 1 and out.dtype == self.tdtype
        assert last_token.dtype == torch.int32 and met_mask.dtype == torch.int64
        rc = lib().synth_gen_logits(out.data_ptr(), int(wl.dtype == "bf16"), wl.R, wl.V, wl.k, out.stride(0),
                                    self.base_key, step, self.sent_ids.data_ptr(), last_token.data_ptr(),
                                    met_mask.data_ptr(), self.ctok.data_ptr(), self.ncon.data_ptr(),
                                    self.table.data_ptr(), self.mu.data_ptr(), float(self.host.sigma), int(wl.zipf),
                                    int(wl.boost), self.end_step.data_ptr(), float(self.host.eos_late),
                                    torch.cuda.current_stream(self.device).cuda_stream)
        if rc != 0:
            raise RuntimeError(f"synth_gen_logits: CUDA error {rc}")
        return out
