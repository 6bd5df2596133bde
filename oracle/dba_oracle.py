"""ctypes wrapper around ``dba_oracle.c`` -- TEST INFRASTRUCTURE, not part of the product.

Only argument marshalling lives here; every step of the method is in the C file.  The CUDA
library never imports this module.  ``build()`` compiles the C file with gcc next to it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dba_oracle.c")
_LIB = os.path.join(_HERE, "libdba_oracle.so")

F32, BF16 = 0, 1
FLAG_ADJUST_OFF, FLAG_LENGTH_NORM, FLAG_PRUNE_NORM = 1, 2, 8

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no optimisation tricks: -O2, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-ffp-contract=off", "-fPIC", "-shared", "-Wall", "-Wextra",
             "-o", _LIB, _SRC, "-lm"])
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        i32p, f32p, u64p = C.POINTER(C.c_int32), C.POINTER(C.c_float), C.POINTER(C.c_uint64)
        L.orc_row_lse.restype = C.c_double
        L.orc_row_lse.argtypes = [C.c_void_p, C.c_int, C.c_int]
        L.orc_row_top.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, f32p, i32p]
        L.orc_project.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, f32p]
        L.orc_project.restype = None
        L.orc_create.restype = C.c_void_p
        L.orc_create.argtypes = [C.c_int] * 6 + [C.c_uint, C.c_int, i32p, i32p]
        L.orc_destroy.argtypes = [C.c_void_p]
        L.orc_num_constraints.argtypes = [C.c_void_p]
        L.orc_steps_done.argtypes = [C.c_void_p]
        L.orc_add.argtypes = [C.c_void_p, C.c_uint64, C.c_int, C.c_int, u64p, i32p]
        L.orc_progress_set.argtypes = [C.c_void_p, C.c_uint64, C.c_int, i32p]
        L.orc_allocate.argtypes = [C.c_int, C.c_int, i32p, C.c_uint, i32p]
        L.orc_get_beam.argtypes = [C.c_void_p, f32p, i32p, i32p, i32p, u64p, i32p, i32p]
        L.orc_set_beam.argtypes = [C.c_void_p, f32p, i32p, u64p, i32p, i32p]
        L.orc_last_candidates.argtypes = [C.c_void_p, C.c_int, i32p, i32p, f32p, i32p, u64p, i32p]
        L.orc_last_allocation.argtypes = [C.c_void_p, i32p, i32p]
        L.orc_step.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_long, f32p]
        L.orc_finalize.argtypes = [C.c_void_p, i32p, i32p, f32p, i32p]
        L.orc_set_prune.argtypes = [C.c_void_p, C.c_float]
        L.orc_set_prune.restype = None
        L.orc_stop_flags.argtypes = [C.c_void_p]
        _lib = L
    return _lib


def _p(a, t):
    return a.ctypes.data_as(C.POINTER(t))


def row_lse(row: np.ndarray) -> float:
    """Double-precision log-sum-exp of one row (float32 array, or uint16 array of bf16 bits)."""
    row = np.ascontiguousarray(row)
    dt = F32 if row.dtype == np.float32 else BF16
    assert row.dtype in (np.float32, np.uint16)
    return lib().orc_row_lse(row.ctypes.data, dt, row.size)


def row_top(row: np.ndarray, n: int):
    """The n largest entries of one row in order (value descending, lower index first)."""
    row = np.ascontiguousarray(row)
    dt = F32 if row.dtype == np.float32 else BF16
    assert row.dtype in (np.float32, np.uint16)
    val = np.zeros(n, np.float32); idx = np.zeros(n, np.int32)
    lib().orc_row_top(row.ctypes.data, dt, row.size, n, _p(val, C.c_float), _p(idx, C.c_int32))
    return val, idx


def project(hidden_bits: np.ndarray, embed_bits: np.ndarray) -> np.ndarray:
    """Output projection: logits[r, w] = <hidden[r], embed[w]> (uint16 arrays of bf16 bits, [R, d] and [V, d]);
    double accumulation, rounded once to fp32."""
    hidden_bits = np.ascontiguousarray(hidden_bits); embed_bits = np.ascontiguousarray(embed_bits)
    assert hidden_bits.dtype == np.uint16 and embed_bits.dtype == np.uint16 and hidden_bits.shape[1] == embed_bits.shape[1]
    R, d = hidden_bits.shape
    V = embed_bits.shape[0]
    out = np.zeros((R, V), np.float32)
    lib().orc_project(hidden_bits.ctypes.data, embed_bits.ctypes.data, R, V, d, _p(out, C.c_float))
    return out


def allocate(k: int, n, flags: int = 0) -> np.ndarray:
    n = np.ascontiguousarray(n, dtype=np.int32)
    alloc = np.zeros_like(n)
    lib().orc_allocate(k, n.size - 1, _p(n, C.c_int32), flags, _p(alloc, C.c_int32))
    return alloc


class Sentence:
    """One sentence's constrained beam: constraints are a list of phrases (lists of token ids)."""

    def __init__(self, k, V, max_steps, phrases, pad=0, bos=1, eos=2, flags=0, prune=0.0):
        self.k, self.V, self.max_steps = k, V, max_steps
        self.pad, self.bos, self.eos, self.flags = pad, bos, eos, flags
        off = np.zeros(len(phrases) + 1, dtype=np.int32)
        for i, p in enumerate(phrases):
            off[i + 1] = off[i] + len(p)
        tok = np.array([w for p in phrases for w in p] or [0], dtype=np.int32)
        self._h = lib().orc_create(k, V, max_steps, pad, bos, eos, flags, len(phrases),
                                   _p(off, C.c_int32), _p(tok, C.c_int32))
        if not self._h:
            raise ValueError("oracle rejected the constraint set")
        self.C = lib().orc_num_constraints(self._h)
        if prune > 0:
            lib().orc_set_prune(self._h, prune)

    def __del__(self):
        if getattr(self, "_h", None) and lib is not None:      # module globals are gone at interpreter exit
            lib().orc_destroy(self._h)
            self._h = None

    def add(self, mask: int, active: int, w: int):
        m, a = C.c_uint64(), C.c_int32()
        lib().orc_add(self._h, mask, active, w, C.byref(m), C.byref(a))
        return m.value, a.value

    def progress_set(self, mask: int, active: int):
        out = np.zeros(64, dtype=np.int32)
        n = lib().orc_progress_set(self._h, mask, active, _p(out, C.c_int32))
        return out[:n].tolist()

    def beam(self):
        k = self.k
        d = dict(score=np.zeros(k, np.float32), token=np.zeros(k, np.int32), backptr=np.zeros(k, np.int32),
                 bank=np.zeros(k, np.int32), met_mask=np.zeros(k, np.uint64), active=np.zeros(k, np.int32),
                 len=np.zeros(k, np.int32))
        lib().orc_get_beam(self._h, _p(d["score"], C.c_float), _p(d["token"], C.c_int32),
                           _p(d["backptr"], C.c_int32), _p(d["bank"], C.c_int32),
                           _p(d["met_mask"], C.c_uint64), _p(d["active"], C.c_int32), _p(d["len"], C.c_int32))
        return d

    def set_beam(self, score, token, met_mask, active, length=None):
        score = np.ascontiguousarray(score, np.float32); token = np.ascontiguousarray(token, np.int32)
        met_mask = np.ascontiguousarray(met_mask, np.uint64); active = np.ascontiguousarray(active, np.int32)
        length = np.ascontiguousarray(length if length is not None else np.zeros(self.k), np.int32)
        lib().orc_set_beam(self._h, _p(score, C.c_float), _p(token, C.c_int32), _p(met_mask, C.c_uint64),
                           _p(active, C.c_int32), _p(length, C.c_int32))

    def step(self, logits: np.ndarray) -> np.ndarray:
        """logits: [k, V] float32, or uint16 holding bf16 bits.  Returns the k row normalisers (fp32)."""
        assert logits.ndim == 2 and logits.shape == (self.k, self.V) and logits.strides[1] == logits.itemsize
        dt = F32 if logits.dtype == np.float32 else BF16
        assert logits.dtype in (np.float32, np.uint16)
        lse = np.zeros(self.k, np.float32)
        rc = lib().orc_step(self._h, logits.ctypes.data, dt, logits.strides[0] // logits.itemsize,
                            _p(lse, C.c_float))
        if rc != 0:
            raise RuntimeError("oracle step refused (max_steps reached)")
        return lse

    def stop_flags(self) -> int:
        """Bit 0: every hypothesis on the (non-empty) beam is completed; bit 1: some hypothesis is."""
        return lib().orc_stop_flags(self._h)

    def candidates(self):
        cap = self.k * (self.C + 3)
        h = np.zeros(cap, np.int32); w = np.zeros(cap, np.int32); sc = np.zeros(cap, np.float32)
        bank = np.zeros(cap, np.int32); mask = np.zeros(cap, np.uint64); act = np.zeros(cap, np.int32)
        n = lib().orc_last_candidates(self._h, cap, _p(h, C.c_int32), _p(w, C.c_int32), _p(sc, C.c_float),
                                      _p(bank, C.c_int32), _p(mask, C.c_uint64), _p(act, C.c_int32))
        return dict(h=h[:n], w=w[:n], score=sc[:n], bank=bank[:n], met_mask=mask[:n], active=act[:n])

    def allocation(self):
        cnt = np.zeros(self.C + 1, np.int32); al = np.zeros(self.C + 1, np.int32)
        lib().orc_last_allocation(self._h, _p(cnt, C.c_int32), _p(al, C.c_int32))
        return cnt, al

    def finalize(self):
        toks = np.zeros(self.max_steps, np.int32)
        n, comp, sc = C.c_int32(), C.c_int32(), C.c_float()
        lib().orc_finalize(self._h, _p(toks, C.c_int32), C.byref(n), C.byref(sc), C.byref(comp))
        return toks[:n.value].tolist(), sc.value, bool(comp.value)


class Batch:
    """B independent sentences stepped together; rows of the logit matrix are r = b*k + h.

    ``threads`` > 1 steps sentences concurrently (the C calls release the GIL); the arithmetic per
    sentence is unchanged.
    """

    def __init__(self, k, V, max_steps, constraints, pad=0, bos=1, eos=2, flags=0, threads=1, prune=0.0):
        self.k, self.V, self.B = k, V, len(constraints)
        self.sent = [Sentence(k, V, max_steps, c, pad, bos, eos, flags, prune) for c in constraints]
        self.threads = threads
        self._pool = ThreadPoolExecutor(threads) if threads > 1 else None

    def step(self, logits: np.ndarray) -> np.ndarray:
        k = self.k
        assert logits.shape == (self.B * k, self.V)
        f = lambda b: self.sent[b].step(logits[b * k:(b + 1) * k])
        res = list(self._pool.map(f, range(self.B))) if self._pool else [f(b) for b in range(self.B)]
        return np.concatenate(res)

    def beam(self):
        bs = [s.beam() for s in self.sent]
        return {key: np.concatenate([b[key] for b in bs]) for key in bs[0]}

    def stop_flags(self):
        return np.array([s.stop_flags() for s in self.sent], np.int32)

    def finalize(self):
        return [s.finalize() for s in self.sent]
