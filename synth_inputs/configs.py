"""The five synthetic workloads (shapes of BPE NMT decoding) and their constraint sets.

Constraint ids are drawn uniformly from [4, V), distinct within a sentence; ids 0..3 are the special
symbols PAD, BOS, EOS, UNK and never appear in a constraint.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

PAD, BOS, EOS, UNK = 0, 1, 2, 3


@dataclass
class Workload:
    name: str
    cfg_id: int
    B: int
    k: int
    V: int
    steps: int
    dtype: str                  # "f32" | "bf16"
    zipf: bool                  # False: plain N(0, 3^2) rows; True: Zipf means + N(0, 1)
    boost: bool                 # hashed +4 on a pending constraint token
    constraints: list = field(default_factory=list)   # per sentence: list of phrases (lists of ids)
    seed: int = 0
    sent_ids: np.ndarray | None = None                # global sentence numbers (subsets keep theirs)

    @property
    def R(self):
        return self.B * self.k

    def subset(self, sent_idx):
        """The same workload restricted to some sentences; their logit streams do not change."""
        sent_idx = list(sent_idx)
        return Workload(self.name, self.cfg_id, len(sent_idx), self.k, self.V, self.steps, self.dtype,
                        self.zipf, self.boost, [self.constraints[i] for i in sent_idx], self.seed,
                        self.sent_ids[sent_idx].copy())

    def csr(self):
        """Two-level ragged layout: sentence -> phrases -> token ids, all int32."""
        sent_off, phr_off, tok = [0], [0], []
        for c in self.constraints:
            for p in c:
                tok.extend(p)
                phr_off.append(len(tok))
            sent_off.append(len(phr_off) - 1)
        return np.array(sent_off, np.int32), np.array(phr_off, np.int32), np.array(tok, np.int32)

    def flat_tokens(self):
        """[B, 64] constraint token ids in position order (-1 padded) and [B] totals."""
        ct = np.full((self.B, 64), -1, np.int32)
        n = np.zeros(self.B, np.int32)
        for b, c in enumerate(self.constraints):
            flat = [w for p in c for w in p]
            ct[b, :len(flat)] = flat
            n[b] = len(flat)
        return ct, n


def _distinct_ids(rng, n, V):
    return (rng.choice(V - 4, size=n, replace=False) + 4).astype(int).tolist() if n else []


def _split(ids, lengths):
    out, i = [], 0
    for L in lengths:
        out.append(ids[i:i + L]); i += L
    return out


def _composition(rng, total, lo, hi, max_parts):
    """Random split of `total` into at most `max_parts` parts, each in [lo, hi] (rejection sampling)."""
    if total == 0:
        return []
    while True:
        parts, left = [], total
        while left > 0 and len(parts) < max_parts:
            L = int(rng.integers(lo, hi + 1))
            L = min(L, left)
            parts.append(L); left -= L
        if left == 0:
            return parts


def _constraints(cfg_id, B, V, rng, C_fixed=None):
    cons = []
    for _ in range(B):
        if cfg_id == 1:
            ids = _distinct_ids(rng, 2, V); cons.append([[i] for i in ids])
        elif cfg_id == 2:
            lens = [int(rng.integers(1, 4)) for _ in range(4)]
            cons.append(_split(_distinct_ids(rng, sum(lens), V), lens))
        elif cfg_id == 3:
            total = int(rng.integers(0, 9))
            lens = _composition(rng, total, 1, 3, 4)
            cons.append(_split(_distinct_ids(rng, total, V), lens))
        elif cfg_id == 4:
            ids = _distinct_ids(rng, C_fixed, V); cons.append([[i] for i in ids])
        elif cfg_id in (5, 6):
            lens = _composition(rng, 10, 1, 4, 10)
            cons.append(_split(_distinct_ids(rng, 10, V), lens))
        else:
            raise ValueError(cfg_id)
    return cons


CONFIGS = {
    "tiny":    dict(cfg_id=1, B=1,   k=5,  V=1000,  steps=20,  dtype="f32",  zipf=False, boost=False),
    "phrasal": dict(cfg_id=2, B=1,   k=10, V=32000, steps=60,  dtype="f32",  zipf=True,  boost=True),
    "ragged":  dict(cfg_id=3, B=64,  k=10, V=32000, steps=80,  dtype="bf16", zipf=True,  boost=True),
    "scaling": dict(cfg_id=4, B=16,  k=20, V=32000, steps=100, dtype="f32",  zipf=True,  boost=True),
    "serving": dict(cfg_id=5, B=256, k=20, V=64000, steps=120, dtype="bf16", zipf=True,  boost=True),
    # not one of the five named configurations: a second shape for the long-row path (a Transformer-sized
    # vocabulary in fp32: rows of 512 KB), constraints as in "serving"
    "transformer": dict(cfg_id=6, B=128, k=20, V=131072, steps=40, dtype="f32", zipf=True, boost=True),
}


def make_workload(name: str, seed: int = 0, C: int | None = None, **override) -> Workload:
    """Build one of the named workloads.  `C` selects the constraint count of the "scaling" sweep
    (1, 5, 10, 20 or 50 single tokens per sentence).  Keyword overrides shrink a workload for tests
    (B, k, V, steps) without changing how it is generated."""
    p = dict(CONFIGS[name]); p.update(override)
    if name == "scaling" and C is None:
        C = 10
    rng = np.random.default_rng([seed, p["cfg_id"], C or 0])
    cons = _constraints(p["cfg_id"], p["B"], p["V"], rng, C)
    return Workload(name=name if C is None else f"{name}-C{C}", cfg_id=p["cfg_id"], B=p["B"], k=p["k"],
                    V=p["V"], steps=p["steps"], dtype=p["dtype"], zipf=p["zipf"], boost=p["boost"],
                    constraints=cons, seed=seed, sent_ids=np.arange(p["B"], dtype=np.int64))
