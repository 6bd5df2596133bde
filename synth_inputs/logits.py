"""Counter-based synthetic logit rows (numpy version; ``gen.cu`` writes the same bits on the GPU).

A row is a pure function of (seed, workload id, step, sentence number, the hypothesis' last token and
the pending-constraint hint), so two beam slots with the same last token and hint get identical rows.

    key   = mix(mix(mix(mix(seed ^ SALT*cfg) + step) + sentence) + last_token)
    u16   = 16-bit lane (w & 3) of mix(key + (w >> 2))            one 64-bit hash feeds four tokens
    z     = NORMAL_TABLE[u16]                                     65536 normal quantiles, fp32
    x[w]  = fl32(fl32(sigma * z) + mu[w])                         one fp32 multiply, one fp32 add

mix() is the splitmix64 output function.  mu[w] is 0 for the plain workload; for the Zipf workloads it
is -1.1*ln(rank(w)) under a seeded permutation of ids 4..V-1, -20 for PAD/BOS/UNK, and for EOS
-1.1*ln(1000) until the sentence's hashed end step and +2 from then on.  With probability 0.3 per
(step, sentence, last token) the row adds +4 to the first constraint token the hypothesis has not yet
met (read off the lowest clear bit of its met mask; no constraint logic is involved).
bf16 rows are the fp32 rows rounded to nearest-even.
"""
from __future__ import annotations

import numpy as np

from .configs import BOS, EOS, PAD, UNK, Workload

M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
GOLDEN = np.uint64(0x9E3779B97F4A7C15)
MIX1 = np.uint64(0xBF58476D1CE4E5B9)
MIX2 = np.uint64(0x94D049BB133111EB)
CFG_SALT = np.uint64(0xD6E8FEB86659FD93)
BOOST_SALT = np.uint64(0xB0057B0057B0057B)
END_SALT = np.uint64(0xE05E05E05E05E05E)
BOOST_P16 = 19661            # 0.3 * 65536, compared with a 16-bit hash lane
BOOST_ADD = np.float32(4.0)


def mix(x):
    """splitmix64 output function on uint64 scalars or arrays (wrapping arithmetic)."""
    with np.errstate(over="ignore"):
        z = (np.asarray(x, dtype=np.uint64) + GOLDEN) & M64
        z = ((z ^ (z >> np.uint64(30))) * MIX1) & M64
        z = ((z ^ (z >> np.uint64(27))) * MIX2) & M64
        return z ^ (z >> np.uint64(31))


def normal_table() -> np.ndarray:
    """65536 standard-normal quantiles at the bucket mid-points, as fp32."""
    from scipy.special import ndtri
    q = ndtri((np.arange(65536, dtype=np.float64) + 0.5) / 65536.0)
    return q.astype(np.float32)


def zipf_means(V: int, seed: int) -> np.ndarray:
    mu = np.empty(V, dtype=np.float64)
    perm = np.random.default_rng([seed, 0x21F]).permutation(V - 4)       # id 4+i -> rank perm[i]+1
    mu[4:] = -1.1 * np.log(perm.astype(np.float64) + 1.0)
    mu[[PAD, BOS, UNK]] = -20.0
    mu[EOS] = -1.1 * np.log(1000.0)
    return mu.astype(np.float32)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round to nearest even; inputs are finite."""
    b = x.view(np.uint32)
    return ((b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


class LogitStream:
    """Generates the [B*k, V] logit matrix of one step from the beam's last tokens and met masks."""

    def __init__(self, wl: Workload):
        self.wl = wl
        self.table = normal_table()
        self.sigma = np.float32(1.0 if wl.zipf else 3.0)
        self.mu = zipf_means(wl.V, wl.seed) if wl.zipf else np.zeros(wl.V, np.float32)
        self.eos_late = np.float32(2.0)
        self.ctok, self.ncon = wl.flat_tokens()
        with np.errstate(over="ignore"):
            self.base_key = mix(np.uint64(wl.seed) ^ (CFG_SALT * np.uint64(wl.cfg_id)))
            u = mix(mix(self.base_key ^ END_SALT) + wl.sent_ids.astype(np.uint64)) & np.uint64(0xFFFF)
        # end step of each sentence: floor((0.5 + 0.4*u/65536) * steps), in integer arithmetic
        self.end_step = ((32768 + (u.astype(np.int64) * 26214 >> 16)) * wl.steps >> 16).astype(np.int32)

    def row_keys(self, step: int, last_token: np.ndarray) -> np.ndarray:
        wl = self.wl
        with np.errstate(over="ignore"):
            ks = mix(self.base_key + np.uint64(step))
            kb = mix(ks + np.repeat(wl.sent_ids.astype(np.uint64), wl.k))
            return mix(kb + last_token.astype(np.int64).astype(np.uint64))

    def boost_tokens(self, keys: np.ndarray, met_mask: np.ndarray) -> np.ndarray:
        """Per row the token that gets +4 this step, or -1."""
        wl = self.wl
        out = np.full(wl.R, -1, np.int32)
        if not wl.boost:
            return out
        fire = (mix(keys ^ BOOST_SALT) & np.uint64(0xFFFF)).astype(np.int64) < BOOST_P16
        for r in np.nonzero(fire)[0]:
            b = r // wl.k
            inv = ~int(met_mask[r]) & 0xFFFFFFFFFFFFFFFF
            j = (inv & -inv).bit_length() - 1 if inv else 64
            if j < self.ncon[b]:
                out[r] = self.ctok[b, j]
        return out

    def step_logits(self, step: int, last_token: np.ndarray, met_mask: np.ndarray) -> np.ndarray:
        """[R, V] float32, or uint16 holding bf16 bits for bf16 workloads."""
        wl = self.wl
        V = wl.V
        keys = self.row_keys(step, np.asarray(last_token))
        boost = self.boost_tokens(keys, np.asarray(met_mask, dtype=np.uint64))
        w = np.arange(V, dtype=np.uint64)
        quad, lane = w >> np.uint64(2), (w & np.uint64(3)) * np.uint64(16)
        out = np.empty((wl.R, V), np.float32)
        for r in range(wl.R):
            with np.errstate(over="ignore"):
                hq = mix(keys[r] + np.arange((V + 3) // 4, dtype=np.uint64))
            u16 = ((hq[quad.astype(np.int64)] >> lane) & np.uint64(0xFFFF)).astype(np.int64)
            x = (self.sigma * self.table[u16]).astype(np.float32) + self.mu
            if wl.zipf and step >= self.end_step[r // wl.k]:
                x[EOS] = np.float32(self.sigma * self.table[u16[EOS]]) + self.eos_late
            if boost[r] >= 0:
                x[boost[r]] = x[boost[r]] + BOOST_ADD
            out[r] = x
        return to_bf16_bits(out) if wl.dtype == "bf16" else out
