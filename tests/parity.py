"""Helpers of the GPU parity tests: run the oracle and the CUDA library side by side on one workload."""
from __future__ import annotations

import numpy as np

from oracle import dba_oracle as O
from synth_inputs import LogitStream

BEAM_FIELDS = ("backptr", "token", "bank", "met_mask", "active")


def torch_dtype(wl):
    import torch
    return torch.bfloat16 if wl.dtype == "bf16" else torch.float32


def to_device_logits(x_np, wl, device="cuda:0"):
    """numpy logits (float32, or uint16 bf16 bits) -> CUDA tensor of the workload's dtype, same bits."""
    import torch
    t = torch.from_numpy(x_np.view(np.int16) if x_np.dtype == np.uint16 else x_np).to(device)
    return t.view(torch.bfloat16) if x_np.dtype == np.uint16 else t


def to_host_logits(x_dev):
    """CUDA logits -> numpy (float32, or uint16 bits for bf16), same bits."""
    import torch
    if x_dev.dtype == torch.bfloat16:
        return x_dev.view(torch.int16).cpu().numpy().view(np.uint16)
    return x_dev.cpu().numpy()


def gpu_beam(out):
    d = {f: out[f].cpu().numpy() for f in ("backptr", "token", "score", "bank", "active", "row_lse")}
    d["met_mask"] = out["met_mask"].cpu().numpy().view(np.uint64)
    if out.get("stop") is not None:
        d["stop"] = out["stop"].cpu().numpy()
    return d


def assert_beam_equal(got, want, where, fields=BEAM_FIELDS + ("score",)):
    """Bit-exact comparison of a GPU beam with the oracle's; reports the first differing (sentence row, field)."""
    for f in fields:
        a, b = got[f], want[f]
        if f == "score":
            same = (a == b) | (np.isinf(a) & np.isinf(b))
        else:
            same = a == b
        if not same.all():
            r = int(np.nonzero(~same)[0][0])
            raise AssertionError(f"{where}: field {f} differs first at row {r}: gpu {a[r]} oracle {b[r]}\n"
                                 f"gpu    {({g: got[g][r] for g in fields})}\noracle {({g: want[g][r] for g in fields})}")


def lockstep(wl, stepper, steps=None, threads=8, gpu_gen=None, lse_tol=1e-5, flags=0, prune=0.0, row_pad=0):
    """Closed loop with the oracle's row normalisers handed to the CUDA step (the direction oracle -> GPU),
    so that both rank the same fp32 score matrix: every selection output must then match bit for bit at
    every step, and the normalisers the GPU computes itself must agree within lse_tol.
    row_pad > 0: the device rows are row_pad elements apart beyond their length, the gaps filled with a value
    larger than any logit (a read past the end of a row would win every selection)."""
    import torch
    steps = wl.steps if steps is None else steps
    orc = O.Batch(wl.k, wl.V, steps, wl.constraints, flags=flags & 11, threads=threads, prune=prune)
    host_gen = LogitStream(wl) if gpu_gen is None else None
    worst = 0.0
    for t in range(steps):
        ob = orc.beam()
        if gpu_gen is not None:      # generate on the device from the ORACLE's state, copy back for the oracle
            x_dev = gpu_gen.step_logits(t, torch.from_numpy(ob["token"]).cuda(),
                                        torch.from_numpy(ob["met_mask"].view(np.int64)).cuda())
            x_np = to_host_logits(x_dev)
        else:
            x_np = host_gen.step_logits(t, ob["token"], ob["met_mask"])
            x_dev = to_device_logits(x_np, wl)
        if row_pad:
            wide = torch.full((x_dev.shape[0], wl.V + row_pad), 3.0e4, dtype=x_dev.dtype, device=x_dev.device)
            wide[:, :wl.V] = x_dev
            x_dev = wide[:, :wl.V]
        open_rows = np.isfinite(ob["score"]) & (ob["token"] != 2)
        lse_o = orc.step(x_np)
        out = stepper.step(x_dev, row_lse_in=torch.from_numpy(lse_o).cuda())
        g = gpu_beam(out)
        assert_beam_equal(g, orc.beam(), f"{wl.name} step {t}")
        assert np.array_equal(g["stop"], orc.stop_flags()), f"{wl.name} step {t}: stop bits differ"
        err = np.abs(g["row_lse"][open_rows].astype(np.float64) - lse_o[open_rows]).max() if open_rows.any() else 0.0
        worst = max(worst, float(err))
        assert err <= lse_tol, f"{wl.name} step {t}: row normaliser off by {err}"
        assert (g["row_lse"][~open_rows] == 0).all()
    return orc, worst


def assert_finalize_equal(stepper, orc):
    tokens, length, score, flags = stepper.finalize()
    for b, (toks, sc, done) in enumerate(orc.finalize()):
        assert length[b] == len(toks) and tokens[b, :length[b]].tolist() == toks, f"sentence {b}: tokens differ"
        assert (tokens[b, length[b]:] == 0).all()
        assert bool(flags[b] & 1) == done and (score[b] == np.float32(sc) or (np.isinf(score[b]) and np.isinf(sc)))


def check_beam_invariants(g, wl, C_per_sentence, where):
    """Properties every beam must have whatever the tie-breaks were (Sections 3.1-3.3)."""
    k = wl.k
    for b in range(wl.B):
        s = slice(b * k, (b + 1) * k)
        sc = g["score"][s]
        live = np.isfinite(sc)
        assert (np.diff(live.astype(int)) <= 0).all(), f"{where}: empty slot before a live one (sentence {b})"
        assert (np.diff(sc[live]) <= 0).all(), f"{where}: beam not in decreasing order (sentence {b})"
        pc = np.array([bin(int(m)).count("1") for m in g["met_mask"][s]])
        assert (g["bank"][s][live] == pc[live]).all() and (g["bank"][s][~live] == -1).all()
        fin = live & (g["token"][s] == 2)
        assert (pc[fin] == C_per_sentence[b]).all(), f"{where}: end token before all constraints (sentence {b})"
        assert ((g["backptr"][s] >= 0) & (g["backptr"][s] < k)).all()


def free_run(wl, stepper, sample, steps, gpu_gen, threads=8, score_tol=1e-5):
    """The CUDA library in its own closed loop over the whole workload (its own normalisers, logits generated
    from its own beam), next to independent oracle runs of the sampled sentences.  Sentences must match
    exactly.  Where a sampled sentence first differs, the difference must be a tie decided by the last bits of
    a normaliser: the two beams hold the same scores rank by rank within the accumulated tolerance, and at the
    first differing slot the oracle's own candidates hold another score within that tolerance (the near-tie);
    the sentence then leaves the comparison.  Returns (compared sentence-steps, [(step, sentence) that left])."""
    import torch
    sub = wl.subset(sample)
    orc = O.Batch(sub.k, sub.V, steps, sub.constraints, threads=threads)
    host_gen = LogitStream(sub)
    C_all = [sum(len(p) for p in c) for c in wl.constraints]
    k = wl.k
    tok = torch.full((wl.R,), 0, dtype=torch.int32, device="cuda"); tok[::k] = 1
    mask = torch.zeros(wl.R, dtype=torch.int64, device="cuda")
    alive = [True] * len(sample)
    compared, departures = 0, []
    for t in range(steps):
        x_dev = gpu_gen.step_logits(t, tok, mask)
        out = stepper.step(x_dev)
        tok, mask = out["token"].clone(), out["met_mask"].clone()
        g = gpu_beam(out)
        check_beam_invariants(g, wl, C_all, f"{wl.name} step {t}")
        ob = orc.beam()
        orc.step(host_gen.step_logits(t, ob["token"], ob["met_mask"]))
        ob = orc.beam()
        for i, b in enumerate(sample):
            if not alive[i]:
                continue
            gs = {f: g[f][b * k:(b + 1) * k] for f in BEAM_FIELDS + ("score",)}
            os_ = {f: ob[f][i * k:(i + 1) * k] for f in BEAM_FIELDS + ("score",)}
            tol = score_tol * (t + 1)
            fin = np.isfinite(os_["score"])
            assert (np.isfinite(gs["score"]) == fin).all(), f"step {t} sentence {b}: live slots differ"
            assert np.abs(gs["score"][fin] - os_["score"][fin]).max(initial=0) <= tol, \
                f"step {t} sentence {b}: scores differ beyond {tol}"
            if all((gs[f] == os_[f]).all() for f in BEAM_FIELDS):
                compared += 1
                continue
            # the first differing slot must sit at a near-tie among the oracle's candidates of this step
            slot = int(np.nonzero(~np.all([gs[f] == os_[f] for f in BEAM_FIELDS], axis=0))[0][0])
            cand = np.sort(orc.sent[i].candidates()["score"].astype(np.float64))
            here = float(os_["score"][slot])
            near = np.abs(cand - here) <= tol
            assert near.sum() >= 2, f"step {t} sentence {b} slot {slot}: selections differ without a tie to explain it"
            alive[i] = False
            departures.append((t, b))
    return compared, departures
