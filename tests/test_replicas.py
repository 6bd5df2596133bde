"""The multi-GPU mode of the benchmark is N independent replicas (sentences never interact: no collective on
the data path).  Its host logic - which sentences a rank gets, how the ranks' times become one rate, which
rank runs the reference arm - is checked here with two gloo processes on the CPU."""
import os
import subprocess
import sys

import numpy as np
import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist            # noqa: E402
import torch.multiprocessing as mp          # noqa: E402

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from synth_inputs import LogitStream, make_workload
    wl = bench.replica_workload(make_workload("ragged", B=3, V=512, steps=4), rank)
    ids = torch.from_numpy(wl.sent_ids.copy())
    gathered = [torch.zeros_like(ids) for _ in range(world)]
    dist.all_gather(gathered, ids)
    # the slower rank decides: rank r pretends to have taken (r + 1) seconds for 10 steps
    rate, secs = bench.job_rate(10, float(rank + 1), world, torch.device("cpu"))
    tok = np.full(wl.R, 5, np.int32); mask = np.zeros(wl.R, np.uint64)
    x = LogitStream(wl).step_logits(0, tok, mask)
    digest = torch.tensor([float(np.asarray(x, np.uint16).astype(np.float64).sum())], dtype=torch.float64)
    sums = [torch.zeros_like(digest) for _ in range(world)]
    dist.all_gather(sums, digest)
    if rank == 0:
        out.put(([g.tolist() for g in gathered], rate, secs, [float(v) for v in sums]))
    dist.destroy_process_group()


def test_two_replicas_take_distinct_sentences_and_the_slowest_rank_sets_the_rate():
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    world, port = 2, 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    ids, rate, secs, sums = out.get()
    assert ids == [[0, 1, 2], [3, 4, 5]]                     # disjoint sentence ids
    assert secs == 2.0 and rate == pytest.approx(2 * 10 / 2.0)     # all ranks' steps over the slowest rank's time
    assert sums[0] != sums[1]                                # different sentences, different logit streams


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
