"""World-size-2 checks of the multi-GPU plumbing, run as gloo ranks on CPU.

The path shards by matrix (independent problems, no data-path collective), so what needs a test
is the host logic: dealing matrices to ranks, the max-over-ranks / summed-work aggregation the
benchmark reports, that a sharded run gives every matrix the result a single process gives it,
and that only rank 0 of the oracle-timing arm does any work.
"""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2412_04180_b200 import inputs, shard

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

# LLaMA-7B layer shapes of one decoder block (Section 5.1 quantises such a model matrix by matrix)
BLOCK = [(4096, 4096)] * 4 + [(11008, 4096)] * 2 + [(4096, 11008)]


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _run_ranks(fn, world, *args):
    port = _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_entry, args=(fn, r, world, port, q) + args) for r in range(world)]
    for p in procs:
        p.start()
    out = {}
    for _ in range(world):
        r, val = q.get(timeout=120)
        out[r] = val
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    return [out[r] for r in range(world)]


def _entry(fn, rank, world, port, q, *args):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        q.put((rank, fn(rank, world, *args)))
    finally:
        dist.destroy_process_group()


def _rank_assignment(rank, world):
    sizes = BLOCK * 32                       # 224 matrices
    table = shard.assign_matrices(sizes, world)
    gathered = [None] * world
    dist.all_gather_object(gathered, table)
    return {"table": table, "same_everywhere": all(t == table for t in gathered)}


def test_assignment_is_a_balanced_partition_and_needs_no_communication():
    res = _run_ranks(_rank_assignment, 2)
    assert all(r["same_everywhere"] for r in res)
    table = res[0]["table"]
    sizes = BLOCK * 32
    assert sorted(i for lst in table for i in lst) == list(range(len(sizes)))
    loads = [sum(sizes[i][0] * sizes[i][1] for i in lst) for lst in table]
    assert max(loads) - min(loads) <= 11008 * 4096
    # odd counts and more ranks than matrices still give a partition
    for world, n in ((3, 7), (8, 5), (1, 4)):
        t = shard.assign_matrices(BLOCK[:n], world)
        assert len(t) == world and sorted(i for lst in t for i in lst) == list(range(n))
    with pytest.raises(ValueError):
        shard.assign_matrices(BLOCK, 0)


def _rank_throughput(rank, world):
    ms = 10.0 if rank == 0 else 25.0        # rank 1 is the slow one
    units = 1000 if rank == 0 else 3000
    return shard.job_throughput(units, ms), shard.max_over_ranks(float(rank)), shard.sum_over_ranks(rank + 1)


def test_job_throughput_is_all_work_over_the_slowest_rank():
    res = _run_ranks(_rank_throughput, 2)
    for (value, total, ms), mx, sm in res:
        assert total == 4000 and ms == 25.0
        assert value == pytest.approx(4000 / 0.025)
        assert mx == 1.0 and sm == 3
    # without a process group the helpers are the identity
    assert shard.job_throughput(10, 2.0) == (5000.0, 10, 2.0)


def _rank_pipeline(rank, world, shapes, seed):
    from oracle import skim_oracle as orc
    orc.build()
    out = {}
    for i in shard.assign_matrices(shapes, world)[rank]:
        rows, cols = shapes[i]
        w, g = inputs.make_matrix(rows, cols, shard.matrix_seed(seed, i))
        res = orc.cluster_rows(w, g, [1, 2, 3, 4], 8, want_codes=False)
        bits, total = orc.allocate_bits(res["err"].astype(np.float32), 1, 3.0)
        out[i] = (bits.tobytes(), int(total), res["err"].astype(np.float32).tobytes())
    return out


def test_sharded_job_gives_every_matrix_its_single_process_result():
    """Rows and budgets of different matrices never mix: whichever rank takes a matrix, its error
    table and allocation are those of a run that has all matrices in one process."""
    shapes = [(48, 160), (32, 96), (64, 64), (16, 200), (40, 128)]
    res = _run_ranks(_rank_pipeline, 2, shapes, 77)
    merged = {}
    for r in res:
        assert not (set(r) & set(merged))
        merged.update(r)
    assert sorted(merged) == list(range(len(shapes)))
    single = _rank_pipeline(0, 1, shapes, 77)
    assert merged == single


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert p.returncode == 0 and p.stdout.strip() == ""
    env["RANK"] = env["LOCAL_RANK"] = "0"
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0, p.stderr[-400:]
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["unit"] == "rows/s"
    assert line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
