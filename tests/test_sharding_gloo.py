"""Host side of the multi-GPU benchmark path, run as two gloo ranks on the CPU.

The path shards over independent permutations only (one replica per rank, no
collective on the data path), so what has to hold is: every rank builds its own
seeded permutation, different from the other ranks' and reproducible; the timing
all ranks report is the slowest rank's; the job value counts every rank's elements."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out_dir: str) -> None:
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    bench.WORKLOADS["tiny"] = (12, 1, 8, 2, "test: 1 x N=2^12")
    bench.WORKLOADS["tinyb"] = (8, 16, 4, 0, "test: 16 x N=2^8")
    perm, x = bench.make_inputs("tiny", rank)
    permb, _ = bench.make_inputs("tinyb", rank)
    # this rank pretends to need (rank + 1) ms per step
    ms = bench.max_over_ranks([1.0 + rank, 10.0 - rank], dist, "cpu")
    np.save(os.path.join(out_dir, "perm%d.npy" % rank), perm)
    np.save(os.path.join(out_dir, "permb%d.npy" % rank), permb)
    np.save(os.path.join(out_dir, "ms%d.npy" % rank), np.array(ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_get_their_own_permutations_and_the_slowest_time(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    perms = [np.load(tmp_path / ("perm%d.npy" % r)) for r in range(world)]
    permbs = [np.load(tmp_path / ("permb%d.npy" % r)).reshape(16, 256) for r in range(world)]
    for p in perms:
        assert np.array_equal(np.sort(p), np.arange(1 << 12))
    assert not np.array_equal(perms[0], perms[1])
    # batched workload: 16 permutations per rank, no seed used twice across ranks
    rows = {pb.tobytes() for pbs in permbs for pb in pbs}
    assert len(rows) == 32
    for pbs in permbs:
        for pb in pbs:
            assert np.array_equal(np.sort(pb), np.arange(256))
    # the same seeds give the same inputs again
    from paper_1912_04050_b200 import inputs
    assert np.array_equal(perms[1], inputs.random_perm(12, 2 + 1))
    # max over ranks, identical on every rank
    for r in range(world):
        assert np.load(tmp_path / ("ms%d.npy" % r)).tolist() == [2.0, 10.0]


def test_job_value_counts_every_replica():
    import bench
    assert bench.whole_job_value(1 << 20, 1, 2.0) == (1 << 20) / 2e-3
    assert bench.whole_job_value(1 << 20, 8, 2.0) == 8 * (1 << 20) / 2e-3


def test_plain_start_with_gpus_2_spawns_two_ranks():
    """`python bench.py --gpus 2` without torchrun's variables must start the two ranks itself;
    driven here through the CPU rank check (gloo): one line, n_gpus = 2, the slowest rank's
    time, every replica counted, a different permutation on each rank."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items()
           if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--rank-check",
                          "--workload", "c1"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["ms_per_step"] == 2.0
    assert line["value"] == 2 * (1 << 10) / 2e-3
    assert len(set(line["rank_inputs"])) == 2


def test_gpus_must_match_the_world_size():
    import subprocess
    env = dict(os.environ, RANK="0", LOCAL_RANK="0", WORLD_SIZE="1", MASTER_ADDR="127.0.0.1",
               MASTER_PORT=str(_free_port()))
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--rank-check",
                          "--workload", "c1"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode != 0 and "WORLD_SIZE" in out.stderr


def test_batch_slices_cover_the_batch_once():
    from paper_1912_04050_b200 import binding, build
    build.build()
    for batch, world in ((16384, 8), (5, 8), (7, 3), (1, 1), (1000, 7)):
        slices = [binding.benes_shard_batch(batch, world, r) for r in range(world)]
        assert slices[0][0] == 0
        for (f0, c0), (f1, _) in zip(slices, slices[1:]):
            assert f1 == f0 + c0
        assert slices[-1][0] + slices[-1][1] == batch
        counts = [c for _, c in slices]
        assert max(counts) - min(counts) <= 1
    with pytest.raises(binding.BenesError):
        binding.benes_shard_batch(4, 2, 2)
