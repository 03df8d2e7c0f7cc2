"""Rank logic of the N > 1 runs, on two gloo ranks on the CPU (no GPU, no NCCL)."""
import os
import socket
import subprocess
import sys
import textwrap

import pytest

from paper_1712_02679_b200 import ranks

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_shards_cover_every_unit_once():
    for n_units in (0, 1, 7, 8, 161):
        for world in (1, 2, 3, 8):
            got = [u for r in range(world) for u in ranks.shard_units(n_units, world, r)]
            assert got == list(range(n_units))
            sizes = [len(ranks.shard_units(n_units, world, r)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1


def test_seeds_never_collide_across_ranks_learners_steps():
    seen = set()
    for r in range(8):
        for l in range(16):
            for s in range(7):
                seen.add(ranks.learner_seed(r, l, s))
    assert len(seen) == 8 * 16 * 7


def test_single_process_defaults():
    assert ranks.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert ranks.whole_job_throughput(4e9, 2, 1000.0) == pytest.approx(8.0)


WORKER = textwrap.dedent("""
    import sys
    sys.path.insert(0, {root!r})
    import torch.distributed as dist
    from paper_1712_02679_b200 import ranks
    rank, world, local = ranks.rank_env()
    dist.init_process_group("gloo")
    assert (dist.get_rank(), dist.get_world_size()) == (rank, world) == (rank, 2)
    dist.barrier()
    # each rank "measured" different times; both must agree on the slowest
    mine = [10.0 + rank, 5.0 - rank, 1.0]
    got = ranks.max_over_ranks(mine)
    assert got == [11.0, 5.0, 1.0], got
    # units split without overlap, seeds differ between the ranks
    units = list(ranks.shard_units(161, world, rank))
    assert len(units) in (80, 81) and (units[0] == 0) == (rank == 0)
    assert ranks.learner_seed(rank, 0, 0) != ranks.learner_seed(1 - rank, 0, 0)
    gbs = ranks.whole_job_throughput(4.0 * 2**30 * 4, world, got[0])
    if rank == 0:
        print("RESULT", round(gbs, 3))
    dist.barrier()
    dist.destroy_process_group()
""")


def test_two_gloo_ranks_agree_on_the_slowest_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (out, err) in zip(procs, outs):
        assert p.returncode == 0, err[-2000:]
    want = 4.0 * 2**30 * 4 * 2 / (11.0e-3) / 1e9
    assert f"RESULT {round(want, 3)}" in outs[0][0]
    assert "RESULT" not in outs[1][0]


def test_reference_arm_prints_only_on_rank_zero():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""
