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


# --------------------------------------------------------------------------
# exchange(): all-gather of variable-length packed streams (Algorithm 1), three gloo ranks on the CPU.
# Every rank packs its own gradient with the oracle, exchanges, and decodes all streams with the
# oracle: the dense sum must be the one computed from all three gradients in rank order, and the
# fused average + SGD step must leave identical weights on every rank.
# --------------------------------------------------------------------------

EXCHANGE_WORKER = textwrap.dedent("""
    import sys, zlib
    sys.path.insert(0, {root!r})
    import numpy as np
    import torch
    import torch.distributed as dist
    from oracle import cref
    from paper_1712_02679_b200 import ranks
    from paper_1712_02679_b200.exchange import exchange, padded_size
    rank, world, local = ranks.rank_env()
    dist.init_process_group("gloo")
    n, L_T = 20011, 50
    def grad(r, step):
        g = np.random.default_rng(ranks.learner_seed(r, 0, step)).normal(0, 1e-3 * (1 + r), n).astype(np.float32)
        if r == 2:
            g[:4000] = 0          # rank 2 sends fewer words: the streams differ in length
        return g
    residues = [np.zeros(n, np.float32) for _ in range(world)]      # every rank replays all learners to know the truth
    w = np.linspace(-1, 1, n, dtype=np.float32)
    v = np.zeros(n, np.float32)
    w_true, v_true = w.copy(), v.copy()
    cap = cref.stream_bytes(n, L_T, n)
    recv = None
    for step in range(3):
        all_streams = [cref.pack(grad(r, step), residues[r], L_T).raw for r in range(world)]
        mine = all_streams[rank]
        buf = torch.full((cap,), 0xAB, dtype=torch.uint8)
        buf[:mine.size] = torch.from_numpy(mine.copy())
        if recv is None:
            recv = torch.empty(world * cap, dtype=torch.uint8)
        got = exchange(buf, mine.size, recv=recv)
        assert len(got) == world
        for r in range(world):
            assert got[r].numel() == all_streams[r].size, (r, got[r].numel(), all_streams[r].size)
            assert np.array_equal(got[r].numpy(), all_streams[r]), r
            assert got[r].data_ptr() % 16 == 0
        assert len(set(s.size for s in all_streams)) > 1, "streams were meant to differ in length"
        streams = [g.numpy() for g in got]
        w, v = cref.average_sgd(streams, n, w, v, 0.1, 0.9)
        w_true, v_true = cref.average_sgd(all_streams, n, w_true, v_true, 0.1, 0.9)
    assert np.array_equal(w.view(np.uint32), w_true.view(np.uint32))
    # all ranks hold the same weights
    crc = torch.tensor([zlib.crc32(w.tobytes())], dtype=torch.int64)
    both = torch.empty(world, dtype=torch.int64)
    dist.all_gather_into_tensor(both, crc)
    assert len(set(int(c) for c in both)) == 1
    assert padded_size([1, 17, 16]) == 32 and padded_size([]) == 0
    if rank == 0:
        print("EXCHANGE_OK", int(crc))
    dist.barrier()
    dist.destroy_process_group()
""")


def test_exchange_three_gloo_ranks(tmp_path):
    script = tmp_path / "exchange_worker.py"
    script.write_text(EXCHANGE_WORKER.format(root=ROOT))
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(3):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="3", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=180) for p in procs]
    for p, (out, err) in zip(procs, outs):
        assert p.returncode == 0, err[-3000:]
    assert "EXCHANGE_OK" in outs[0][0]


def test_exchange_without_a_process_group_is_the_identity():
    import torch
    from paper_1712_02679_b200.exchange import exchange
    buf = torch.arange(64, dtype=torch.uint8)
    got = exchange(buf, 40)
    assert len(got) == 1 and got[0].numel() == 40 and got[0].data_ptr() == buf.data_ptr()
    with pytest.raises(ValueError):
        exchange(buf, 65)
    with pytest.raises(ValueError):
        exchange(buf.to(torch.int32), 4)
