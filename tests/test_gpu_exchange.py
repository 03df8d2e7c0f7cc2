"""exchange() between ranks that pack and decode with the CUDA library (Algorithm 1, "Computation Steps":
pack(), exchange(), unpack(), averageGradients(), updateWeights()).

Three ranks share the one GPU and meet over gloo (the streams are staged through the host for the gather; on
a node with a GPU per rank the same code gathers device tensors over NCCL).  Every rank packs its own seeded
gradient with adacomp_compress, receives all three streams into its own memory, decodes them in rank order
with adacomp_decompress_accumulate_ex and applies adacomp_decompress_average_sgd.  Each rank also replays all
three learners with the CPU oracle and asserts: the bytes it received are the oracle's streams, the dense sum
is the oracle's, and after three steps every rank holds the same weights, the oracle's."""
import os
import socket
import subprocess
import sys
import textwrap

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import sys, zlib
    sys.path.insert(0, {root!r})
    import numpy as np
    import torch
    import torch.distributed as dist
    from oracle import cref
    from paper_1712_02679_b200 import binding as B
    from paper_1712_02679_b200 import ranks
    from paper_1712_02679_b200.exchange import exchange, exchange_v2
    rank, world, local = ranks.rank_env()
    dist.init_process_group("gloo")
    dev = torch.device("cuda", 0)            # every rank on the one GPU
    torch.cuda.set_device(dev)
    B.adacomp_set_device(0)
    for L_T, n in ((50, 4000 * 61 + 17), (500, 4000 * 23 + 5)):
        def grad(r, step):
            g = np.random.default_rng(ranks.learner_seed(r, L_T, step)).normal(0, 1e-3 * (1 + r), n).astype(np.float32)
            if r == 2:
                g[:8000] = 0                 # rank 2 sends fewer words: the streams differ in length
            return g
        oracle_res = [np.zeros(n, np.float32) for _ in range(world)]
        w_true = np.linspace(-1, 1, n, dtype=np.float32)
        v_true = np.zeros(n, np.float32)
        residue = torch.zeros(n, device=dev)
        cap = B.adacomp_packed_capacity(n, L_T)
        packed = torch.empty(cap, dtype=torch.uint8, device=dev)
        count = torch.zeros(2, dtype=torch.int64, device=dev)
        recv = torch.empty(world * cap, dtype=torch.uint8, device=dev)
        wire = torch.empty(B.adacomp_v2_capacity(n, L_T), dtype=torch.uint8, device=dev)
        recv_wire = torch.empty(world * wire.numel(), dtype=torch.uint8, device=dev)
        recv_packed = [torch.empty(cap, dtype=torch.uint8, device=dev) for _ in range(world)]
        w = torch.from_numpy(w_true.copy()).to(dev)
        v = torch.zeros(n, device=dev)
        dst = torch.empty(n, device=dev)
        for step in range(3):
            want = [cref.pack(grad(r, step), oracle_res[r], L_T).raw for r in range(world)]
            B.adacomp_compress(torch.from_numpy(grad(rank, step)).to(dev), residue, n, L_T, packed, count)
            torch.cuda.synchronize()
            got = exchange(packed, int(count[1]), recv=recv)
            assert len(got) == world and len(set(g.numel() for g in got)) > 1
            for r in range(world):
                assert got[r].is_cuda and got[r].data_ptr() % 16 == 0
                assert np.array_equal(got[r].cpu().numpy(), want[r]), (step, r)
            B.adacomp_decompress_accumulate_ex(got, world, dst, n, L_T)
            torch.cuda.synchronize()
            assert np.array_equal(dst.cpu().numpy().view(np.uint32), cref.unpack_sum(want, n).view(np.uint32)), step
            # the same exchange with version-2 streams on the wire: fewer bytes, the same streams on arrival
            streams2, wire_bytes = exchange_v2(packed, n, L_T, wire, recv_wire, recv_packed)
            for r in range(world):
                assert np.array_equal(streams2[r].cpu().numpy(), want[r]), (step, r)
                assert wire_bytes[r] == cref.to_v2(want[r]).size < want[r].size
            B.adacomp_decompress_accumulate_ex(streams2, world, dst, n, L_T)
            torch.cuda.synchronize()
            assert np.array_equal(dst.cpu().numpy().view(np.uint32), cref.unpack_sum(want, n).view(np.uint32)), step
            B.adacomp_decompress_average_sgd(got, world, w, v, n, L_T, 0.1, 0.9)
            torch.cuda.synchronize()
            w_true, v_true = cref.average_sgd(want, n, w_true, v_true, 0.1, 0.9)
        assert np.array_equal(residue.cpu().numpy().view(np.uint32), oracle_res[rank].view(np.uint32))
        assert np.array_equal(w.cpu().numpy().view(np.uint32), w_true.view(np.uint32))
        assert np.array_equal(v.cpu().numpy().view(np.uint32), v_true.view(np.uint32))
        crc = torch.tensor([zlib.crc32(w.cpu().numpy().tobytes())], dtype=torch.int64)
        every = torch.empty(world, dtype=torch.int64)
        dist.all_gather_into_tensor(every, crc)
        assert len(set(int(c) for c in every)) == 1
        assert B.adacomp_device_status() == 0
    if rank == 0:
        print("GPU_EXCHANGE_OK")
    dist.barrier()
    dist.destroy_process_group()
""")


def test_three_ranks_pack_exchange_decode_and_update_on_the_gpu(tmp_path):
    script = tmp_path / "gpu_exchange_worker.py"
    script.write_text(WORKER.format(root=ROOT))
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "3", "--master-addr",
           "127.0.0.1", "--master-port", str(port), str(script)]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    assert "GPU_EXCHANGE_OK" in out.stdout


def test_bench_exchange_workload_on_two_ranks_sharing_the_gpu():
    """bench.py --workload exchange: pack, all-gather, decode on every rank; here only its control flow (two
    ranks on the one GPU over gloo): one line, the sums agree across ranks, no device flag."""
    import json
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    env = dict(os.environ, ADACOMP_BENCH_BACKEND="gloo", ADACOMP_BENCH_SHARE_GPU="1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "2",
           "--warmup", "1", "--log2n", "22", "--workload", "exchange"]
    out = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-3000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, out.stdout[-2000:]
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["device_status"] == 0 and d["same_sum_on_every_rank"] is True
    assert d["config"]["exchange"].startswith("all-gather")
