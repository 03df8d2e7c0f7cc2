"""bench.py's N > 1 control flow on a box with one GPU: two ranks share the device and meet over gloo
(a measurement needs one GPU per rank and NCCL; this only checks barriers, the max over ranks, the
aggregate and that rank 0 alone prints)."""
import json
import os
import socket
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_two_ranks_print_one_aggregated_line():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    env = dict(os.environ, ADACOMP_BENCH_BACKEND="gloo", ADACOMP_BENCH_SHARE_GPU="1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "2",
           "--warmup", "1", "--log2n", "22", "--no-cpu", "--no-e2e"]
    out = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-3000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, out.stdout[-2000:]
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["scaling"] == "weak" and d["device_status"] == 0
    # the aggregate counts both ranks' gradients: value = 2 ranks x 4 learners x 4n bytes / slowest rank's time
    n, k = d["config"]["n"], d["config"]["learners_per_gpu"]
    assert d["value"] == pytest.approx(2 * k * 4.0 * n / (d["ms_per_step"] * 1e-3) / 1e9, rel=1e-6)
    for key in ("roofline", "clocks", "gpu_launches", "lazy_scale", "fused_update"):
        assert key in d
