"""The multi-GPU plumbing's GPU branch on the one GPU there is: a one-rank NCCL process group runs the score
all-gather (`all_gather_into_tensor` on CUDA tensors) and the library's selection on the gathered scores; and the
benchmark launched by torch.distributed.run with one rank (gather on) selects the same windows as the plain run."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest
import torch

import oracle
from paper_2605_14978_b200 import sharding as S

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.fixture()
def nccl_group():
    import torch.distributed as dist
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", init_method="tcp://127.0.0.1:%d" % _free_port(), rank=0, world_size=1)
    yield dist
    dist.destroy_process_group()


@pytest.mark.parametrize("n_total,n_keep", [(2048, 512), (777, 78), (5, 5), (40000, 4000)])
def test_sharded_select_on_a_one_rank_nccl_group(nccl_group, n_total, n_keep):
    g = torch.Generator(device="cuda:0").manual_seed(n_total)
    score = torch.rand(n_total, generator=g, device="cuda:0")
    score[::7] = score[3]                                            # ties: lower index first
    gathered = S.gather_scores(score, n_total)
    assert gathered.is_cuda and torch.equal(gathered, score)
    selected, local = S.sharded_select(score, n_total, n_keep)       # default selection: the CUDA library's
    torch.cuda.synchronize()
    want = oracle.select_windows(score.cpu().numpy().astype(np.float64), n_keep)
    np.testing.assert_array_equal(selected.cpu().numpy(), want)
    np.testing.assert_array_equal(local.cpu().numpy(), want)         # one rank owns every window


def _bench_line(cmd, env=None):
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=900, env=env, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-3000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.strip().startswith("{")]
    assert len(lines) == 1
    return json.loads(lines[0])


def test_bench_under_torchrun_with_one_rank_selects_the_same_windows_as_the_plain_run():
    args = ["bench.py", "--windows", "192", "--steps", "3", "--warmup", "3", "--no-e2e", "--no-cpu-baseline",
            "--no-sustained", "--no-workloads", "--no-probe"]
    plain = _bench_line([sys.executable] + args)
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    spawned = _bench_line([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "1",
                           "--master-addr", "127.0.0.1", "--master-port", str(_free_port())] + args + ["--gpus", "1"], env)
    assert plain["score_exchange"].startswith("none") and spawned["score_exchange"].startswith("all_gather")
    assert spawned["selected_checksum"] == plain["selected_checksum"] and plain["selected_checksum"] > 0
    assert spawned["n_gpus"] == 1 and spawned["config"] == plain["config"]
