"""Measurement aids of the library: the read-only streaming probe and the launch-count query."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

from paper_2605_14978_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("n_bytes", [16, 4096, 16 * 1000003, 64 << 20])
def test_stream_read_probe_folds_every_word(n_bytes):
    g = torch.Generator(device=DEV).manual_seed(n_bytes % 1000)
    data = torch.randint(-2 ** 31, 2 ** 31 - 1, (n_bytes // 4,), generator=g, device=DEV, dtype=torch.int32)
    checksum = torch.full((1,), 12345, dtype=torch.int32, device=DEV)        # cleared by the call
    B.ppow_stream_read_probe(data, checksum)
    torch.cuda.synchronize()
    want = np.bitwise_xor.reduce(data.cpu().numpy().view(np.uint32))
    assert int(checksum.cpu().numpy().view(np.uint32)[0]) == int(want)       # every word was read exactly once
    with pytest.raises(B.PpowError):
        B.ppow_stream_read_probe(data[1:], checksum)                         # not 16-byte aligned / sized


def test_launch_count_query_names_the_one_launch_path():
    assert B.ppow_score_kernel_launches(B.make_params(64, 4, 1000, B.PPOW_F32, B.PPOW_GREEDY, 0.05)) == 1
    assert B.ppow_score_kernel_launches(B.make_params(2048, 8, 128256, B.PPOW_BF16, B.PPOW_STOCHASTIC, 0.04)) == 2
    assert B.ppow_score_kernel_launches(B.make_params(132, 4, 1000, B.PPOW_F32, B.PPOW_GREEDY, 0.05)) == 2
    assert B.ppow_score_kernel_launches(B.make_params(64, 40, 1000, B.PPOW_F32, B.PPOW_GREEDY, 0.05)) == 0


def test_timeline_build_records_every_warp_and_the_ordinary_library_declines():
    status, _ = B.ppow_timeline_read(8)
    assert status == B.PPOW_ERR_UNSUPPORTED
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, PPOW_LIBRARY="timeline")
    res = subprocess.run([sys.executable, "-m", "paper_2605_14978_b200.timeline", "llama3_like:64"], capture_output=True,
                         text=True, timeout=900, env=env, cwd=root)
    assert res.returncode == 0, res.stderr[-2000:]
    assert "== llama3_like:64: 2368 warps" in res.stdout and "start to first data" in res.stdout, res.stdout[-2000:]
