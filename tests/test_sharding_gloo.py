"""Window sharding over two CPU ranks (gloo): partition arithmetic, the score all-gather and the
global selection agree with the single-process result.  The selection callable injected here is the
oracle's (CPU); on GPUs the CUDA library's selection is used with the same plumbing."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2605_14978_b200 import sharding as S
from paper_2605_14978_b200 import workloads as W


def test_window_range_partitions_exactly():
    for n_total in (0, 1, 7, 64, 65, 2048, 4099):
        for world in (1, 2, 3, 4, 8):
            ranges = [S.window_range(n_total, world, r) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == n_total
            assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
            sizes = S.shard_sizes(n_total, world)
            assert max(sizes) - min(sizes) <= 1 and sum(sizes) == n_total
            for i in sorted({0, n_total // 2, n_total - 1} & set(range(n_total))):
                r, loc = S.owner_of(i, n_total, world)
                assert ranges[r][0] + loc == i and 0 <= loc < sizes[r]
    with pytest.raises(ValueError):
        S.window_range(10, 2, 2)
    with pytest.raises(ValueError):
        S.owner_of(10, 10, 2)


def _oracle_select(scores, n_keep):
    return torch.from_numpy(oracle.select_windows(scores.double().numpy(), n_keep).astype(np.int64))


def _scores_of(w, lo, hi):
    """Oracle window scores of windows [lo, hi) of workload w (generated chunk-wise, so shards line up)."""
    x = W.generate(w, "cpu")
    o = oracle.score_windows(x["draft_logits"][lo:hi], x["target_logits"][lo:hi], x["draft_tokens"][lo:hi],
                             mode=oracle.GREEDY, c=w.c, temperature=w.temperature, n_threads=2)
    return torch.from_numpy(o["score"]).float()


def _worker(rank, world, port, n_total, n_keep, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = W.scaled(W.WORKLOADS[0], n_total)
        lo, hi = S.window_range(n_total, world, rank)
        local = _scores_of(w, lo, hi)
        gathered = S.gather_scores(local, n_total)
        sel, sel_local = S.sharded_select(local, n_total, n_keep, select_fn=_oracle_select)
        ret[rank] = (gathered.numpy().copy(), sel.numpy().copy(), sel_local.numpy().copy(), lo, hi)
        with pytest.raises(ValueError):
            S.gather_scores(local[:-1], n_total)          # a shard of the wrong length is refused before any collective
    finally:
        dist.destroy_process_group()


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


@pytest.mark.parametrize("n_total,n_keep", [(64, 16), (65, 17)])    # equal shards, ragged shards
def test_two_rank_selection_matches_single_process(n_total, n_keep):
    world = 2
    ret = mp.Manager().dict()
    mp.spawn(_worker, args=(world, _free_port(), n_total, n_keep, ret), nprocs=world, join=True)
    w = W.scaled(W.WORKLOADS[0], n_total)
    full = _scores_of(w, 0, n_total).numpy()
    want = oracle.select_windows(full.astype(np.float64), n_keep)
    seen = []
    for rank in range(world):
        gathered, sel, sel_local, lo, hi = ret[rank]
        np.testing.assert_array_equal(gathered, full)                   # shards land in window order
        np.testing.assert_array_equal(sel, want)                        # every rank holds the same selection
        np.testing.assert_array_equal(sel_local + lo, [i for i in want if lo <= i < hi])
        seen.extend((sel_local + lo).tolist())
    assert sorted(seen) == sorted(want.tolist())                        # each kept window has exactly one owner
