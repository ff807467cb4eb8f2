"""The N > 1 path on CPU: two gloo ranks shard a batch, run the oracle's forward and backward on
their shards, and exchange only the LCE weight gradients.  The result must equal the
single-process oracle on the whole batch: images are independent (no forward collective), and
d_lce_w / d_lce_b are plain sums over the batch."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import bra_oracle as orc
from paper_2303_08810_b200 import sharding, synthetic
from paper_2303_08810_b200.synthetic import BraConfig

CFG = BraConfig("two-ranks", 5, 8, 8, 32, 2, 2, 2, "f32")


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        x = synthetic.make_inputs(CFG, seed=3, with_do=True)
        lo, hi = sharding.shard_range(CFG.B, world, rank)
        q, k, v, do = (x[n][lo:hi] for n in ("Q", "K", "V", "dO"))
        O, index, _, _ = orc.bra_forward(q, k, v, x["w"], CFG.heads, CFG.S, CFG.topk)
        dq, dk, dv, dw, db = orc.bra_backward(q, k, v, index, x["w"], do, CFG.heads, CFG.S)
        tw, tb = torch.from_numpy(np.ascontiguousarray(dw)), torch.from_numpy(np.ascontiguousarray(db))
        sharding.allreduce_lce_grads(tw, tb)
        slowest = sharding.max_over_ranks(1.0 + rank)
        np.savez(os.path.join(out_dir, f"rank{rank}.npz"), O=O, dq=dq, dk=dk, dv=dv, dw=tw.numpy(),
                 db=tb.numpy(), lo=lo, hi=hi, slowest=slowest)
    finally:
        dist.destroy_process_group()


def test_shard_range_covers_the_batch_once():
    for B in (1, 2, 5, 64):
        for world in (1, 2, 3, 8):
            spans = [sharding.shard_range(B, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == B
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.shard_range(4, 2, 2)


def test_two_gloo_ranks_reproduce_the_whole_batch(tmp_path):
    world = 2
    mp.spawn(worker, args=(world, free_port(), str(tmp_path)), nprocs=world, join=True)
    x = synthetic.make_inputs(CFG, seed=3, with_do=True)
    O, index, _, _ = orc.bra_forward(x["Q"], x["K"], x["V"], x["w"], CFG.heads, CFG.S, CFG.topk)
    dq, dk, dv, dw, db = orc.bra_backward(x["Q"], x["K"], x["V"], index, x["w"], x["dO"], CFG.heads, CFG.S)
    parts = [np.load(tmp_path / f"rank{r}.npz") for r in range(world)]
    assert [int(p["lo"]) for p in parts] == [0, 3] and [int(p["hi"]) for p in parts] == [3, 5]
    for name, full in (("O", O), ("dq", dq), ("dk", dk), ("dv", dv)):
        np.testing.assert_allclose(np.concatenate([p[name] for p in parts]), full, rtol=0, atol=1e-12)
    for p in parts:                       # every rank holds the batch-wide sums after the all-reduce
        np.testing.assert_allclose(p["dw"], dw, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(p["db"], db, rtol=1e-12, atol=1e-12)
        assert float(p["slowest"]) == 2.0
