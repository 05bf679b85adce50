"""Multi-GPU path = row sharding with no exchange step.  The host logic (which rank owns which rows) is
checked here with two gloo ranks on CPU: each rank evaluates its shard with the oracle, the shards are
gathered, and the result must equal the unsharded layer bit for bit (rows are independent)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle as O
from paper_2507_14811_b200 import workloads as WL
from paper_2507_14811_b200.layer import shard_rows


def test_shard_rows_partitions_exactly():
    for M in [0, 1, 7, 128, 8858, 32768]:
        for world in [1, 2, 3, 4, 8]:
            spans = [shard_rows(M, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == M
            for a, b in zip(spans, spans[1:]):
                assert a[1] == b[0]
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1


def _layer(spec, data, rows):
    X = data.X.float().numpy()[rows[0]:rows[1]]
    s_pos, s_neg = O.calib_act(data.X_cal.float().numpy(), spec.kb, spec.dual)
    s_w = O.calib_weight(data.W.numpy(), spec.kb, spec.nb)
    Wq = O.quantize_weight(data.W.numpy(), spec.kb, spec.nb, s_w)
    if X.shape[0] == 0:
        return np.zeros((0, spec.N))
    return O.layer_forward(X, Wq, O.SegTable(spec.kb, spec.nb), s_pos, s_neg, s_w, data.bias.numpy()).y64


def _worker(rank, world, port, out_path):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    spec = WL.small_variant(WL.WORKLOADS["sdxl_skip"][0], 37, 64, 24)
    data = WL.make_layer(spec)                        # same seed on every rank: replicated weights
    r0, r1 = shard_rows(spec.M, rank, world)
    y = torch.from_numpy(_layer(spec, data, (r0, r1)))
    pad = torch.zeros((spec.M, spec.N), dtype=torch.float64)
    pad[r0:r1] = y
    dist.all_reduce(pad)                               # test-side gather; the product path has no collective
    if rank == 0:
        full = _layer(spec, data, (0, spec.M))
        np.save(out_path, np.array([float(np.array_equal(pad.numpy(), full))]))
    dist.destroy_process_group()


def test_two_gloo_ranks_reproduce_the_unsharded_layer(tmp_path):
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    out = str(tmp_path / "ok.npy")
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    assert np.load(out)[0] == 1.0
