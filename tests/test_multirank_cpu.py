"""The N>1 host logic on two gloo ranks (CPU): column shards tile the parameter range, every rank
derives identical finished counts / masks / MATCHA activation words from the host library without
talking to the others, timing is combined as the max over ranks, and - because columns never
interact - a column-sharded oracle run equals the unsharded one."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import nb_oracle as O
    from paper_2211_00889_b200 import binding as B
    from paper_2211_00889_b200 import sharding as S
    from paper_2211_00889_b200 import workloads as WL

    res = {}
    # (1) every rank computes the same counts / activation words on its own
    w = WL.WORKLOADS["cfg4_matcha_vgg16"]
    topo, _ = B.make_topology("random_regular", degree=w.degree, seed=w.seed, alpha=w.alpha, act_prob=w.act_prob)
    agree = True
    for t in range(50):
        n, mask, _ = B.straggler_sample(w.straggler_model, w.seed, t, w.K, w.M, w.straggler_params)
        agree &= S.counts_agree(n)
        agree &= S.counts_agree(mask.reshape(-1))
        _, bits = B.mixing_matrix(topo, B.NB_MATCHA, w.K, t)
        agree &= S.counts_agree(np.array([bits]))
    res["agree"] = bool(agree)
    # a rank that disagrees is detected
    res["detects_mismatch"] = not S.counts_agree(np.array([1, 2, 3 + rank]))
    # (2) timing: max over ranks
    res["tmax"] = S.max_over_ranks(1.0 + rank)
    S.barrier()
    # (3) shards of a ragged range
    P = 3 * 512 * 5 + 77
    res["shard"] = S.column_shard(P, world, rank)
    # (4) sharded oracle == full oracle on the shard's columns
    ws = WL.scaled(WL.WORKLOADS["cfg3_dpsgd_ring_resnet50"], 4 * 512 + 33, steps=3)
    c0, c1 = S.column_shard(ws.P, world, rank)
    full = O.Oracle(ws.K, ws.P, ws.M, ws.lr, ws.mom, "dpsgd", W=O.ring_W(ws.K))
    part = O.Oracle(ws.K, c1 - c0, ws.M, ws.lr, ws.mom, "dpsgd", W=O.ring_W(ws.K))
    x0 = WL.init_params(ws)
    full.set_params(x0)
    part.set_params(x0[c0:c1])
    for t in range(ws.steps):
        n = O.straggler_counts(ws.straggler_model, ws.seed, t, ws.K, ws.M, ws.straggler_params)
        G = WL.gradients_np(ws, t)[1]
        full.step(G, n)
        part.step(G[:, :, c0:c1], n)
    res["shard_equals_full"] = bool(np.array_equal(full.X[:, c0:c1], part.X))
    torch.save(res, os.path.join(out_dir, "rank%d.pt" % rank))
    dist.destroy_process_group()


def test_two_gloo_ranks(tmp_path):
    from paper_2211_00889_b200.build import build_library
    build_library()
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    res = [torch.load(os.path.join(str(tmp_path), "rank%d.pt" % r)) for r in range(world)]
    assert all(r["agree"] for r in res)
    assert all(r["detects_mismatch"] for r in res)
    assert [r["tmax"] for r in res] == [2.0, 2.0]
    assert all(r["shard_equals_full"] for r in res)
    (a0, a1), (b0, b1) = res[0]["shard"], res[1]["shard"]
    P = 3 * 512 * 5 + 77
    assert a0 == 0 and a1 == b0 and b1 == P and a1 % 512 == 0
    assert abs((a1 - a0) - (b1 - b0 - 77)) <= 512


def test_column_shards_tile_any_range():
    from paper_2211_00889_b200.sharding import column_shard
    for P in (0, 1, 511, 512, 513, 25_600_000, 138_000_000, 124_000_001):
        for world in (1, 2, 3, 4, 8):
            edges = [column_shard(P, world, r) for r in range(world)]
            assert edges[0][0] == 0 and edges[-1][1] == P
            for (a0, a1), (b0, b1) in zip(edges, edges[1:]):
                assert a1 == b0 and a0 <= a1
            sizes = [(b - a) // 512 for a, b in edges]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        column_shard(10, 2, 2)
