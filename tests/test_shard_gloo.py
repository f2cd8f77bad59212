"""The N > 1 host logic on CPU: two gloo ranks shard one layer by KV-head group, each runs the (oracle)
path on its shard only, and the gathered lists equal the unsharded ones; timings reduce as max, work as sum."""
import os

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2607_25291_b200.shard import kv_head_shard, reduce_job, shard_tensors


def test_shards_partition_the_heads():
    for hq, hkv in ((32, 8), (4, 1), (12, 3), (8, 8)):
        for world in (1, 2, 3, 4, 8):
            seen_kv, seen_q = [], []
            for r in range(world):
                a, b, c, d = kv_head_shard(hq, hkv, world, r)
                assert (c, d) == (a * (hq // hkv), b * (hq // hkv))
                seen_kv += list(range(a, b)); seen_q += list(range(c, d))
            assert seen_kv == list(range(hkv)) and seen_q == list(range(hq))
            sizes = [kv_head_shard(hq, hkv, world, r)[1] - kv_head_shard(hq, hkv, world, r)[0] for r in range(world)]
            assert max(sizes) - min(sizes) <= 1


def _worker(rank, world, port, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import cosa_oracle as O
    from synth.configs import tiny
    from synth.generator import bf16_bits_to_f64
    qb, kb, vb, _ = tiny(seed=5, hq=4, hkv=2, n=512, needles=1).make()
    q, k, v = (bf16_bits_to_f64(x)[None] for x in (qb, kb, vb))
    qs, ks, vs = shard_tensors(q, k, v, world, rank)
    order, count = O.kap_select(qs[0], ks[0], s=8, budget=0.5, order_stride=4)
    r = O.osk_attention(qs[0], ks[0], vs[0], order, count, skip_scale=100.0, tightened_budget=0.4)
    gathered = [None] * world
    dist.all_gather_object(gathered, (order, count, r["visited"]))
    ms, units = reduce_job(10.0 + rank, float(r["visited"].sum()))
    if rank == 0:
        ret["order"] = np.concatenate([g[0] for g in gathered]); ret["count"] = np.concatenate([g[1] for g in gathered])
        ret["visited"] = np.concatenate([g[2] for g in gathered]); ret["ms"] = ms; ret["units"] = units
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_reproduce_the_unsharded_result():
    from oracle import cosa_oracle as O
    from synth.configs import tiny
    from synth.generator import bf16_bits_to_f64
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        ret = mgr.dict()
        mp.spawn(_worker, args=(2, port, ret), nprocs=2, join=True)
        got = dict(ret)
    qb, kb, vb, _ = tiny(seed=5, hq=4, hkv=2, n=512, needles=1).make()
    q, k, v = (bf16_bits_to_f64(x) for x in (qb, kb, vb))
    order, count = O.kap_select(q, k, s=8, budget=0.5, order_stride=4)
    r = O.osk_attention(q, k, v, order, count, skip_scale=100.0, tightened_budget=0.4)
    assert np.array_equal(got["order"], order) and np.array_equal(got["count"], count)
    assert np.array_equal(got["visited"], r["visited"])
    assert got["ms"] == 11.0 and got["units"] == float(r["visited"].sum())
