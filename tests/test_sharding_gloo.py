"""The N > 1 path on CPU: two gloo ranks shard a packed batch by sequence, each evaluates its shard alone
(with the oracle standing in for the device), and the pieces put side by side equal the whole-batch result:
sequences are independent, so the path needs no data-path collective (Section 3.2: the hook acts per token
and head; the attention per sequence).  Also covers the timing bookkeeping bench.py uses across ranks."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2603_01281_b200 import inputs, sharding


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = inputs.make_custom(seed=41, dtype="bf16", lens=[70, 33, 0, 129, 5], n_q_heads=4, n_kv_heads=2, head_dim=64,
                               rank=8, gain=[0.5, 1.0, 2.0, -0.5, 1.5], mask_kind="runs", highlight=0.3)
        t0, t1, cu = sharding.shard_tokens(w.cu_seqlens, world, rank)
        first, last = sharding.shard_sequences(w.batch, world, rank)
        O, lse, _ = oracle.seka_attention(w.Q[t0:t1], w.K[t0:t1], w.V[t0:t1], w.mask[t0:t1], np.asarray(cu, dtype=np.int32),
                                          w.U, gain=w.gain[first:last])
        np.save(os.path.join(out_dir, "O_%d.npy" % rank), O)
        # the decode step over the (edited) cache shards by sequence in the same way
        q = np.stack([w.Q[c - 1] if c > w.cu_seqlens[i] else np.zeros_like(w.Q[0])
                      for i, c in enumerate(w.cu_seqlens[1:])])
        Od, _ = oracle.seka_decode(q[first:last], w.K[t0:t1], w.V[t0:t1], w.mask[t0:t1], cu, w.U, gain=w.gain[first:last])
        np.save(os.path.join(out_dir, "Od_%d.npy" % rank), Od)
        # the offline learner shards by slot
        h, hp, hn, ans, _, _ = inputs.contrastive_embeddings(seed=2, n=300, slots=6, head_dim=16, rank=3, dtype="f32")
        s0, s1 = sharding.shard_slots(6, world, rank, pair=True)
        res = oracle.learn_projections(h[:, s0:s1], hp[:, s0:s1], hn[:, s0:s1], 0.7, answer_tokens=ans)
        np.save(os.path.join(out_dir, "S_%d.npy" % rank), np.concatenate([res["S_pos"], res["D"][:, None]], axis=1))
        # timing bookkeeping: the slowest rank decides, every rank learns it
        slow = sharding.max_over_ranks(10.0 + rank)
        assert slow == 10.0 + world - 1
        sharding.barrier()
        rate = sharding.whole_job_rate(units_per_rank_step=100.0, steps=4, ms=slow, world=world)
        assert abs(rate - world * 100.0 * 4 / (slow * 1e-3)) < 1e-6
        # the ranks' batches of the weak-scaling bench differ
        assert sharding.rank_seed_offset(rank) == rank
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_by_sequence_without_exchange(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    w = inputs.make_custom(seed=41, dtype="bf16", lens=[70, 33, 0, 129, 5], n_q_heads=4, n_kv_heads=2, head_dim=64,
                           rank=8, gain=[0.5, 1.0, 2.0, -0.5, 1.5], mask_kind="runs", highlight=0.3)
    whole, _, _ = oracle.seka_attention(w.Q, w.K, w.V, w.mask, w.cu_seqlens, w.U, gain=w.gain)
    parts = np.concatenate([np.load(tmp_path / ("O_%d.npy" % r)) for r in range(world)], axis=0)
    assert parts.shape == whole.shape
    assert np.array_equal(parts, whole)         # the same arithmetic on the same rows: bit-identical
    q = np.stack([w.Q[c - 1] if c > w.cu_seqlens[i] else np.zeros_like(w.Q[0]) for i, c in enumerate(w.cu_seqlens[1:])])
    whole_d, _ = oracle.seka_decode(q, w.K, w.V, w.mask, w.cu_seqlens, w.U, gain=w.gain)
    parts_d = np.concatenate([np.load(tmp_path / ("Od_%d.npy" % r)) for r in range(world)], axis=0)
    assert np.array_equal(parts_d, whole_d)
    h, hp, hn, ans, _, _ = inputs.contrastive_embeddings(seed=2, n=300, slots=6, head_dim=16, rank=3, dtype="f32")
    res = oracle.learn_projections(h, hp, hn, 0.7, answer_tokens=ans)
    parts_s = np.concatenate([np.load(tmp_path / ("S_%d.npy" % r)) for r in range(world)], axis=0)
    assert np.array_equal(parts_s, np.concatenate([res["S_pos"], res["D"][:, None]], axis=1))


def test_slot_ranges_partition_the_slots():
    for n in (2, 6, 288):
        for world in (1, 2, 4, 8):
            for pair in (False, True):
                r = [sharding.shard_slots(n, world, k, pair=pair) for k in range(world)]
                assert r[0][0] == 0 and r[-1][1] == n and all(r[k][1] == r[k + 1][0] for k in range(world - 1))
                assert not pair or all(a % 2 == 0 and b % 2 == 0 for a, b in r)


def test_shard_ranges_partition_the_batch():
    for n in (0, 1, 5, 8, 13):
        for world in (1, 2, 3, 8):
            ranges = [sharding.shard_sequences(n, world, r) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
            sizes = [b - a for a, b in ranges]
            assert max(sizes) - min(sizes) <= 1
    t0, t1, cu = sharding.shard_tokens([0, 4, 9, 9, 20], 2, 1)
    assert (t0, t1, cu) == (9, 20, [0, 0, 11])
