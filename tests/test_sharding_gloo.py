"""Host side of the multi-GPU path on CPU: two gloo ranks each own a shard of the tensors, exchange
only the squared norm, and together reproduce the unsharded step bit for bit."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle as O
from paper_2608_11919_b200 import sharding as S
from paper_2608_11919_b200 import workloads as W

BLOCK = 2048


def test_partition_is_balanced_and_complete():
    spec = W.ragged_spec(n_tensors=300, max_numel=1 << 16, seed=2)
    for world in (1, 2, 3, 8):
        parts = S.partition_tensors(spec.sizes, world)
        assert sorted(i for p in parts for i in p) == list(range(300))
        loads = [sum(spec.sizes[i] for i in p) for p in parts]
        assert max(loads) - min(loads) <= max(spec.sizes)
        assert parts == S.partition_tensors(spec.sizes, world)      # deterministic
    dec = W.qwen3b_spec()
    loads = [sum(dec.sizes[i] for i in p) for p in S.partition_tensors(dec.sizes, 8)]
    assert max(loads) / (sum(loads) / 8) < 1.26                     # the tied embedding is 10 % of the model


def test_block_partition_is_balanced_to_one_block():
    for spec in (W.ragged_spec(n_tensors=300, max_numel=1 << 16, seed=2), W.qwen3b_spec(), W.dense27b_spec()):
        nbs = [(s + BLOCK - 1) // BLOCK for s in spec.sizes]
        for world in (1, 2, 3, 8):
            parts = S.partition_blocks(spec.sizes, BLOCK, world)
            flat = [x for p in parts for x in p]
            covered = {}
            for t, b0, nb in flat:                                  # every block exactly once, in list order
                assert nb > 0 and b0 == covered.get(t, 0)
                covered[t] = b0 + nb
            assert covered == {t: n for t, n in enumerate(nbs) if n}
            assert [x[0] for x in flat] == sorted(x[0] for x in flat)
            loads = [sum(nb for _, _, nb in p) for p in parts]
            assert max(loads) - min(loads) <= 1


def test_shard_specs_cover_one_list():
    """What `bench.py --scaling strong` gives each rank: together the ranks own every element exactly once."""
    for spec in (W.qwen3b_spec(), W.dense27b_spec()):
        for world in (2, 8):
            shards = [W.shard_spec(spec, BLOCK, r, world) for r in range(world)]
            assert sum(s.numel for s in shards) == spec.numel
            loads = [s.n_blocks(BLOCK) for s in shards]
            assert max(loads) - min(loads) <= 1 and sum(loads) == spec.n_blocks(BLOCK)
            per_name = {}
            for s in shards:
                for n, z in zip(s.names, s.sizes):
                    per_name[n] = per_name.get(n, 0) + z
            assert per_name == dict(zip(spec.names, spec.sizes))
            assert all(len(W.layer_groups(s, 8)) >= 1 for s in shards)


def _make(spec, step):
    buf = W.Buffers(spec, BLOCK, "cpu")
    W.fill_params(buf)
    W.fill_grads(buf, step)
    ts = [O.OracleTensor(W.numpy_view(buf.view("param", t)).copy(), W.numpy_view(buf.view("grad", t)).copy(), BLOCK)
          for t in range(len(spec.sizes))]
    return buf, ts


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        spec = W.ragged_spec(n_tensors=40, max_numel=1 << 13, seed=7)
        mine = S.partition_tensors(spec.sizes, world)[rank]
        hp = O.HParams(max_norm=0.5)
        _, ts = _make(spec, 1)
        local = [ts[i] for i in mine]
        out = {}
        for k in (1, 2):
            if k > 1:
                buf, _ = _make(spec, k)
                for i in mine:
                    ts[i].set_grad(W.numpy_view(buf.view("grad", i)).copy())
            s = torch.tensor([O.sqnorm(local)], dtype=torch.float64)
            S.allreduce_sqnorm(s)                                   # the path's only exchange
            hp.step = k
            assert O.hybrid8_step(local, BLOCK, hp, float(s.item())) == 0
            out[k] = float(s.item())
        q.put((rank, out, {i: (ts[i].param.copy(), ts[i].m_code.copy(), ts[i].v_code.copy(),
                               ts[i].m_absmax.copy(), ts[i].v_absmax.copy()) for i in mine}))
    finally:
        dist.destroy_process_group()


def test_two_ranks_reproduce_the_unsharded_step():
    world = 2
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = [q.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    norms = results[0][1]
    assert all(r[1] == norms for r in results)                      # every rank saw the same global norm
    # unsharded run with the same global norms
    spec = W.ragged_spec(n_tensors=40, max_numel=1 << 13, seed=7)
    _, ts = _make(spec, 1)
    hp = O.HParams(max_norm=0.5)
    for k in (1, 2):
        if k > 1:
            buf, _ = _make(spec, k)
            for i, t in enumerate(ts):
                t.set_grad(W.numpy_view(buf.view("grad", i)).copy())
        seq = O.sqnorm(ts)
        assert abs(norms[k] - seq) <= 1e-12 * seq                   # all-reduced partial sums vs one sum
        hp.step = k
        O.hybrid8_step(ts, BLOCK, hp, norms[k])
    seen = set()
    for _, _, state in results:
        for i, arrs in state.items():
            seen.add(i)
            ref = (ts[i].param, ts[i].m_code, ts[i].v_code, ts[i].m_absmax, ts[i].v_absmax)
            for a, b in zip(arrs, ref):
                assert np.array_equal(a, b)
    assert seen == set(range(len(spec.sizes)))


def test_contiguous_partition_covers_in_order():
    spec = W.ragged_spec(n_tensors=300, max_numel=1 << 16, seed=2)
    total = sum(spec.sizes)
    for world in (1, 2, 3, 8):
        runs = S.partition_contiguous(spec.sizes, world)
        assert [i for r in runs for i in r] == list(range(300))
        loads = [sum(spec.sizes[i] for i in r) for r in runs]
        assert max(abs(l - total / world) for l in loads) <= max(spec.sizes)
    assert [len(r) for r in S.partition_contiguous([5, 5], 4)] in ([1, 0, 1, 0], [0, 1, 0, 1], [1, 0, 0, 1], [0, 1, 1, 0])
    assert [list(r) for r in S.partition_contiguous([], 2)] == [[], []]


def _gather_worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        spec = W.ragged_spec(n_tensors=24, max_numel=1 << 12, seed=11)
        runs = S.partition_contiguous(spec.sizes, world)
        buf, ts = _make(spec, 1)                                     # every rank holds all parameters
        mine = [ts[i] for i in runs[rank]]
        s = torch.tensor([O.sqnorm(mine)], dtype=torch.float64)
        S.allreduce_sqnorm(s)
        assert O.hybrid8_step(mine, BLOCK, O.HParams(max_norm=0.5), float(s.item())) == 0
        for i in runs[rank]:                                         # write the owned slice back into the replica
            buf.view("param", i).copy_(torch.from_numpy(ts[i].param))
        ends = [(buf.off[r[0]], buf.off[r[-1]] + spec.sizes[r[-1]]) if len(r) else (0, 0) for r in runs]
        S.allgather_params(buf.param, ends)
        q.put((rank, float(s.item()), buf.param.numpy().copy()))
    finally:
        dist.destroy_process_group()


def test_allgather_rebuilds_the_replicated_parameters():
    world = 3
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_gather_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = [q.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    spec = W.ragged_spec(n_tensors=24, max_numel=1 << 12, seed=11)
    buf, ts = _make(spec, 1)
    O.hybrid8_step(ts, BLOCK, O.HParams(max_norm=0.5), results[0][1])
    for i, t in enumerate(ts):
        buf.view("param", i).copy_(torch.from_numpy(t.param))
    want = buf.param.numpy()
    for _, _, got in results:                                       # every replica equals the unsharded update
        assert np.array_equal(got, want)
