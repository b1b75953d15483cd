"""The N > 1 plumbing of bench.py on CPU: two gloo ranks, table-wise shards, MAX-of-times / SUM-of-rows."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2010_11305_b200 import workloads as wl
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = bench.shard_config(wl.scaled(wl.config(1), rows_div=10, batch_div=4), rank)
    idx, off, grad = wl.Stream(cfg, "cpu").batch(1)
    times, rows = bench.aggregate([10.0 + rank, 1.0 - 0.25 * rank], [float(idx.numel()), 7.0], world, "cpu")
    out.put((rank, cfg.seed, int(idx.sum()), times, rows, int(idx.numel())))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_tables_and_aggregate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, seed0, sum0, t0, rows0, n0), (r1, seed1, sum1, t1, rows1, n1) = res
    assert seed0 != seed1 and sum0 != sum1            # each rank owns different tables / streams
    assert t0 == t1 == [11.0, 1.0]                    # the slowest rank's time
    assert rows0 == rows1 == [float(n0 + n1), 14.0]   # everybody's rows


def test_single_rank_aggregate_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate([3.0, 4.0], [5.0, 6.0], 1, "cpu") == ([3.0, 4.0], [5.0, 6.0])


def _routed_worker(rank, world, port, out):
    """bench.py --routed on two gloo ranks: the real ShardedMpe plumbing over a fake device layer."""
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import bench
    from paper_2010_11305_b200 import sharded, workloads as wl
    from test_sharded import _FakeBackend
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)

    class Cpu(sharded.ShardedMpe):
        def _wrap(self, address, shape):
            return torch.zeros(*shape)

        def _empty(self, shape):
            return torch.zeros(*shape)

        def _sync(self):
            pass

    cfg = wl.scaled(wl.config(1), rows_div=10, batch_div=4)            # 1 table per rank, batch 32
    be = _FakeBackend(rank)
    sm, st = bench.make_routed(cfg, rank, world, 0, sharded_cls=Cpu, backend=be, stream_device="cpu")
    b1, b2 = st.batch(1), st.batch(2)
    bench.routed_step(sm, b1, cfg.lr, 1)
    bench.routed_step(sm, b2, cfg.lr, 2)
    sm.close()
    out.put((rank, sm.ranges, tuple(sm.pooled_shape) if hasattr(sm, "pooled_shape") else None, be.log, int(b1[0].sum())))
    dist.barrier()
    dist.destroy_process_group()


def test_routed_bench_plumbing_on_two_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 33500 + os.getpid() % 2000
    procs = [ctx.Process(target=_routed_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][4] != res[1][4]                                       # each rank draws its own tables' indices
    for rank, ranges, _, log, _ in res:
        assert ranges == [(0, 1), (1, 2)]                               # two equal tables, one per rank
        create = [e for e in log if e[0] == "create"][0]
        assert create[1] == [1000] and create[2] == rank                # the configuration's table, seed + rank
        names = [e[0] for e in log if e[0] in ("forward_routed", "gather_grad", "backward")]
        assert names == ["forward_routed", "gather_grad", "backward"] * 2
        fr = [e for e in log if e[0] == "forward_routed"]
        assert all(e[1] == 32 and e[3] == 2 and e[4] == rank for e in fr)          # whole batch, 2 tables in all, own table first
        bw = [e for e in log if e[0] == "backward"]
        assert [e[2] for e in bw] == [1, 2] and all(e[1] == (32, 16) for e in bw)  # step numbers; [batch][own tables * dim]
