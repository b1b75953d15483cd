"""Tables partitioned over ranks (Section 1: model parallelism with no replication): the partition, the host-side
plumbing on two gloo ranks with a fake device layer (CPU), and on the GPU the routed forward / gradient gather against
the oracle — first with the ranks emulated inside one process over all ranks' data, then as two processes that map one
another's buffers on the same GPU."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))


# ------------------------------------------------------------------------------------------- partition (CPU) -
def test_partition_is_contiguous_complete_and_balanced():
    from paper_2010_11305_b200.sharded import partition_tables
    assert partition_tables([5] * 8, 72, 4) == [(0, 2), (2, 4), (4, 6), (6, 8)]
    assert partition_tables([5] * 8, 72, 1) == [(0, 8)]
    assert partition_tables([1, 1, 1], 24, 3) == [(0, 1), (1, 2), (2, 3)]
    # one huge table first: it gets a rank of its own, the small ones share the rest
    r = partition_tables([10_000_000, 10, 10, 10, 10], 24, 3)
    assert r[0] == (0, 1) and r[-1][1] == 5 and all(b > a for a, b in r)
    # huge table last: every earlier rank still keeps at least one table
    r = partition_tables([10, 10, 10, 10, 10_000_000], 24, 3)
    assert r[-1][1] == 5 and all(b > a for a, b in r) and [a for a, _ in r[1:]] == [b for _, b in r[:-1]]
    rng = np.random.default_rng(0)
    for _ in range(50):
        T = int(rng.integers(1, 40))
        G = int(rng.integers(1, T + 1))
        rows = rng.integers(3, 10_000_000, T).tolist()
        r = partition_tables(rows, 40, G)
        assert len(r) == G and r[0][0] == 0 and r[-1][1] == T
        assert all(b > a for a, b in r) and all(r[g][1] == r[g + 1][0] for g in range(G - 1))
        loads = [sum(rows[a:b]) for a, b in r]
        assert max(loads) <= sum(rows) / G + max(rows)            # never worse than one table over the even share
    with pytest.raises(ValueError):
        partition_tables([1, 2], 24, 3)


# ---------------------------------------------------------------------- plumbing on two gloo ranks, fake device -
class _FakeHandle:
    def __init__(self, log, *args):
        self.log = log
        log.append(("create", list(args[0]), args[10]))

    def forward_routed(self, idx, off, batch, ptrs, tables_global, table_base, stream=None):
        self.log.append(("forward_routed", batch, list(ptrs), tables_global, table_base))

    def gather_grad(self, ptrs, tables_global, table_base, batch, local, stream=None):
        self.log.append(("gather_grad", list(ptrs), tables_global, table_base, batch, tuple(local.shape)))

    def backward(self, grad, lr, step):
        self.log.append(("backward", tuple(grad.shape), step))

    def close(self):
        self.log.append(("close",))


class _FakeBackend:
    """Stands in for the binding: addresses are made up, a handle just names (rank, buffer)."""

    def __init__(self, rank):
        self.rank, self.log, self.n = rank, [], 0

    def Mpe(self, *args):
        return _FakeHandle(self.log, *args)

    def peer_buffer_alloc(self, device, nbytes):
        self.n += 1
        return 0x1000 * (self.rank + 1) + 0x10 * self.n, bytes([self.rank, self.n]) + bytes(62)

    def peer_buffer_open(self, device, handle):
        assert handle[0] != self.rank                              # a rank never opens its own handle
        self.log.append(("open", handle[0], handle[1]))
        return 0x100000 + 0x1000 * (handle[0] + 1) + 0x10 * handle[1]

    def peer_buffer_close(self, device, p):
        self.log.append(("closed", p))

    def peer_buffer_free(self, device, p):
        self.log.append(("freed", p))


def _plumbing_worker(rank, world, port, out):
    from paper_2010_11305_b200 import sharded
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

    be = _FakeBackend(rank)
    rows = [100, 200, 300, 400, 500]
    s = Cpu(rows, 8, 8, 0.1, 4, 0, 0, 1e-8, -0.05, 0.05, 7, 6, 0, backend=be)
    s.forward(torch.zeros(3, dtype=torch.int32), torch.zeros(4, dtype=torch.int32))
    s.backward(0.1, 1)
    s.close()
    out.put((rank, s.ranges, be.log, tuple(s.local_grad.shape)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_exchange_handles_and_route_by_owner():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_plumbing_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ranges, log, lg in res:
        assert ranges == res[0][1] and ranges[0][0] == 0 and ranges[-1][1] == 5
        first, last = ranges[rank]
        create = [e for e in log if e[0] == "create"][0]
        assert create[1] == [100, 200, 300, 400, 500][first:last] and create[2] == 7 + rank
        other = 1 - rank
        own_pooled, own_grad = 0x1000 * (rank + 1) + 0x10, 0x1000 * (rank + 1) + 0x20
        peer_pooled, peer_grad = 0x100000 + 0x1000 * (other + 1) + 0x10, 0x100000 + 0x1000 * (other + 1) + 0x20
        want_pooled = [own_pooled, peer_pooled] if rank == 0 else [peer_pooled, own_pooled]
        want_grad = [own_grad, peer_grad] if rank == 0 else [peer_grad, own_grad]
        fr = [e for e in log if e[0] == "forward_routed"][0]
        assert fr == ("forward_routed", 6, want_pooled, 5, first)
        gg = [e for e in log if e[0] == "gather_grad"][0]
        assert gg == ("gather_grad", want_grad, 5, first, 6, (6, (last - first) * 8)) and lg == (6, (last - first) * 8)
        assert sorted(e[1] for e in log if e[0] == "closed") == sorted([peer_pooled, peer_grad])
        assert sorted(e[1] for e in log if e[0] == "freed") == sorted([own_pooled, own_grad])
        names = [e[0] for e in log]
        assert names.index("gather_grad") < names.index("backward") < names.index("closed") < names.index("freed")


# --------------------------------------------------------------------------------------------------- GPU ------
def _shard_cfgs(world):
    """Per-rank configurations the way ShardedMpe builds them: contiguous table ranges, seed + rank."""
    from dataclasses import replace
    from paper_2010_11305_b200 import workloads as wl
    from paper_2010_11305_b200.sharded import partition_tables
    base = wl.Config(name="sharded", num_rows=[3000, 700, 5000, 40, 2500, 900], dim=32, bits=4, cache_fraction=0.05, ways=8,
                     policy=wl.LFU, optimizer=wl.SGD, lr=0.05, batch=96, bag=("poisson_cap", 6.0, 40), zipf=[1.1] * 6, steps=4, seed=11)
    ranges = partition_tables(base.num_rows, base.dim * base.bits // 8 + 8, world)
    cfgs = [replace(base, num_rows=base.num_rows[a:b], zipf=base.zipf[a:b], seed=base.seed + g) for g, (a, b) in enumerate(ranges)]
    return base, ranges, cfgs


def _oracle_for(cfg):
    from oracle import mpe_oracle as orc
    return orc.Oracle(cfg.num_rows, cfg.dim, cfg.bits, cfg.cache_fraction, cfg.ways, cfg.policy, cfg.optimizer, cfg.eps,
                      cfg.init_lo, cfg.init_hi, cfg.seed)


@pytest.mark.gpu
@pytest.mark.parametrize("world", [1, 2, 3])
def test_routed_forward_and_gradient_gather_with_ranks_emulated_in_one_process(world):
    """All ranks' handles and buffers live in this process on one GPU; nothing waits on anything."""
    from paper_2010_11305_b200 import binding as mpe, workloads as wl
    from parity_util import compare_state
    base, ranges, cfgs = _shard_cfgs(world)
    dev = torch.device("cuda:0")
    B, Bl, Tg, d = base.batch, base.batch // world, base.num_tables, base.dim
    hs = [mpe.Mpe(c.num_rows, c.dim, c.bits, c.cache_fraction, c.ways, c.policy, c.optimizer, c.eps, c.init_lo, c.init_hi, c.seed, 0)
          for c in cfgs]
    os_ = [_oracle_for(c) for c in cfgs]
    streams = [wl.Stream(c, "cpu") for c in cfgs]
    pooled = [torch.full((Bl, Tg * d), float("nan"), device=dev) for _ in range(world)]
    gen = torch.Generator().manual_seed(3)
    rng = np.random.default_rng(0)
    for step in range(1, base.steps + 1):
        batches = [st.batch(step) for st in streams]
        ref_full = np.zeros((B, Tg * d), np.float32)
        for g, (a, b) in enumerate(ranges):
            idx, off, _ = batches[g]
            hs[g].forward_routed(idx.to(dev), off.to(dev), B, [p.data_ptr() for p in pooled], Tg, a)
            ref_full[:, a * d:b * d] = os_[g].forward(idx.numpy(), off.numpy(), B)
        torch.cuda.synchronize()
        for g in range(world):                                   # rank g holds its samples, every table
            assert np.array_equal(pooled[g].cpu().numpy(), ref_full[g * Bl:(g + 1) * Bl]), (step, g)
        grads = [(torch.randn(Bl, Tg * d, generator=gen) * 1e-2).to(dev) for _ in range(world)]
        grad_full = torch.cat([x.cpu() for x in grads]).numpy()
        for g, (a, b) in enumerate(ranges):
            local = torch.full((B, (b - a) * d), float("nan"), device=dev)
            hs[g].gather_grad([x.data_ptr() for x in grads], Tg, a, B, local)
            want = np.ascontiguousarray(grad_full[:, a * d:b * d])
            assert np.array_equal(local.cpu().numpy(), want), (step, g)
            hs[g].backward(local, base.lr, step)
            os_[g].backward(want, base.lr, step)
    for g, c in enumerate(cfgs):
        assert hs[g].last_error() == (0, 0)
        compare_state(hs[g], os_[g], c, range(c.num_tables), rng)
        hs[g].close()


@pytest.mark.gpu
def test_routed_calls_refuse_bad_arguments():
    from paper_2010_11305_b200 import binding as mpe
    dev = torch.device("cuda:0")
    h = mpe.Mpe([100, 50], 8, 8, 0.1, 4, 0, 0, 1e-8, -0.05, 0.05, 1, 0)
    idx = torch.zeros(4, dtype=torch.int32, device=dev)
    off = torch.tensor([0, 1, 2, 3, 4], dtype=torch.int32, device=dev)
    buf = torch.zeros(64, device=dev)
    p = buf.data_ptr()
    for args in ((3, [p, p], 2, 0),          # batch not a multiple of the ranks
                 (2, [p], 1, 0),             # fewer global tables than this handle owns
                 (2, [p], 3, 2),             # table_base + own tables beyond tables_global
                 (2, [p + 4], 2, 0),         # unaligned destination
                 (2, [0], 2, 0),             # null destination
                 (2, [p] * 73, 2, 0)):       # more ranks than the routing table holds
        batch, ptrs, tg, tb = args
        with pytest.raises(mpe.MpeError) as e:
            h.forward_routed(idx, off, batch, ptrs, tg, tb)
        assert e.value.code == mpe.ERR_ARG
        with pytest.raises(mpe.MpeError):
            h.gather_grad(ptrs, tg, tb, batch, buf)
    h.close()


def _ipc_worker(rank, world, port, out):
    try:
        from paper_2010_11305_b200 import sharded, workloads as wl
        from parity_util import compare_state
        os.environ["MASTER_ADDR"] = "127.0.0.1"
        os.environ["MASTER_PORT"] = str(port)
        dist.init_process_group("gloo", rank=rank, world_size=world)
        base, ranges, cfgs = _shard_cfgs(world)
        c = cfgs[rank]
        dev = torch.device("cuda:0")                             # both ranks share the one GPU; their kernels never wait on each other
        s = sharded.ShardedMpe(base.num_rows, base.dim, base.bits, base.cache_fraction, base.ways, base.policy, base.optimizer,
                               base.eps, base.init_lo, base.init_hi, base.seed, base.batch, 0)
        assert s.ranges == ranges
        os_ = [_oracle_for(x) for x in cfgs]                     # every rank replays all shards on the CPU to know the full answer
        streams = [wl.Stream(x, "cpu") for x in cfgs]
        Bl, d, Tg = s.B_local, base.dim, base.num_tables
        for step in range(1, base.steps + 1):
            batches = [st.batch(step) for st in streams]
            ref = np.zeros((base.batch, Tg * d), np.float32)
            for g, (a, b) in enumerate(ranges):
                ref[:, a * d:b * d] = os_[g].forward(batches[g][0].numpy(), batches[g][1].numpy(), base.batch)
            idx, off, _ = batches[rank]
            pooled = s.forward(idx.to(dev), off.to(dev))
            assert np.array_equal(pooled.cpu().numpy(), ref[rank * Bl:(rank + 1) * Bl]), f"rank {rank} step {step}: pooled"
            gen = torch.Generator().manual_seed(100 + step)      # the same full gradient on every rank; each writes its samples
            grad_full = torch.randn(base.batch, Tg * d, generator=gen) * 1e-2
            s.grad.copy_(grad_full[rank * Bl:(rank + 1) * Bl].to(dev))
            s.backward(base.lr, step)
            for g, (a, b) in enumerate(ranges):
                os_[g].backward(np.ascontiguousarray(grad_full[:, a * d:b * d].numpy()), base.lr, step)
        assert s.h.last_error() == (0, 0)
        compare_state(s.h, os_[rank], c, range(c.num_tables), np.random.default_rng(rank))
        s.close()
        out.put((rank, "ok"))
        dist.barrier()
        dist.destroy_process_group()
    except Exception as e:                                       # report instead of leaving the peer at a barrier
        import traceback
        out.put((rank, traceback.format_exc()))
        raise e


@pytest.mark.gpu
def test_two_processes_map_each_other_s_buffers_on_one_gpu():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 33500 + os.getpid() % 2000
    procs = [ctx.Process(target=_ipc_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = []
    try:
        for _ in procs:
            res.append(out.get(timeout=240))
            assert res[-1][1] == "ok", res[-1][1]
    finally:
        for p in procs:
            p.join(timeout=30)
            if p.is_alive():
                p.kill()
    assert sorted(r for r, _ in res) == [0, 1] and all(p.exitcode == 0 for p in procs)
