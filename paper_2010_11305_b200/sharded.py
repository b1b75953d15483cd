"""Table-wise model parallelism: every rank owns a contiguous range of the tables (Section 1 of the paper: embeddings are
partitioned across GPUs with no replication) and the pooled vectors / their gradients change hands through buffers that
the ranks map into one another's address space.

Only plumbing lives here: which rank owns which tables, the exchange of buffer handles over `torch.distributed`, and the
host-side ordering (a barrier between "every rank has written" and "a rank reads").  The stores into the owners' buffers
are made by the pooling kernel itself and the gradient columns are pulled by a copy kernel, both behind the C ABI
(`mpe_forward_routed`, `mpe_gather_grad`).  Kernels of different ranks never wait for one another.
"""
import numpy as np
import torch
import torch.distributed as dist

from . import binding as mpe


def partition_tables(num_rows, row_bytes, n_ranks):
    """Contiguous ranges [(first, last+1)] of table ids, one per rank, balanced by stored bytes (rows x bytes per row).

    Ranges are contiguous so that a rank's pooled vectors land in one run of columns of the [B_local][T * dim] buffers.
    Greedy on the prefix sums: rank g ends at the table where the running total first reaches (g + 1) / n_ranks of the
    whole, and every rank keeps at least one table while enough tables remain.
    """
    T = len(num_rows)
    if n_ranks < 1 or T < n_ranks:
        raise ValueError(f"{T} tables cannot be spread over {n_ranks} ranks")
    weight = np.asarray(num_rows, np.float64) * float(row_bytes)
    prefix = np.concatenate([[0.0], np.cumsum(weight)])
    total = prefix[-1]
    ranges, first = [], 0
    for g in range(n_ranks):
        if g == n_ranks - 1:
            last = T
        else:
            target = total * (g + 1) / n_ranks
            last = int(np.searchsorted(prefix, target, side="left"))
            # the boundary table goes to whichever side leaves the smaller error
            if last > first + 1 and abs(prefix[last - 1] - target) <= abs(prefix[last] - target):
                last -= 1
            last = max(last, first + 1)
            last = min(last, T - (n_ranks - 1 - g))
        ranges.append((first, last))
        first = last
    return ranges


class _DeviceArray:
    """View of raw device memory for torch.as_tensor (CUDA array interface)."""

    def __init__(self, address, shape):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": "<f4", "data": (int(address), False), "version": 3,
                                         "strides": None}


class ShardedMpe:
    """One rank's share of an embedding collection plus its exchange buffers.

    pooled : float32 [B_local, T_global * dim] — after forward(), the pooled vectors of this rank's samples for ALL tables.
    grad   : float32 [B_local, T_global * dim] — the caller writes dLoss/dpooled for its samples here before backward().
    """

    def __init__(self, num_rows, dim, bits, cache_fraction, ways, policy, optimizer, eps, init_lo, init_hi, seed, batch,
                 device, group=None, backend=mpe):
        self.group, self.mpe = group, backend
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)
        if batch % self.world:
            raise ValueError("the batch must be a multiple of the number of ranks")
        self.device = int(device)
        self.T_global, self.dim, self.batch, self.B_local = len(num_rows), dim, batch, batch // self.world
        row_bytes = dim * bits // 8 + (0 if bits == 16 else 8)
        self.ranges = partition_tables(num_rows, row_bytes, self.world)
        self.first, self.last = self.ranges[self.rank]
        self.local_rows = list(num_rows[self.first:self.last])
        # every rank numbers its tables from 0, so the per-rank seed keeps the ranks' hash salts and random streams apart
        self.h = self.mpe.Mpe(self.local_rows, dim, bits, cache_fraction, ways, policy, optimizer, eps, init_lo, init_hi,
                         seed + self.rank, self.device)
        nbytes = self.B_local * self.T_global * dim * 4
        self._own = [self.mpe.peer_buffer_alloc(self.device, max(nbytes, 16)) for _ in range(2)]       # pooled, grad
        handles = [None] * self.world
        dist.all_gather_object(handles, [hd for _, hd in self._own], group=group)
        self._opened = []
        self.pooled_ptrs, self.grad_ptrs = [], []
        for g in range(self.world):
            if g == self.rank:
                p, q = self._own[0][0], self._own[1][0]
            else:
                p, q = (self.mpe.peer_buffer_open(self.device, hd) for hd in handles[g])
                self._opened += [p, q]
            self.pooled_ptrs.append(p)
            self.grad_ptrs.append(q)
        shape = (self.B_local, self.T_global * dim)
        self.pooled = self._wrap(self._own[0][0], shape)
        self.grad = self._wrap(self._own[1][0], shape)
        self.local_grad = self._empty((batch, len(self.local_rows) * dim))
        self._rendezvous()

    # the three places that touch the device from Python (a CPU test of the plumbing replaces them)
    def _wrap(self, address, shape):
        return torch.as_tensor(_DeviceArray(address, shape), device=torch.device("cuda", self.device))

    def _empty(self, shape):
        return torch.empty(*shape, dtype=torch.float32, device=torch.device("cuda", self.device))

    def _sync(self):
        torch.cuda.synchronize(self.device)

    def _rendezvous(self):
        """Everything this rank has launched is finished, and every rank has got here."""
        self._sync()
        dist.barrier(group=self.group)

    def forward(self, d_indices, d_offsets):
        """d_indices / d_offsets: the WHOLE batch's bags for this rank's tables (CSR over table-major bags)."""
        self.h.forward_routed(d_indices, d_offsets, self.batch, self.pooled_ptrs, self.T_global, self.first)
        self._rendezvous()
        return self.pooled

    def backward(self, lr, step):
        """`grad` holds this rank's samples; the columns of this rank's tables are pulled from every rank, then applied."""
        self._rendezvous()                     # every rank's grad buffer is complete
        self.h.gather_grad(self.grad_ptrs, self.T_global, self.first, self.batch, self.local_grad)
        self.h.backward(self.local_grad, lr, step)
        # the next forward's rendezvous comes before any rank overwrites `grad` or `pooled` again

    def close(self):
        if self.h is None:
            return
        self._rendezvous()
        for p in self._opened:
            self.mpe.peer_buffer_close(self.device, p)
        self._rendezvous()
        self.pooled = self.grad = None
        for p, _ in self._own:
            self.mpe.peer_buffer_free(self.device, p)
        self.h.close()
        self.h = None
