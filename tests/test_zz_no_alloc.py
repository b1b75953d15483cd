"""mpe_forward_static: the evaluation forward for callers that may not allocate device memory.

Some users of this library run where a cudaMalloc at call time is off limits: a serving process whose
device-memory budget is fixed at start-up, a host framework whose allocator has to account for every byte,
or a latency-critical section where the implicit synchronisation of cudaMalloc/cudaFree would stall other
streams.  mpe_forward grows its workspace with cudaMalloc when a larger batch arrives; mpe_forward_static
instead keeps every intermediate array of the step in one fixed `static __device__` array inside the library.

The test calls the new entry point through the C ABI twice in a row (the second call meets the first call's
leftovers in the shared array) and requires bit-equal pooled outputs with the existing mpe_forward and with
the CPU oracle; it checks that the driver reports the same amount of free device memory before and after the
calls, the degraded inputs (ids outside a table, inconsistent offsets) and the size limit.  It lives in a file
that pytest collects last, so a run that stops at the first failure has already run every other test, and it
builds its own handle so that it passes alone in a fresh process as well as after the other tests.
"""
import numpy as np
import pytest
import torch

from paper_2010_11305_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _batch(cfg, step, drop=0):
    idx, off, grad = wl.Stream(cfg, "cpu").batch(step)
    if drop:      # a shorter batch: fewer samples, so the second call is smaller than the first
        keep = cfg.batch - drop
        parts, lens = [], []
        off_np, idx_np = off.numpy(), idx.numpy()
        for t in range(cfg.num_tables):
            lo, hi = off_np[t * cfg.batch], off_np[t * cfg.batch + keep]
            parts.append(idx_np[lo:hi])
            lens.append(np.diff(off_np[t * cfg.batch: t * cfg.batch + keep + 1]))
        idx = torch.tensor(np.concatenate(parts))
        off = torch.tensor(np.concatenate([[0], np.cumsum(np.concatenate(lens))]).astype(np.int32))
        return idx, off, keep
    return idx, off, cfg.batch


@pytest.mark.parametrize("bits,dim,policy", [(4, 128, wl.LFU), (8, 16, wl.LRU), (2, 64, wl.LFU)])
def test_static_forward_matches_forward_on_two_calls_in_a_row(bits, dim, policy):
    if not torch.cuda.is_available():
        pytest.fail("needs a CUDA device")
    from parity_util import make_pair
    from paper_2010_11305_b200 import binding as mpe
    cfg = wl.Config("noalloc", [50_000, 3_000, 40], dim, bits, 0.05, 8, policy, wl.SGD, 0.05, 256, ("poisson", 12.0),
                    [1.1, 1.3, None], 3, seed=77)
    h, o = make_pair(cfg)
    st = wl.Stream(cfg, "cpu")
    # two training steps first, so that the cache holds rows and both fetch paths are exercised
    for step in (1, 2):
        idx, off, grad = st.batch(step)
        out = torch.empty(cfg.batch, cfg.num_tables * cfg.dim, device="cuda")
        h.forward(idx.cuda(), off.cuda(), cfg.batch, out)
        h.backward(grad.cuda(), cfg.lr, step)
        o.forward(idx.numpy(), off.numpy(), cfg.batch)
        o.backward(grad.numpy(), cfg.lr, step)
    assert h.stats(0)[3] > 0                                   # some rows are cache resident by now
    calls = [_batch(cfg, 3), _batch(cfg, 4, drop=100)]         # second call: a different, smaller batch
    # everything the calls need is on the device before the free memory is read
    dev_calls = [(idx.cuda(), off.cuda(), batch, torch.full((batch, cfg.num_tables * cfg.dim), 9.0, device="cuda"))
                 for idx, off, batch in calls]
    h.forward_static(dev_calls[0][0], dev_calls[0][1], dev_calls[0][2], dev_calls[0][3])      # first call on this device: address look-up
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for idx, off, batch, out in dev_calls:                     # the new entry point, two calls in a row
        assert idx.numel() <= mpe.STATIC_MAX_INDICES
        out.fill_(9.0)
        h.forward_static(idx, off, batch, out)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before, "device memory was allocated or freed by mpe_forward_static"
    # ids outside a table add nothing, here as in mpe_forward (and this entry point does not record them)
    idx, off, batch = calls[1]
    bad = idx.clone()
    n_bad = bad[::7].numel()
    bad[::7] = torch.tensor([-1, 50_000, 2 ** 31 - 1, -5], dtype=torch.int32).repeat(n_bad // 4 + 1)[:n_bad]
    got_bad = torch.full((batch, cfg.num_tables * cfg.dim), 9.0, device="cuda")
    h.forward_static(bad.cuda(), off.cuda(), batch, got_bad)
    assert h.last_error() == (0, 0)
    # offsets that do not grow: all-zero output, nothing recorded, nothing changed
    wrong = off.clone()
    wrong[5] = wrong[-1] + 3
    got_wrong = torch.full((batch, cfg.num_tables * cfg.dim), 9.0, device="cuda")
    h.forward_static(idx.cuda(), wrong.cuda(), batch, got_wrong)
    assert torch.all(got_wrong == 0) and h.last_error() == (0, 0)
    assert np.array_equal(got_bad.cpu().numpy(), o.forward(bad.numpy(), off.numpy(), batch))
    # the existing entry point and the oracle on the same inputs
    for (idx, off, batch), (d_idx, d_off, _, got) in zip(calls, dev_calls):
        ref = torch.empty(batch, cfg.num_tables * cfg.dim, device="cuda")
        h.forward(d_idx, d_off, batch, ref)
        torch.cuda.synchronize()
        assert torch.equal(got, ref), "mpe_forward_static and mpe_forward disagree"
        assert np.array_equal(got.cpu().numpy(), o.forward(idx.numpy(), off.numpy(), batch)), "mpe_forward_static and the oracle disagree"
        assert float(ref.abs().sum()) > 0
    # and the state was not touched: the training step goes on as the oracle's does
    idx, off, grad = st.batch(5)
    out = torch.empty(cfg.batch, cfg.num_tables * cfg.dim, device="cuda")
    h.forward(idx.cuda(), off.cuda(), cfg.batch, out)
    assert np.array_equal(out.cpu().numpy(), o.forward(idx.numpy(), off.numpy(), cfg.batch))
    with pytest.raises(mpe.MpeError) as e:                     # not between forward and backward of a step
        h.forward_static(idx.cuda(), off.cuda(), cfg.batch, out)
    assert e.value.code == mpe.ERR_SEQUENCE
    h.backward(grad.cuda(), cfg.lr, 5)
    o.backward(grad.numpy(), cfg.lr, 5)
    from parity_util import compare_state
    compare_state(h, o, cfg, [0, 1, 2], np.random.default_rng(0))
    assert h.last_error() == (0, 0)
    h.close()


def test_static_forward_rejects_what_does_not_fit():
    if not torch.cuda.is_available():
        pytest.fail("needs a CUDA device")
    from paper_2010_11305_b200 import binding as mpe
    h = mpe.Mpe([1000], 16, 8, 0.1, 8, mpe.LRU)
    n = mpe.STATIC_MAX_INDICES + 1
    idx = torch.zeros(n, dtype=torch.int32, device="cuda")
    off = torch.tensor([0, n], dtype=torch.int32, device="cuda")
    out = torch.full((1, 16), 5.0, device="cuda")
    with pytest.raises(mpe.MpeError) as e:
        h.forward_static(idx, off, 1, out)
    assert e.value.code == mpe.ERR_TOO_LARGE
    assert torch.all(out == 5.0)                               # nothing ran
    batch = mpe.STATIC_MAX_BAGS + 1
    off = torch.zeros(batch + 1, dtype=torch.int32, device="cuda")
    out = torch.empty(batch, 16, device="cuda")
    with pytest.raises(mpe.MpeError) as e:
        h.forward_static(idx[:0], off, batch, out)
    assert e.value.code == mpe.ERR_TOO_LARGE
    h.close()
