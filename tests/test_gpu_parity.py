"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle
on the same seeded inputs.  Integer state (codes, tags, timestamps, counters,
statistics) and the FP32 scale/bias/cached rows must be bit-equal; pooled
outputs must be within 1e-5 of the sum of absolute terms (they are bit-equal
too, because both sides add in index order)."""
import numpy as np
import pytest
import torch

from paper_2010_11305_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_cuda():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device; run them with -m gpu on a GPU box")


def _cfg(**kw):
    base = dict(name="t", num_rows=[1000], dim=16, bits=8, cache_fraction=0.05, ways=8, policy=wl.LRU, optimizer=wl.SGD,
                lr=0.05, batch=64, bag=("fixed", 4), zipf=[1.05], steps=4, seed=1)
    base.update(kw)
    return wl.Config(**base)


def test_config1_all_steps():
    from parity_util import run_parity
    cfg = wl.config(1)
    h, o, info = run_parity(cfg, cfg.steps)
    assert info[0][0] == 512 and 0 < info[0][1] <= 512


def test_config2_all_tables_all_hundred_steps():
    from parity_util import run_parity
    cfg = wl.config(2)
    assert cfg.steps == 100 and cfg.num_tables == 26
    run_parity(cfg, cfg.steps, check_every=25)


def test_config2_with_the_table_sizes_the_paper_prints():
    """Configuration 2 on the 26 row counts of the paper's Table 1 (tables of 3 rows up to 10 M rows, some smaller than one cache set)."""
    import os
    from dataclasses import replace
    from parity_util import run_parity
    path = os.path.join(os.path.dirname(__file__), "golden", "kaggle_table_sizes.txt")
    sizes = [int(x) for l in open(path) if not l.startswith("#") for x in l.split()]
    base = wl.config(2)
    cfg = replace(base, name="cfg2b", num_rows=sizes, zipf=[base.zipf[0]] * len(sizes))
    run_parity(cfg, 8, check_every=4)


@pytest.mark.parametrize("bits,policy,opt,ways,dim", [
    (8, wl.LRU, wl.SGD, 8, 16), (4, wl.LRU, wl.ROWWISE_ADAGRAD, 16, 64), (4, wl.LFU, wl.SGD, 32, 128),
    (8, wl.LFU, wl.ROWWISE_ADAGRAD, 32, 64), (4, wl.LFU, wl.SGD, 2, 32), (8, wl.LRU, wl.SGD, 1, 8),
    (4, wl.LFU, wl.SGD, 1, 4), (8, wl.LRU, wl.SGD, 4, 128), (2, wl.LFU, wl.SGD, 32, 128), (2, wl.LRU, wl.ROWWISE_ADAGRAD, 8, 16),
    (2, wl.LFU, wl.SGD, 2, 4), (16, wl.LRU, wl.SGD, 32, 128), (16, wl.LFU, wl.ROWWISE_ADAGRAD, 4, 16), (16, wl.LFU, wl.SGD, 1, 4),
])
def test_small_tables_every_variant(bits, policy, opt, ways, dim):
    """Small tables with a skewed stream: many hits, admissions, evictions, bypasses and chains per step."""
    from parity_util import run_parity
    cfg = _cfg(num_rows=[3000, 500, 7], dim=dim, bits=bits, policy=policy, optimizer=opt, ways=ways, cache_fraction=0.1,
               batch=96, bag=("poisson", 6.0), zipf=[1.1, 0.9, None], steps=8, seed=bits + ways)
    h, o, _ = run_parity(cfg, 8)
    s = h.stats(0)
    assert s[3] > 0 and s[4] > 0 and s[5] > 0                  # hits, admissions and evictions all occurred
    assert s[6] > 0 or (ways == 1 and policy == wl.LRU)        # bypasses too (direct-mapped LRU never bypasses)


def test_config3_scaled_and_ragged():
    from parity_util import run_parity
    cfg = wl.scaled(wl.config(3), rows_div=100, batch_div=8, steps=6)
    run_parity(cfg, 6, check_every=2)


def test_config4_scaled_hot_rows():
    """Poisson bags capped at 100, per-table skew, LFU, INT4 d=128; the hottest rows exceed 1024 occurrences."""
    from parity_util import run_parity
    cfg = wl.scaled(wl.config(4), rows_div=50, batch_div=8, tables=6, steps=4)
    h, o, info = run_parity(cfg, 4, check_every=2)
    assert info[0][3] > 0        # rows that needed the multi-block gradient tree


def test_config5_points():
    from parity_util import run_parity
    pts = list(wl.sweep5())
    for cfg in (pts[2], pts[len(pts) // 2 + 5], pts[-1]):
        cfg = wl.scaled(cfg, rows_div=20, batch_div=4, steps=4)
        run_parity(cfg, 4, check_every=2)


def test_no_cache_is_pure_low_precision_training():
    from parity_util import run_parity
    run_parity(_cfg(cache_fraction=0.0, bits=4, dim=32), 4)


def test_very_hot_row_uses_three_tree_levels():
    """One row with > 32768 occurrences in a batch: partial sums of 1024, then of 32768, then the rest."""
    from parity_util import make_pair, compare_state
    cfg = _cfg(num_rows=[50], dim=8, batch=40000, bag=("fixed", 1), zipf=[3.0], cache_fraction=0.2, ways=2)
    h, o = make_pair(cfg)
    st = wl.Stream(cfg, "cpu")
    rng = np.random.default_rng(0)
    for step in (1, 2):
        idx, off, grad = st.batch(step)
        assert np.bincount(idx.numpy()).max() > 32768
        out = torch.empty(cfg.batch, cfg.dim, device="cuda")
        h.forward(idx.cuda(), off.cuda(), cfg.batch, out)
        ref = o.forward(idx.numpy(), off.numpy(), cfg.batch)
        assert np.array_equal(out.cpu().numpy(), ref)
        h.backward(grad.cuda(), 0.01, step)
        o.backward(grad.numpy(), 0.01, step)
        compare_state(h, o, cfg, [0], rng)


def test_empty_bags_empty_batch_and_duplicates_inside_a_bag():
    from parity_util import make_pair, compare_state
    cfg = _cfg(num_rows=[40, 40], dim=16, batch=5, cache_fraction=0.25, ways=2)
    h, o = make_pair(cfg)
    rng = np.random.default_rng(0)
    bags = [[[1, 1, 1], [], [2, 3, 2], [], []], [[], [], [], [], []]]
    idx = np.array([r for tb in bags for bag in tb for r in bag], np.int32)
    off = np.cumsum([0] + [len(bag) for tb in bags for bag in tb]).astype(np.int32)
    grad = rng.normal(0, 0.1, (5, 32)).astype(np.float32)
    out = torch.full((5, 32), 7.0, device="cuda")
    h.forward(torch.tensor(idx).cuda(), torch.tensor(off).cuda(), 5, out)
    ref = o.forward(idx, off, 5)
    assert np.array_equal(out.cpu().numpy(), ref) and np.all(ref[1] == 0) and np.all(ref[:, 16:] == 0)
    h.backward(torch.tensor(grad).cuda(), 0.1, 1)
    o.backward(grad, 0.1, 1)
    compare_state(h, o, cfg, [0, 1], rng)
    # a batch with no index at all
    off0 = np.zeros(11, np.int32)
    out = torch.full((5, 32), 7.0, device="cuda")
    h.forward(torch.zeros(0, dtype=torch.int32, device="cuda"), torch.tensor(off0).cuda(), 5, out)
    o.forward(np.zeros(0, np.int32), off0, 5)
    assert torch.all(out == 0)
    h.backward(torch.tensor(grad).cuda(), 0.1, 2)
    o.backward(grad, 0.1, 2)
    compare_state(h, o, cfg, [0, 1], rng)
    assert h.last_error() == (0, 0)


def test_out_of_range_indices_are_dropped_and_reported():
    from parity_util import make_pair, compare_state
    from paper_2010_11305_b200 import binding as mpe
    cfg = _cfg(num_rows=[100, 30], dim=8, batch=4, cache_fraction=0.2, ways=4)
    h, o = make_pair(cfg)
    rng = np.random.default_rng(1)
    idx = np.array([5, 100, 7, -1, 5, 99, 2 ** 31 - 1, 0, 29, 30, 3, 3, -7, 12], np.int32)
    off = np.array([0, 2, 4, 6, 8, 10, 12, 13, 14], np.int32)
    grad = rng.normal(0, 0.1, (4, 16)).astype(np.float32)
    for step in (1, 2):
        out = torch.empty(4, 16, device="cuda")
        h.forward(torch.tensor(idx).cuda(), torch.tensor(off).cuda(), 4, out)
        ref = o.forward(idx, off, 4)
        assert np.array_equal(out.cpu().numpy(), ref)
        info = h.step_info()
        assert info[0] == 9 and info[2] == 5 and info[1] == 7
        h.backward(torch.tensor(grad).cuda(), 0.1, step)
        o.backward(grad, 0.1, step)
        assert h.last_error() == (mpe.ERR_INDEX, 5)
        assert h.last_error() == (0, 0)
        compare_state(h, o, cfg, [0, 1], rng)
    assert o.dropped() == 10


def test_bad_offsets_are_refused_without_touching_state():
    from parity_util import make_pair, compare_state
    from paper_2010_11305_b200 import binding as mpe
    cfg = _cfg(num_rows=[100], dim=8, batch=4)
    h, o = make_pair(cfg)
    rng = np.random.default_rng(1)
    idx = torch.tensor([1, 2, 3, 4, 5, 6], dtype=torch.int32).cuda()
    grad = torch.ones(4, 8, device="cuda")
    for step, bad in enumerate(([0, 2, 1, 4, 6], [1, 2, 3, 4, 6], [0, 2, 3, 4, 5], [0, 2, 9, 4, 6], [0, -2, 3, 4, 6]), start=1):
        out = torch.full((4, 8), 3.0, device="cuda")
        h.forward(idx, torch.tensor(bad, dtype=torch.int32).cuda(), 4, out)
        if step % 2:
            h.backward(grad, 0.1, step)        # the abandoned step's backward must be a no-op too
        code, detail = h.last_error()
        assert code == mpe.ERR_OFFSETS and detail >= 1
        assert torch.all(out == 0)
    rows = np.arange(100)
    codes, scale, bias = h.export_rows(0, rows)
    rc, rs, rb = o.rows(0, rows)
    assert np.array_equal(codes, rc) and np.array_equal(scale, rs) and np.array_equal(bias, rb)
    assert np.all(h.export_cache(0)[0] == -1) and np.all(h.stats(0)[:7] == 0)
    # and the handle still works afterwards
    good = torch.tensor([0, 2, 3, 4, 6], dtype=torch.int32).cuda()
    out = torch.empty(4, 8, device="cuda")
    h.forward(idx, good, 4, out)
    ref = o.forward(idx.cpu().numpy(), good.cpu().numpy(), 4)
    assert np.array_equal(out.cpu().numpy(), ref)
    h.backward(grad, 0.1, 10)
    o.backward(grad.cpu().numpy(), 0.1, 10)
    assert h.last_error() == (0, 0)
    tags, crow, ts = h.export_cache(0)
    otags, ocrow, ots = o.cache(0)
    assert np.array_equal(tags, otags) and np.array_equal(crow, ocrow) and np.array_equal(ts, ots)
    del rng, compare_state


def test_sequence_and_argument_errors():
    from paper_2010_11305_b200 import binding as mpe
    with pytest.raises(mpe.MpeError) as e:
        mpe.Mpe([100], 12, 8, 0.1, 8, mpe.LRU)
    assert e.value.code == mpe.ERR_UNSUPPORTED
    with pytest.raises(mpe.MpeError):
        mpe.Mpe([100], 16, 3, 0.1, 8, mpe.LRU)
    with pytest.raises(mpe.MpeError):
        mpe.Mpe([100], 16, 8, 0.1, 6, mpe.LRU)
    with pytest.raises(mpe.MpeError):
        mpe.Mpe([100], 16, 8, 1.5, 8, mpe.LRU)
    h = mpe.Mpe([100], 16, 8, 0.1, 8, mpe.LRU)
    g = torch.zeros(2, 16, device="cuda")
    with pytest.raises(mpe.MpeError) as e:
        h.backward(g, 0.1, 1)
    assert e.value.code == mpe.ERR_SEQUENCE
    idx = torch.tensor([1, 2], dtype=torch.int32).cuda()
    off = torch.tensor([0, 1, 2], dtype=torch.int32).cuda()
    out = torch.empty(2, 16, device="cuda")
    h.forward(idx, off, 2, out)
    h.backward(g, 0.1, 5)
    h.forward(idx, off, 2, out)
    with pytest.raises(mpe.MpeError) as e:
        h.backward(g, 0.1, 5)          # step must increase
    assert e.value.code == mpe.ERR_SEQUENCE
    h.backward(g, 0.1, 6)


def test_step_is_deterministic_and_forward_is_read_only():
    from paper_2010_11305_b200 import binding as mpe
    cfg = wl.scaled(wl.config(4), rows_div=100, batch_div=16, tables=3)
    st = wl.Stream(cfg, "cpu")
    results = []
    for rep in range(2):
        h = mpe.Mpe(cfg.num_rows, cfg.dim, cfg.bits, cfg.cache_fraction, cfg.ways, cfg.policy, seed=cfg.seed)
        for step in (1, 2, 3):
            idx, off, grad = (x.cuda() for x in st.batch(step))
            out = torch.empty(cfg.batch, cfg.num_tables * cfg.dim, device="cuda")
            h.forward(idx, off, cfg.batch, out)
            out2 = torch.empty_like(out)
            h.forward(idx, off, cfg.batch, out2)       # a second forward sees the same state
            assert torch.equal(out, out2)
            h.backward(grad, cfg.lr, step)
        rows = np.arange(0, cfg.num_rows[0], 3)
        results.append((h.export_rows(0, rows), h.export_cache(0), out.cpu().numpy()))
    (r0, c0, o0), (r1, c1, o1) = results
    assert all(np.array_equal(a, b) for a, b in zip(r0, r1))
    assert all(np.array_equal(a, b) for a, b in zip(c0, c1))
    assert np.array_equal(o0, o1)


def test_host_buffer_step_matches_device_step():
    from parity_util import make_pair, compare_state
    cfg = _cfg(num_rows=[2000, 300], dim=32, bits=4, batch=64, zipf=[1.05, 1.2], policy=wl.LFU, ways=4)
    h, o = make_pair(cfg)
    st = wl.Stream(cfg, "cpu")
    rng = np.random.default_rng(0)
    for step in (1, 2, 3):
        idx, off, grad = st.batch(step)
        out = np.zeros((cfg.batch, cfg.num_tables * cfg.dim), np.float32)
        h.step_host(idx.numpy(), off.numpy(), cfg.batch, grad.numpy(), out, cfg.lr, step)
        ref = o.forward(idx.numpy(), off.numpy(), cfg.batch)
        o.backward(grad.numpy(), cfg.lr, step)
        assert np.array_equal(out, ref)
    compare_state(h, o, cfg, [0, 1], rng)
    # overlapped: several steps submitted before anything is waited for, batches of different sizes (the staging
    # buffers regrow in between), pinned inputs; results are those of the same steps run one after the other
    pending = []
    step = 3
    for batch in (64, 64, 200, 32, 64, 64, 64):
        step += 1
        cfg.batch = batch
        idx, off, grad = wl.Stream(cfg, "cpu").batch(step)
        hb = [x.pin_memory() for x in (idx, off, grad)]
        out = torch.zeros(batch, cfg.num_tables * cfg.dim).pin_memory()
        h.step_host_submit(hb[0], hb[1], batch, hb[2], out, cfg.lr, step)
        pending.append((hb, out, batch, step))
    h.step_host_wait()
    for (idx, off, grad), out, batch, stp in pending:
        ref = o.forward(idx.numpy(), off.numpy(), batch)
        o.backward(grad.numpy(), cfg.lr, stp)
        assert np.array_equal(out.numpy(), ref), f"overlapped step {stp}"
    compare_state(h, o, cfg, [0, 1], rng)
    from paper_2010_11305_b200 import binding as mpe
    with pytest.raises(mpe.MpeError) as e:                 # the step number still has to grow
        h.step_host_submit(hb[0], hb[1], batch, hb[2], out, cfg.lr, step)
    assert e.value.code == mpe.ERR_SEQUENCE
    assert h.last_error() == (0, 0)


def test_memory_accounting_matches_the_appendix_table():
    import os
    from paper_2010_11305_b200 import binding as mpe
    rows = [l.split() for l in open(os.path.join(os.path.dirname(__file__), "golden", "compression_factor_table.txt"))
            if not l.startswith("#")]
    for bits, ratio, factor in rows:
        if int(bits) == 2:
            continue
        h = mpe.Mpe([320_000], 128, int(bits), float(ratio), 32, mpe.LFU)
        m = h.memory_bytes().astype(np.float64)
        assert abs((m[0] + m[1] + m[2] + m[3]) / m[5] - float(factor)) < 6e-6
        h.close()


# ---------------------------------------------------------------------------------------------
# Full-size configurations, in the launch configuration the benchmark times.  The oracle follows a
# sample of the tables (tables are independent); everything observable of those tables is compared.
# ---------------------------------------------------------------------------------------------
def _full_size(cfg, tables, steps, check_at=(), prepare_ahead=False):
    """A configuration at its full size in the launch configuration the benchmark times; the oracle follows the
    sampled tables only.  State is compared at the steps in check_at, at the last step, and again after a flush.
    prepare_ahead: as the benchmark does for steps too large to be replayed from a graph, the next batch is sorted and
    de-duplicated on a second stream while the current step runs."""
    from parity_util import make_pair, compare_state
    h, o = make_pair(cfg, tables)
    st = wl.Stream(cfg, "cuda")
    rng = np.random.default_rng(0)
    cols = np.concatenate([np.arange(t * cfg.dim, (t + 1) * cfg.dim) for t in tables])
    side = torch.cuda.Stream()
    nxt = st.batch(1)
    if prepare_ahead:
        h.reserve(cfg.batch, int(nxt[0].numel() * 1.05))
    for step in range(1, steps + 1):
        idx, off, grad = nxt
        out = torch.empty(cfg.batch, cfg.num_tables * cfg.dim, device="cuda")
        h.forward(idx, off, cfg.batch, out)
        if step < steps:
            nxt = st.batch(step + 1)
            if prepare_ahead:
                side.wait_stream(torch.cuda.current_stream())      # the next batch has been generated on the current stream
                h.prepare(nxt[0], nxt[1], cfg.batch, side.cuda_stream)
        ref = o.forward(idx.cpu().numpy(), off.cpu().numpy(), cfg.batch)
        assert np.array_equal(out[:, torch.as_tensor(cols, device="cuda")].cpu().numpy(), ref[:, cols]), f"step {step}: pooled outputs"
        h.backward(grad, cfg.lr, step)
        o.backward(grad.cpu().numpy(), cfg.lr, step)
        assert h.last_error() == (0, 0)
        if step in check_at:
            compare_state(h, o, cfg, tables, rng)
    compare_state(h, o, cfg, tables, rng)
    h.flush()
    o.flush()
    compare_state(h, o, cfg, tables, rng)
    return h


def test_full_size_config4_all_twenty_steps():
    """64 tables x 5M rows, all 20 steps of the configuration; the oracle follows the tables with the largest and the
    smallest Zipf exponent (the most and the fewest rows on the multi-block gradient path) and one in between."""
    cfg = wl.config(4)
    assert cfg.steps == 20
    z = np.array(cfg.zipf)
    tables = sorted({int(z.argmax()), int(z.argmin()), 37})
    h = _full_size(cfg, tables, cfg.steps, check_at=(3, 10), prepare_ahead=True)
    info = h.step_info()
    assert info[0] > 25_000_000 and info[3] > 500      # ~31M indices, thousands of hot rows
    assert h.workspace_bytes()[0] > 4_000_000_000      # two workspaces: batches were prepared ahead
    s = h.stats(tables[0])
    assert s[4] > 0 and s[5] > 0 and s[6] > 0          # past the fill phase: admissions, evictions and bypasses all happen
    h.close()


def test_full_size_config3_all_fifty_steps():
    cfg = wl.config(3)
    assert cfg.steps == 50
    _full_size(cfg, [0, 5], cfg.steps, check_at=(4, 25)).close()


@pytest.mark.parametrize("point", [1, 6, 11, 19, 30, 40, 53, 58, 63])
def test_full_size_config5_points_fifty_plus_fifty_steps(point):
    """Points of the policy/skew sweep at full size, over the 50 warm-up + 50 measured steps the sweep runs: both code
    widths, both policies, all four cache sizes, uniform indices and every Zipf exponent occur among them."""
    cfg = list(wl.sweep5())[point]
    assert cfg.steps == 100
    _full_size(cfg, [point % 4], cfg.steps, check_at=(50,)).close()


def test_batches_prepared_ahead_give_the_same_results():
    """mpe_prepare sorts the next batch on another stream while the current step runs; the forward of that batch takes
    the result over.  Prepared, unprepared, discarded (other batch than the one prepared) and ignored (does not fit the
    reservation) batches in one run, all equal to the oracle; ids outside a table in a prepared batch are reported."""
    from parity_util import make_pair, compare_state
    from paper_2010_11305_b200 import binding as mpe
    cfg = _cfg(num_rows=[30000, 900, 40], dim=64, bits=4, batch=512, bag=("poisson", 9.0), zipf=[1.1, 0.9, None], policy=wl.LFU, ways=8,
               cache_fraction=0.05, seed=21)
    h, o = make_pair(cfg)
    h.use_graphs(False)                                  # replayed steps ignore the call: this test is about the plain path
    st = wl.Stream(cfg, "cpu")
    rng = np.random.default_rng(0)
    side = torch.cuda.Stream()
    steps = 9
    batches = [st.batch(s) for s in range(1, steps + 2)]
    batches[4][0][::50] = 30000                          # step 5's batch has ids outside its tables
    dev = [(i.cuda(), f.cuda(), g.cuda()) for i, f, g in batches]
    h.reserve(cfg.batch, max(b[0].numel() for b in batches[:7]))
    torch.cuda.synchronize()
    mode = ["prepare", "prepare", "none", "prepare", "wrong", "prepare", "prepare", "too_large", "prepare"]
    for k in range(steps):
        idx, off, grad = dev[k]
        out = torch.empty(cfg.batch, cfg.num_tables * cfg.dim, device="cuda")
        h.forward(idx, off, cfg.batch, out)
        nxt = mode[k]                                    # what happens for step k + 1 while step k runs
        if nxt in ("prepare", "too_large"):
            h.prepare(dev[k + 1][0], dev[k + 1][1], cfg.batch, side.cuda_stream)
        elif nxt == "wrong":
            h.prepare(dev[k][0], dev[k][1], cfg.batch, side.cuda_stream)
        h.backward(grad, cfg.lr, k + 1)
        ref = o.forward(batches[k][0].numpy(), batches[k][1].numpy(), cfg.batch)
        o.backward(batches[k][2].numpy(), cfg.lr, k + 1)
        assert np.array_equal(out.cpu().numpy(), ref), f"step {k + 1}"
        if k == 4:
            code, detail = h.last_error()
            assert code == mpe.ERR_INDEX and detail == int((batches[4][0] == 30000).sum())
        if k % 3 == 2 or k == steps - 1:
            compare_state(h, o, cfg, [0, 1, 2], rng)
    assert h.last_error() == (0, 0)
    one, _ = h.workspace_bytes()
    assert one > 0


def test_launch_mode_cannot_change_between_a_forward_and_its_backward():
    """Replayed kernels read the step's arguments from device memory, plainly launched ones get them by value: the two
    halves of a step must be launched the same way, whatever the caller toggles in between."""
    from parity_util import make_pair, compare_state
    from paper_2010_11305_b200 import binding as mpe
    cfg = _cfg(num_rows=[3000, 400], dim=16, bits=4, batch=48, bag=("poisson", 4.0), zipf=[1.1, 0.9], policy=wl.LFU, ways=4,
               cache_fraction=0.1, seed=12)
    h, o = make_pair(cfg)
    rng = np.random.default_rng(0)
    st = wl.Stream(cfg, "cpu")
    step = 0
    for graphs_fwd, toggle in ((True, "graphs"), (False, "graphs"), (True, "profile"), (False, "profile"), (True, None)):
        step += 1
        h.use_graphs(graphs_fwd)
        idx, off, grad = st.batch(step)
        out = torch.empty(cfg.batch, cfg.num_tables * cfg.dim, device="cuda")
        h.forward(idx.cuda(), off.cuda(), cfg.batch, out)
        with pytest.raises(mpe.MpeError) as e:
            if toggle == "profile":
                h.profile(True)
            else:
                h.use_graphs(not graphs_fwd)
        assert e.value.code == mpe.ERR_SEQUENCE
        h.backward(grad.cuda(), cfg.lr, step)
        assert np.array_equal(out.cpu().numpy(), o.forward(idx.numpy(), off.numpy(), cfg.batch))
        o.backward(grad.numpy(), cfg.lr, step)
        compare_state(h, o, cfg, [0, 1], rng)
    assert h.last_error() == (0, 0)


def test_a_look_back_that_gives_up_is_reported_and_the_handle_goes_on():
    """The sort's tiles learn their output positions from the tiles before them; every such wait is bounded.  The
    library's self-check makes one wait run out (a tile nobody owns, the limit cut to a millisecond): the condition must
    arrive through mpe_last_error, be cleared by it, and leave the handle training exactly as the oracle does."""
    from parity_util import make_pair, compare_state
    from paper_2010_11305_b200 import binding as mpe
    cfg = _cfg(num_rows=[6000, 700], dim=16, bits=8, batch=96, bag=("poisson", 5.0), zipf=[1.1, 1.0], policy=wl.LRU, ways=4,
               cache_fraction=0.1, seed=21)
    rng = np.random.default_rng(0)
    for graphs in (True, False):
        h, o = make_pair(cfg)
        h.use_graphs(graphs)
        st = wl.Stream(cfg, "cpu")
        with pytest.raises(mpe.MpeError) as e:          # no workspace yet
            h.selftest(mpe.SELFTEST_LOOK_BACK_TIMEOUT)
        assert e.value.code == mpe.ERR_SEQUENCE
        for step in range(1, 7):
            idx, off, grad = st.batch(step)
            out = torch.empty(cfg.batch, cfg.num_tables * cfg.dim, device="cuda")
            h.forward(idx.cuda(), off.cuda(), cfg.batch, out)
            if step == 3:
                with pytest.raises(mpe.MpeError) as e:  # not in the middle of a step
                    h.selftest(mpe.SELFTEST_LOOK_BACK_TIMEOUT)
                assert e.value.code == mpe.ERR_SEQUENCE
            h.backward(grad.cuda(), cfg.lr, step)
            assert np.array_equal(out.cpu().numpy(), o.forward(idx.numpy(), off.numpy(), cfg.batch))
            o.backward(grad.numpy(), cfg.lr, step)
            if step in (2, 4):
                assert h.last_error() == (0, 0)
                h.selftest(mpe.SELFTEST_LOOK_BACK_TIMEOUT)
                if step == 4:
                    h.selftest(mpe.SELFTEST_LOOK_BACK_TIMEOUT)
                assert h.last_error() == (mpe.ERR_TIMEOUT, 1 if step == 2 else 2)
                assert h.last_error() == (0, 0)
        compare_state(h, o, cfg, [0, 1], rng)
        assert h.last_error() == (0, 0)
        h.close()


def test_sort_pass_numbers_can_start_over_at_any_step():
    """The per-tile words of the sort carry a pass number that is started over long before it can repeat; forcing that
    between arbitrary steps (also with a batch prepared ahead in the second workspace) must not change any result."""
    from parity_util import make_pair, compare_state
    from paper_2010_11305_b200 import binding as mpe
    cfg = _cfg(num_rows=[9000, 1200, 50], dim=32, bits=4, batch=300, bag=("poisson", 6.0), zipf=[1.1, 1.0, None], policy=wl.LFU,
               ways=8, cache_fraction=0.1, seed=22)
    rng = np.random.default_rng(0)
    for graphs in (True, False):
        h, o = make_pair(cfg)
        h.use_graphs(graphs)
        st = wl.Stream(cfg, "cpu")
        side = torch.cuda.Stream()
        batches = [tuple(x.cuda() for x in st.batch(step)) for step in range(1, 10)]
        host = [st.batch(step) for step in range(1, 10)]
        for i, step in enumerate(range(1, 10)):
            idx, off, grad = batches[i]
            if step in (1, 4, 5, 8):
                if step > 1:
                    h.selftest(mpe.SELFTEST_RENEW_TAGS)
                else:
                    h.reserve(cfg.batch, max(int(b[0].numel()) for b in batches))
                    h.selftest(mpe.SELFTEST_RENEW_TAGS)
            out = torch.empty(cfg.batch, cfg.num_tables * cfg.dim, device="cuda")
            h.forward(idx, off, cfg.batch, out)
            if i + 1 < len(batches):
                h.prepare(batches[i + 1][0], batches[i + 1][1], cfg.batch, side.cuda_stream)
            h.backward(grad, cfg.lr, step)
            hi, ho, hg = host[i]
            assert np.array_equal(out.cpu().numpy(), o.forward(hi.numpy(), ho.numpy(), cfg.batch))
            o.backward(hg.numpy(), cfg.lr, step)
        compare_state(h, o, cfg, [0, 1, 2], rng)
        assert h.last_error() == (0, 0)
        torch.cuda.synchronize()
        h.close()


def test_graph_replay_and_plain_launches_agree_with_the_oracle():
    """Small steps are replayed from a captured CUDA graph; the same handle must give the oracle's results when
    the batch shrinks and grows under one graph, when the workspace regrows, and with graphs switched off."""
    from parity_util import make_pair, compare_state
    cfg = _cfg(num_rows=[4000, 900], dim=32, bits=4, batch=64, bag=("poisson", 5.0), zipf=[1.1, 1.0], policy=wl.LFU, ways=4,
               cache_fraction=0.1, seed=5)
    h, o = make_pair(cfg)
    rng = np.random.default_rng(0)
    step = 0
    for batch, graphs in ((64, True), (64, True), (16, True), (64, True), (200, True), (64, False), (32, True)):
        cfg.batch = batch
        h.use_graphs(graphs)
        step += 1
        idx, off, grad = wl.Stream(cfg, "cpu").batch(step)
        out = torch.empty(batch, cfg.num_tables * cfg.dim, device="cuda")
        h.forward(idx.cuda(), off.cuda(), batch, out)
        ref = o.forward(idx.numpy(), off.numpy(), batch)
        assert np.array_equal(out.cpu().numpy(), ref), f"step {step}"
        h.backward(grad.cuda(), cfg.lr, step)
        o.backward(grad.numpy(), cfg.lr, step)
        compare_state(h, o, cfg, [0, 1], rng)
    assert h.last_error() == (0, 0)


@pytest.mark.parametrize("bits", [8, 4, 2, 16])
def test_round_to_nearest_while_training(bits):
    """Section 3 "Rounding": the nearest-even option instead of stochastic rounding, for updates, evictions and flush."""
    from parity_util import make_pair, compare_state
    from paper_2010_11305_b200 import binding as mpe
    cfg = _cfg(num_rows=[2500, 300], dim=32, bits=bits, batch=80, bag=("poisson", 5.0), zipf=[1.1, 0.9], policy=wl.LFU, ways=4,
               cache_fraction=0.1, seed=9 + bits)
    h, o = make_pair(cfg)
    rng = np.random.default_rng(0)
    st = wl.Stream(cfg, "cpu")
    for step in range(1, 7):
        if step == 1:
            h.set_rounding(mpe.ROUND_NEAREST)
            o.set_rounding(0)
        if step == 5:                                   # and back, on the same handle
            h.set_rounding(mpe.ROUND_STOCHASTIC)
            o.set_rounding(1)
        idx, off, grad = st.batch(step)
        out = torch.empty(cfg.batch, cfg.num_tables * cfg.dim, device="cuda")
        h.forward(idx.cuda(), off.cuda(), cfg.batch, out)
        ref = o.forward(idx.numpy(), off.numpy(), cfg.batch)
        assert np.array_equal(out.cpu().numpy(), ref)
        if step == 3:
            with pytest.raises(mpe.MpeError) as e:      # not between a forward and its backward
                h.set_rounding(mpe.ROUND_STOCHASTIC)
            assert e.value.code == mpe.ERR_SEQUENCE
        h.backward(grad.cuda(), cfg.lr, step)
        o.backward(grad.numpy(), cfg.lr, step)
        compare_state(h, o, cfg, [0, 1], rng)
        if step in (4, 6):
            h.flush()
            o.flush()
            compare_state(h, o, cfg, [0, 1], rng)


@pytest.mark.parametrize("bits,policy", [(4, wl.LFU), (16, wl.LRU)])
def test_table_in_host_memory_gives_the_same_results(bits, policy):
    """Capacity tiering (Section 5.2): the low-precision table in pinned host memory, the FP32 cache in HBM."""
    from parity_util import make_pair, compare_state
    from paper_2010_11305_b200 import binding as mpe
    cfg = _cfg(num_rows=[20000, 700], dim=64, bits=bits, batch=128, bag=("poisson", 8.0), zipf=[1.1, 1.0], policy=policy, ways=8,
               cache_fraction=0.05, seed=31)
    h, o = make_pair(cfg, table_placement=mpe.TABLE_HOST)
    rng = np.random.default_rng(0)
    st = wl.Stream(cfg, "cpu")
    for step in range(1, 6):
        idx, off, grad = st.batch(step)
        out = torch.empty(cfg.batch, cfg.num_tables * cfg.dim, device="cuda")
        h.forward(idx.cuda(), off.cuda(), cfg.batch, out)
        ref = o.forward(idx.numpy(), off.numpy(), cfg.batch)
        assert np.array_equal(out.cpu().numpy(), ref)
        h.backward(grad.cuda(), cfg.lr, step)
        o.backward(grad.numpy(), cfg.lr, step)
    compare_state(h, o, cfg, [0, 1], rng)
    h.flush()
    o.flush()
    compare_state(h, o, cfg, [0, 1], rng)


@pytest.mark.parametrize("seed", range(40))
def test_random_configurations(seed):
    """Configurations drawn at random: table counts and sizes (down to a few rows), every code width, both policies and
    optimizers, every associativity, bag shapes from one-hot to long ragged bags, cache sizes from none to most of a table.
    Rows with 65..1024 occurrences (the boundary between the per-warp and the multi-block gradient paths) and tables
    that end inside a block of distinct rows come up by construction."""
    from parity_util import run_parity
    rng = np.random.default_rng(1000 + seed)
    T = int(rng.integers(1, 7))
    num_rows = [int(rng.choice([3, 17, 200, 2000, 30000, 400000])) for _ in range(T)]
    dim = int(rng.choice([4, 8, 16, 32, 64, 128]))
    bits = int(rng.choice([2, 4, 8, 16]))
    ways = int(rng.choice([1, 2, 4, 8, 16, 32]))
    policy = int(rng.choice([wl.LRU, wl.LFU]))
    opt = int(rng.choice([wl.SGD, wl.ROWWISE_ADAGRAD]))
    bag = [("fixed", 1), ("fixed", 7), ("poisson", 3.0), ("poisson_cap", 25.0, 60), ("poisson", 0.4)][int(rng.integers(0, 5))]
    zipf = [[None, 0.7, 1.05, 1.3, 2.0][int(rng.integers(0, 5))] for _ in range(T)]
    cfg = _cfg(name=f"rnd{seed}", num_rows=num_rows, dim=dim, bits=bits, ways=ways, policy=policy, optimizer=opt,
               cache_fraction=float(rng.choice([0.0, 0.01, 0.1, 0.6])), batch=int(rng.choice([1, 33, 256, 1500])), bag=bag, zipf=zipf,
               lr=0.05, steps=5, seed=seed)
    run_parity(cfg, 5, check_every=2)


@pytest.mark.parametrize("policy,ways", [(wl.LFU, 8), (wl.LFU, 1), (wl.LRU, 4)])
def test_many_steps_keep_the_recorded_set_bounds_valid(policy, ways):
    """Sixty steps on small tables: residents are replaced again and again, counts and time stamps keep growing, and the
    per-set lower bounds that let the priority kernel bypass candidates early must never reject a row that Algorithm 2
    would admit (state, counters and statistics stay bit-equal to the oracle throughout)."""
    from parity_util import run_parity
    cfg = _cfg(num_rows=[600, 90, 2500], dim=16, bits=4, policy=policy, ways=ways, cache_fraction=0.1, batch=48,
               bag=("poisson", 3.0), zipf=[1.1, 0.8, 1.3], steps=60, seed=77)
    h, o, _ = run_parity(cfg, 60, check_every=10)
    s = h.stats(0)
    assert s[4] > 0 and s[6] > 0            # admissions and bypasses both happened
