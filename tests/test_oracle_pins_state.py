"""Pins of the oracle's snapshot operation and of its input handling (no GPU).

Covers what the step-by-step pins leave open: `flush` (every resident row is
down-converted into the table with its own random stream and stays resident),
row ids outside the table (dropped everywhere), inconsistent offsets (refused,
state untouched) and the table mask (a masked run equals a run in which the
masked tables simply receive no indices).  Expected values come from the
independent single-array emulator's quantizer, from closed forms, or from a
second oracle run on inputs that make the feature under test a no-op.
"""
import numpy as np
import pytest

from oracle import literal_emulator as emu
from oracle import mpe_oracle as orc

F = np.float32
FLUSH_DOMAIN = 3          # the emulator's spelling of the flush stream; the step's own stream is 2


def _arrays(bags_per_table):
    batch = len(bags_per_table[0])
    idx, off = [], [0]
    for bags in bags_per_table:
        assert len(bags) == batch
        for bag in bags:
            idx.extend(bag)
            off.append(len(idx))
    return np.array(idx, np.int32), np.array(off, np.int32), batch


def _random_bags(rng, num_rows, batch, hot=None):
    out = []
    for t, N in enumerate(num_rows):
        bags = []
        for _ in range(batch):
            n = int(rng.integers(0, 5))
            bag = [int(hot[t]) if hot is not None and rng.random() < 0.3 else int(rng.integers(0, N)) for _ in range(n)]
            bags.append(bag)
        out.append(bags)
    return out


def _entries(o, num_rows):
    return [[o.row(t, r) for r in range(N)] for t, N in enumerate(num_rows)]


def _same_entry(a, b):
    return np.array_equal(a[0], b[0]) and a[1].tobytes() == b[1].tobytes() and a[2].tobytes() == b[2].tobytes()


def _expected_entry(x, bits, mode, key):
    """Low-precision entry of the FP32 row x, by the emulator's own quantizer (not the oracle's)."""
    if bits == 16:
        vals = emu.fake_half(x, mode, key)[0]
        return vals.astype(np.float16).view(np.uint8), F(1.0), F(0.0)      # the values are FP16-representable: exact
    _, codes, s, b = emu.fake_quantize(x, bits, mode, key)
    return orc.pack(codes.astype(np.uint8), bits), F(s), F(b)


def _train(o, num_rows, d, steps, rng, first_step=1, hot=None, lr=0.05):
    B = 6
    for step in range(first_step, first_step + steps):
        idx, off, _ = _arrays(_random_bags(rng, num_rows, B, hot))
        o.forward(idx, off, B)
        o.backward(rng.normal(0, 0.05, (B, len(num_rows) * d)).astype(F), lr, step)
    return first_step + steps - 1


# ------------------------------------------------------------------ flush ---
@pytest.mark.parametrize("bits,policy,ways,nearest", [(8, orc.LRU, 4, False), (4, orc.LFU, 2, False), (2, orc.LFU, 4, False),
                                                       (16, orc.LRU, 2, False), (8, orc.LFU, 4, True), (16, orc.LFU, 4, True)])
def test_flush_down_converts_every_resident_with_its_own_stream_and_changes_nothing_else(bits, policy, ways, nearest):
    num_rows, d, seed = [48, 30], 8, 17
    o = orc.Oracle(num_rows, d, bits, 0.25, ways, policy, seed=seed)
    if nearest:
        o.set_rounding(orc.RTN)
    mode = "nearest" if nearest else "stochastic"
    rng = np.random.default_rng(bits + ways)
    last = _train(o, num_rows, d, 6, rng, hot=[3, 5])
    before_entries = _entries(o, num_rows)
    before_cache = [tuple(a.copy() for a in o.cache(t)) for t in range(2)]
    before_values = [[o.fetch_value(t, r) for r in range(N)] for t, N in enumerate(num_rows)]
    before_cnt = [[o.cnt(t, r) for r in range(N)] for t, N in enumerate(num_rows)]
    before_stats = [o.stats(t).copy() for t in range(2)]
    o.flush()
    differs_from_step_stream = 0
    residents = 0
    for t, N in enumerate(num_rows):
        tags, rows, ts = o.cache(t)
        assert tags[0] >= 0                                               # the very first slot is occupied, so it is covered below
        for a, b in zip(before_cache[t], (tags, rows, ts)):               # the cache is bit-unchanged: rows stay resident
            assert a.tobytes() == b.tobytes()
        res = set()
        for slot, r in enumerate(tags):
            if r < 0:
                continue
            res.add(int(r))
            residents += 1
            want = _expected_entry(rows[slot], bits, mode, emu.rowkey(seed, FLUSH_DOMAIN, t, int(r), last))
            got = o.row(t, int(r))
            assert _same_entry(got, want), (t, slot, int(r))
            if not nearest:
                other = _expected_entry(rows[slot], bits, mode, emu.rowkey(seed, 2, t, int(r), last))
                differs_from_step_stream += not _same_entry(got, other)
            if bits != 16:                                                # closed forms of Algorithm 1 on the cached row
                x = rows[slot]
                assert got[2] == x.min() + F(0.0) and got[1] == F((x.max() - x.min()) / F(2 ** bits - 1))
                y = (x.astype(np.float64) - float(got[2])) / float(got[1])
                assert np.all(np.abs(orc.unpack(got[0], d, bits) - y) < 1.0 + 1e-4)
        for r in range(N):
            if r not in res:
                assert _same_entry(o.row(t, r), before_entries[t][r]), (t, r)     # non-resident entries untouched
            assert np.array_equal(o.fetch_value(t, r), before_values[t][r])         # what fetch returns is unchanged
            assert o.cnt(t, r) == before_cnt[t][r]
        assert np.array_equal(o.stats(t), before_stats[t])
    assert residents >= 6
    if not nearest:
        assert differs_from_step_stream >= residents // 2          # the flush draws its own bits, not the step's
    again = _entries(o, num_rows)
    o.flush()                                                      # same step, same bits: flushing twice is idempotent
    for t, N in enumerate(num_rows):
        for r in range(N):
            assert _same_entry(o.row(t, r), again[t][r])


@pytest.mark.parametrize("policy", [orc.LRU, orc.LFU])
def test_training_is_the_same_with_and_without_flushes_and_a_later_eviction_overwrites_the_flushed_entry(policy):
    """In the single-array emulation a flush changes nothing (residents stay FP32): every fetched value, tag and
    priority value of a run with flushes equals the run without, and so does the table entry of every row that is
    not resident (an eviction after a flush writes the eviction's entry over the flushed one)."""
    num_rows, d, seed, bits, ways = [40], 8, 5, 8, 2
    a = orc.Oracle(num_rows, d, bits, 0.2, ways, policy, seed=seed)
    b = orc.Oracle(num_rows, d, bits, 0.2, ways, policy, seed=seed)
    rng = np.random.default_rng(11)
    flushed_at = {}                      # row -> step of the last flush that saw it resident
    evicted_after_flush = 0
    B = 6
    for step in range(1, 25):
        idx, off, _ = _arrays(_random_bags(rng, num_rows, B))
        grad = rng.normal(0, 0.05, (B, d)).astype(F)
        assert np.array_equal(a.forward(idx, off, B), b.forward(idx, off, B))
        tags_before, rows_before, _ = (x.copy() for x in b.cache(0))
        a.backward(grad, 0.05, step)
        b.backward(grad, 0.05, step)
        ta, ra, tsa = a.cache(0)
        tb, rb, tsb = b.cache(0)
        assert np.array_equal(ta, tb) and ra.tobytes() == rb.tobytes() and np.array_equal(tsa, tsb)
        resident = set(int(r) for r in tb if r >= 0)
        for r in range(num_rows[0]):
            assert np.array_equal(a.fetch_value(0, r), b.fetch_value(0, r))
            if r not in resident:
                assert _same_entry(a.row(0, r), b.row(0, r)), (step, r)
        urows = set(int(r) for r in b.last_unique(0)[0])
        for slot, r in enumerate(tags_before):
            r = int(r)
            if r >= 0 and r not in resident and r in flushed_at and r not in urows:
                # resident at a flush, evicted now without being updated: the entry is the eviction's, drawn from this step's stream
                want = _expected_entry(rows_before[slot], bits, "stochastic", emu.rowkey(seed, 2, 0, r, step))
                assert _same_entry(b.row(0, r), want)
                evicted_after_flush += 1
                del flushed_at[r]
        if step % 3 == 0:
            b.flush()
            for r in resident:
                flushed_at[r] = step
    assert evicted_after_flush >= 3


# ------------------------------------------------- ids outside the table ---
@pytest.mark.parametrize("policy", [orc.LRU, orc.LFU])
def test_ids_outside_the_table_are_dropped_everywhere(policy):
    num_rows, d = [20, 12], 4
    bad0, bad1 = [-1, 20, 2 ** 31 - 1, -7], [12, 13, -2 ** 31]
    bags = [[[5, bad0[0], 7], [bad0[1]], [7, 7, bad0[2], 3], [], [bad0[3], 19, 0]],
            [[11, bad1[0]], [bad1[1], bad1[2]], [2], [11, 11], []]]
    clean = [[[r for r in bag if 0 <= r < N] for bag in tb] for tb, N in zip(bags, num_rows)]
    o = orc.Oracle(num_rows, d, 8, 0.25, 2, policy, seed=3)
    ref = orc.Oracle(num_rows, d, 8, 0.25, 2, policy, seed=3)
    rng = np.random.default_rng(0)
    for step in (1, 2, 3):
        grad = rng.normal(0, 0.1, (5, 2 * d)).astype(F)
        idx, off, B = _arrays(bags)
        cidx, coff, _ = _arrays(clean)
        out = o.forward(idx, off, B)
        assert o.dropped() == 7 * step                                   # every bad occurrence counted once per forward
        assert np.array_equal(out, ref.forward(cidx, coff, B))           # they add nothing to any bag
        o.backward(grad, 0.1, step)
        ref.backward(grad, 0.1, step)
        for t, N in enumerate(num_rows):
            urows, mult, grads = o.last_unique(t)
            rrows, rmult, rgrads = ref.last_unique(t)
            assert urows.min() >= 0 and urows.max() < N                  # and are no key of the de-duplication
            assert np.array_equal(urows, rrows) and np.array_equal(mult, rmult) and np.array_equal(grads, rgrads)
            assert sorted(o.touched(t)) == sorted(ref.touched(t))        # no record was made for them either
            for r in range(N):
                assert _same_entry(o.row(t, r), ref.row(t, r))
                assert o.cnt(t, r) == ref.cnt(t, r)
            for x, y in zip(o.cache(t), ref.cache(t)):
                assert x.tobytes() == y.tobytes()
            assert np.array_equal(o.stats(t), ref.stats(t))
            assert o.stats(t)[0] == step * sum(len(bag) for bag in clean[t])    # lookups count valid indices only
    assert ref.dropped() == 0


# ------------------------------------------------------ bad offset vectors ---
def test_inconsistent_offsets_are_refused_and_leave_the_state_alone():
    o = orc.Oracle([100], 8, 8, 0.1, 2, orc.LRU, seed=1)
    idx = np.array([1, 2, 3, 4, 5, 6], np.int32)
    good = np.array([0, 2, 3, 4, 6], np.int32)
    grad = np.ones((4, 8), F)
    o.forward(idx, good, 4)
    o.backward(grad, 0.1, 1)
    entries = [o.row(0, r) for r in range(100)]
    cache = [x.copy() for x in o.cache(0)]
    stats = o.stats(0).copy()
    # decreasing in the middle, not starting at 0, not ending at the total, running past the total, negative
    for bad in ([0, 2, 1, 4, 6], [1, 2, 3, 4, 6], [0, 2, 3, 4, 5], [0, 2, 9, 4, 6], [0, -2, 3, 4, 6]):
        with pytest.raises(orc.OracleError) as e:
            o.forward(idx, np.array(bad, np.int32), 4)
        assert e.value.code == orc.ERR_OFFSETS
        with pytest.raises(orc.OracleError) as e:                         # the refused forward is no forward: nothing to back-propagate
            o.backward(grad, 0.1, 2)
        assert e.value.code == orc.ERR_SEQUENCE
        assert all(_same_entry(o.row(0, r), entries[r]) for r in range(100))
        assert all(x.tobytes() == y.tobytes() for x, y in zip(o.cache(0), cache))
        assert np.array_equal(o.stats(0), stats) and o.dropped() == 0
    out = o.forward(idx, good, 4)                                         # and the oracle still works
    assert np.array_equal(out[0], (o.fetch_value(0, 1) + o.fetch_value(0, 2)).astype(F))
    o.backward(grad, 0.1, 2)
    assert o.stats(0)[7] == 2


# -------------------------------------------------------------- table mask ---
@pytest.mark.parametrize("policy", [orc.LRU, orc.LFU])
def test_masked_tables_are_skipped_and_the_others_do_not_notice(policy):
    """A run restricted to tables {0, 2} equals, on those tables, an unrestricted run whose table 1 receives no
    indices (same table ids, hence the same hash streams); the masked table keeps its initial state."""
    num_rows, d, B = [30, 25, 40], 4, 5
    m = orc.Oracle(num_rows, d, 4, 0.2, 2, policy, seed=9)
    m.set_table_mask([1, 0, 1])
    u = orc.Oracle(num_rows, d, 4, 0.2, 2, policy, seed=9)
    rng = np.random.default_rng(4)
    cols = np.r_[0:d, 2 * d:3 * d]
    for step in range(1, 7):
        bags = _random_bags(rng, num_rows, B)
        bags[1][0] = [1, 2, 3]                                            # the masked table always has work on offer
        idx, off, _ = _arrays(bags)
        eidx, eoff, _ = _arrays([bags[0], [[] for _ in range(B)], bags[2]])
        grad = rng.normal(0, 0.1, (B, 3 * d)).astype(F)
        om, ou = m.forward(idx, off, B), u.forward(eidx, eoff, B)
        assert np.array_equal(om[:, cols], ou[:, cols])
        assert not om[:, d:2 * d].any()                                   # nothing is written for the masked table
        m.backward(grad, 0.1, step)
        u.backward(grad, 0.1, step)
        if step == 4:
            m.flush()
            u.flush()
        for t in (0, 2):
            for r in range(num_rows[t]):
                assert _same_entry(m.row(t, r), u.row(t, r))
                assert m.cnt(t, r) == u.cnt(t, r)
            for x, y in zip(m.cache(t), u.cache(t)):
                assert x.tobytes() == y.tobytes()
            assert np.array_equal(m.stats(t), u.stats(t))
            a, b = m.last_unique(t), u.last_unique(t)
            assert all(np.array_equal(x, y) for x, y in zip(a, b))
        assert m.touched(1).size == 0 and not m.stats(1).any() and np.all(m.cache(1)[0] == -1)
    assert u.stats(1)[7] == 6 and u.stats(1)[0] == 0                      # the unrestricted run did visit table 1, with nothing to do
    m.set_table_mask(None)                                                # lifting the mask brings the table back
    idx, off, _ = _arrays([[[0]] * B, [[1, 2]] * B, [[0]] * B])
    out = m.forward(idx, off, B)
    assert np.array_equal(out[0, d:2 * d], (m.fetch_value(1, 1) + m.fetch_value(1, 2)).astype(F))
    # a flush under the mask leaves the masked table's stale entries alone and still snapshots the others
    m.backward(np.ones((B, 3 * d), F), 0.1, 7)
    assert (m.cache(1)[0] >= 0).any()
    m.set_table_mask([1, 0, 1])
    stale = [m.row(1, r) for r in range(num_rows[1])]
    before0 = [m.row(0, r) for r in range(num_rows[0])]
    m.flush()
    assert all(_same_entry(m.row(1, r), stale[r]) for r in range(num_rows[1]))
    assert any(not _same_entry(m.row(0, r), before0[r]) for r in range(num_rows[0]))
