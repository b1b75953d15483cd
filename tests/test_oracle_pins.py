"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests needs a GPU.  Each one is chosen so that a plausible
mistake in the oracle (dropped term, wrong sign or index, transposed operand,
wrong comparison direction) makes it fail.
"""
import os

import numpy as np
import pytest
import torch

from oracle import mpe_oracle as orc
from oracle import literal_emulator as emu

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
F = np.float32


def _bags_to_arrays(bags_per_table):
    """bags_per_table[t][b] = list of rows -> (indices, offsets, batch) in table-major layout."""
    batch = len(bags_per_table[0])
    idx, off = [], [0]
    for bags in bags_per_table:
        assert len(bags) == batch
        for bag in bags:
            idx.extend(bag)
            off.append(len(idx))
    return np.array(idx, np.int32), np.array(off, np.int32), batch


# ---------------------------------------------------------------- hash ---
def test_mix32_is_a_bijection_with_avalanche():
    rng = np.random.default_rng(0)
    xs = rng.integers(0, 2 ** 32, 2000, dtype=np.uint64)
    flips = []
    for x in xs[:300]:
        h = orc.mix32(int(x))
        for bit in range(32):
            flips.append(bin(h ^ orc.mix32(int(x) ^ (1 << bit))).count("1"))
    assert 15.0 < np.mean(flips) < 17.0            # half of the output bits flip on average
    assert len({orc.mix32(int(x)) for x in range(100000)}) == 100000
    assert orc.mix32(12345) == emu.mix32(12345)    # two independent spellings of the convention


def test_uniform_draws_are_uniform_and_distinct_per_field():
    key = orc.rowkey(7, orc.DOMAIN_SR, 3, 11, 5)
    u = np.array([orc.uniform(key, c) for c in range(20000)])
    assert 0.0 <= u.min() and u.max() < 1.0
    assert abs(u.mean() - 0.5) < 0.01 and abs(u.var() - 1 / 12) < 0.005
    keys = {orc.rowkey(7, orc.DOMAIN_SR, 3, 11, 5), orc.rowkey(8, orc.DOMAIN_SR, 3, 11, 5),
            orc.rowkey(7, orc.DOMAIN_FLUSH, 3, 11, 5), orc.rowkey(7, orc.DOMAIN_SR, 4, 11, 5),
            orc.rowkey(7, orc.DOMAIN_SR, 3, 12, 5), orc.rowkey(7, orc.DOMAIN_SR, 3, 11, 6),
            orc.rowkey(7 + (1 << 32), orc.DOMAIN_SR, 3, 11, 5), orc.rowkey(7, orc.DOMAIN_SR, 3, 11, 5 + (1 << 32))}
    assert len(keys) == 8
    assert key == emu.rowkey(7, 2, 3, 11, 5)


def test_set_hash_range_and_spread():
    s = orc.salt(0, 0)
    n = 62
    sets = np.array([orc.set_index(r, s, n) for r in range(10000)])
    assert sets.min() == 0 and sets.max() == n - 1
    counts = np.bincount(sets, minlength=n)
    assert counts.min() > 100 and counts.max() < 230     # 10000/62 = 161 expected per set
    assert orc.set_index(123, s, n) == emu.set_hash(123, 0, 0, n)


def test_num_sets_follows_the_budget():
    assert orc.num_sets(10_000, 0.05, 8) == 62           # 500 rows -> 62 sets of 8 (never exceeds the budget)
    assert orc.num_sets(5_000_000, 0.01, 32) == 1562
    assert orc.num_sets(20_000_000, 0.01, 16) == 12500
    assert orc.num_sets(3, 0.05, 32) == 1                # tiny table: one set, effectively FP32
    assert orc.num_sets(1000, 0.0, 32) == 0              # no cache


# ----------------------------------------------------------- quantizer ---
@pytest.mark.parametrize("bits", [8, 4, 2])
@pytest.mark.parametrize("d", [4, 16, 64, 128])
def test_quantizer_closed_forms(bits, d):
    rng = np.random.default_rng(bits * 100 + d)
    qmax = 2 ** bits - 1
    for trial in range(200):
        x = rng.uniform(-0.05, 0.05, d).astype(F)
        q, s, b = orc.quantize(x, bits, orc.RTN)
        assert b == x.min() and s == F((x.max() - x.min()) / F(qmax))      # b = min, s = (max-min)/(2^N-1)
        assert q[np.argmin(x)] == 0 and q[np.argmax(x)] == qmax
        xd = orc.dequantize(q, s, b)
        assert np.all(np.abs(xd.astype(np.float64) - x) <= 0.5 * float(s) * (1 + 1e-5))   # nearest: error <= s/2
        # exact value of y, then nearest-even rounding, in float64 as an independent route
        y = (x.astype(np.float64) - float(b)) / float(s)
        assert np.all(np.abs(q - y) <= 0.5 + 1e-4)
        # Algorithm 1 applied twice changes nothing (fake quantization is idempotent)
        q2, s2, b2 = orc.quantize(xd, bits, orc.RTN)
        assert np.array_equal(q, q2) and b2 == b
        # stochastic rounding returns one of the two neighbours
        key = orc.rowkey(1, orc.DOMAIN_SR, 0, trial, 1)
        qs, ss, bs = orc.quantize(x, bits, orc.SR, key)
        assert ss == s and bs == b
        assert np.all((qs == np.floor(y + 1e-4)) | (qs == np.ceil(y - 1e-4)) | (np.abs(qs - y) < 1.0))
        assert np.all(np.abs(qs.astype(np.float64) - y) < 1.0 + 1e-4)
        assert qs.min() >= 0 and qs.max() <= qmax


def test_nearest_rounding_breaks_ties_to_even():
    # codes 0..255 with scale exactly 1: inputs k + 0.5 must go to the even neighbour
    x = np.array([0.0, 0.5, 1.5, 2.5, 3.5, 100.5, 101.5, 255.0], F)
    q, s, b = orc.quantize(x, 8, orc.RTN)
    assert s == 1.0 and b == 0.0
    assert list(q) == [0, 0, 2, 2, 4, 100, 102, 255]
    x4 = np.array([0.0, 0.5, 1.5, 2.5, 7.5, 8.5, 14.5, 15.0], F)
    q4, s4, _ = orc.quantize(x4, 4, orc.RTN)
    assert s4 == 1.0 and list(q4) == [0, 0, 2, 2, 8, 8, 14, 15]


def test_constant_and_degenerate_rows_round_trip():
    for v in (0.0, -0.0, 0.125, -3.5, 1e-30):
        x = np.full(16, v, F)
        for mode in (orc.RTN, orc.SR):
            q, s, b = orc.quantize(x, 8, mode, 99)
            assert s == 0.0 and not np.signbit(s) and np.all(q == 0)
            assert np.array_equal(orc.dequantize(q, s, b), x + F(0.0))
    x = np.zeros(16, F)
    x[3] = 1e-44   # range below the smallest normal scale: treated as constant, must not divide by ~0
    q, s, b = orc.quantize(x, 8, orc.RTN)
    assert s == 0.0 and np.all(q == 0)


def test_int4_packing_low_nibble_first():
    q = np.arange(16, dtype=np.uint8)
    p = orc.pack(q, 4)
    assert list(p) == [0x10, 0x32, 0x54, 0x76, 0x98, 0xBA, 0xDC, 0xFE]
    assert np.array_equal(orc.unpack(p, 16, 4), q)
    assert np.array_equal(orc.pack(q, 8), q)
    q2 = np.array([0, 1, 2, 3, 3, 2, 1, 0], np.uint8)          # INT2: four codes per byte, lowest column in the lowest bits
    p2 = orc.pack(q2, 2)
    assert list(p2) == [0b11100100, 0b00011011]
    assert np.array_equal(orc.unpack(p2, 8, 2), q2)


@pytest.mark.parametrize("bits", [8, 4, 2])
def test_stochastic_rounding_is_unbiased_and_nearest_is_not(bits):
    rng = np.random.default_rng(5)
    d, K = 16, 100_000
    x = rng.uniform(-0.05, 0.05, d).astype(F)
    acc = np.zeros(d, np.float64)
    for step in range(1, K + 1):
        q, s, b = orc.quantize(x, bits, orc.SR, orc.rowkey(3, orc.DOMAIN_SR, 0, 17, step))
        acc += orc.dequantize(q, s, b)
    mean = acc / K
    s = float(s)
    # a Bernoulli rounding error has standard deviation <= s/2; allow 4.5 sigma of the mean
    assert np.all(np.abs(mean - x) <= 4.5 * (s / 2) / np.sqrt(K) + 1e-9)
    qn, sn, bn = orc.quantize(x, bits, orc.RTN)
    bias_rtn = np.abs(orc.dequantize(qn, sn, bn).astype(np.float64) - x)
    assert bias_rtn.max() > 20 * (s / 2) / np.sqrt(K)     # nearest rounding keeps a systematic error
    # successive steps really draw different bits
    q1, _, _ = orc.quantize(x, bits, orc.SR, orc.rowkey(3, orc.DOMAIN_SR, 0, 17, 1))
    q2, _, _ = orc.quantize(x, bits, orc.SR, orc.rowkey(3, orc.DOMAIN_SR, 0, 17, 2))
    assert not np.array_equal(q1, q2)


def test_stochastic_rounding_probability_matches_fraction():
    # y = 0, 0.25, ..., 3 with scale 1: P(round up) must equal the fractional part
    x = np.array([0.0, 0.25, 0.5, 0.75, 1.0, 1.25, 2.9, 255.0], F)
    ups = np.zeros(8)
    K = 40000
    for step in range(K):
        q, s, b = orc.quantize(x, 8, orc.SR, orc.rowkey(0, orc.DOMAIN_SR, 0, 0, step))
        ups += q - np.floor(x)
    frac = (x - np.floor(x)).astype(np.float64)
    assert np.all(np.abs(ups / K - frac) < 0.012)
    assert ups[0] == 0 and ups[4] == 0 and ups[7] == 0    # exact integers never move


# ------------------------------------------------------ gradient merge ---
def test_dedup_example_from_section_5_1():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "dedup_example.txt")) if not l.startswith("#")]
    d = 4
    g1 = np.array([1.0, -2.0, 0.5, 4.0], F)
    g2 = np.array([0.25, 8.0, -1.0, 2.0], F)
    o = orc.Oracle([8], d, 8, 0.0, 8, orc.LRU)
    idx, off, B = _bags_to_arrays([[[1, 2], [2, 3]]])
    before = {r: o.fetch_value(0, r) for r in (0, 1, 2, 3, 4)}
    o.forward(idx, off, B)
    o.backward(np.stack([g1, g2]), 0.0, 1)
    urows, mult, grads = o.last_unique(0)
    assert list(urows) == [1, 2, 3] and list(mult) == [1, 2, 1]
    for r, c1, c2 in rows:
        k = list(urows).index(int(r))
        assert np.array_equal(grads[k], F(c1) * g1 + F(c2) * g2)
    del before


def test_tree_sum_shape():
    rng = np.random.default_rng(1)
    for m in (1, 2, 31, 32, 33, 64, 65, 1000, 1024, 1025, 1057, 33000):
        terms = rng.normal(0, 1, (m, 4)).astype(F)
        got = orc.tree_sum(terms)
        # exact sum in float64 bounds the error; and the tree equals the independent Python spelling
        assert np.allclose(got, terms.astype(np.float64).sum(0), rtol=0, atol=1e-3 * np.sqrt(m))
        if m <= 1100:
            assert np.array_equal(got, emu.tree_sum([t for t in terms]))
    # up to 32 terms the order is plain left to right
    t = np.array([[1e8], [1.0], [-1e8], [1.0]], F)
    assert orc.tree_sum(t)[0] == F(F(F(F(1e8) + F(1.0)) + F(-1e8)) + F(1.0))
    # 33 terms: first 32 are summed, then the 33rd is added to that sum
    t = np.ones((33, 1), F)
    t[0] = 2 ** 24
    assert orc.tree_sum(t)[0] == F(2 ** 24) + F(1.0)      # 31 ones are lost one by one, the last one too
    t = np.ones((64, 1), F)
    t[0] = 2 ** 24
    assert orc.tree_sum(t)[0] == F(2 ** 24 + 32)          # the second chunk sums to 32 before it meets 2^24


# ------------------------------------------- Algorithm 2 by hand (P3) ----
def _run_stream(policy, N, frac, ways, steps, d=4):
    o = orc.Oracle([N], d, 8, frac, ways, policy, seed=1)
    assert o.sets(0) == 1
    hist = []
    for step, rows in enumerate(steps, start=1):
        idx, off, B = _bags_to_arrays([[rows]])
        o.forward(idx, off, B)
        o.backward(np.full((1, d), 0.01, F), 0.1, step)
        tags, _, ts = o.cache(0)
        hist.append((list(tags), list(ts)))
    return o, hist


def test_algorithm2_lru_two_way_by_hand():
    o, h = _run_stream(orc.LRU, 10, 0.2, 2, [[3], [5], [3, 7], [5, 8], [5, 1, 2]])
    assert h[0] == ([3, -1], [1, 0])            # empty way filled first
    assert h[1] == ([3, 5], [1, 2])
    assert h[2] == ([3, 7], [3, 3])             # 3 is refreshed, 7 evicts the older 5
    assert h[3] == ([5, 8], [4, 4])             # tie on timestamp 3 -> lowest way first
    assert h[4] == ([5, 1], [5, 5])             # 2 meets only rows touched in this step: PV[i] <= PV[j] -> bypass
    s = o.stats(0)
    assert s[4] == 6 and s[5] == 4 and s[6] == 1 and s[3] == 2   # admissions, evictions, bypasses, unique hits


def test_algorithm2_lfu_two_way_by_hand():
    o, h = _run_stream(orc.LFU, 10, 0.2, 2, [[3, 3, 3], [5], [7], [7], [5, 5, 5, 5], [7, 7, 7, 7, 3]])
    tags = [x[0] for x in h]
    assert tags[0] == [3, -1]
    assert tags[1] == [3, 5]
    assert tags[2] == [3, 5]                    # count(7)=1 is not higher than the lowest resident count 1: bypass
    assert tags[3] == [3, 7]                    # count(7)=2 > 1: replace 5
    assert tags[4] == [3, 5]                    # count(5)=5 > count(7)=2
    assert tags[5] == [7, 5]                    # 3 is hit (count 4) and still the minimum: evicted in the same step
    assert [o.cnt(0, r) for r in (3, 5, 7)] == [4, 5, 6]
    assert o.cnt(0, 0) == 0


def test_algorithm2_direct_mapped():
    _, h = _run_stream(orc.LRU, 10, 0.1, 1, [[2], [2, 4], [6, 8]])
    assert [x[0] for x in h] == [[2], [4], [8]]           # direct-mapped LRU always replaces
    _, h = _run_stream(orc.LFU, 10, 0.1, 1, [[2, 2], [4], [4, 4]])
    assert [x[0] for x in h] == [[2], [2], [4]]           # LFU still compares counts


def test_evicted_row_is_down_converted_and_newcomer_is_verbatim():
    d = 8
    o = orc.Oracle([10], d, 8, 0.1, 1, orc.LRU, seed=3)
    g = np.linspace(-1, 1, d).astype(F)[None, :]
    x2 = o.fetch_value(0, 2)
    idx, off, B = _bags_to_arrays([[[2]]])
    o.forward(idx, off, B)
    o.backward(g, 0.5, 1)
    want2 = (x2 - F(0.5) * g[0]).astype(F)
    assert np.allclose(o.fetch_value(0, 2), want2, rtol=1e-6, atol=0)        # FP32, not re-quantized
    codes_stale, _, _ = o.row(0, 2)
    x4 = o.fetch_value(0, 4)
    idx, off, B = _bags_to_arrays([[[4]]])
    o.forward(idx, off, B)
    o.backward(g, 0.5, 2)
    tags, rows, _ = o.cache(0)
    assert list(tags) == [4] and np.allclose(rows[0], x4 - F(0.5) * g[0], rtol=1e-6, atol=0)
    # row 2 was evicted: its table entry is now the stochastic rounding of its FP32 value
    codes, s, b = o.row(0, 2)
    q, s_ref, b_ref = orc.quantize(o.fetch_value(0, 2) * 0 + want2, 8, orc.SR, orc.rowkey(3, orc.DOMAIN_SR, 0, 2, 2))
    assert b == want2.min() and s == F((want2.max() - want2.min()) / F(255))
    y = (want2.astype(np.float64) - float(b)) / float(s)
    assert np.all(np.abs(orc.unpack(codes, d, 8) - y) < 1.0 + 1e-4)
    assert np.array_equal(orc.unpack(codes, d, 8), q) and s == s_ref and b == b_ref
    del codes_stale


# ----------------------------------------------- full cache == FP32 (P5) -
@pytest.mark.parametrize("policy", [orc.LRU, orc.LFU])
@pytest.mark.parametrize("opt", [orc.SGD, orc.ROWWISE_ADAGRAD])
def test_full_cache_equals_fp32_embedding_bag_training(policy, opt):
    N, d, B, T, lr, eps = 32, 16, 24, 2, 0.1, 1e-8
    o = orc.Oracle([N] * T, d, 8, 1.0, 32, policy, optimizer=opt, eps=eps, seed=11)
    assert o.sets(0) == 1
    W = [torch.tensor(np.stack([o.fetch_value(t, r) for r in range(N)])) for t in range(T)]
    G = [torch.zeros(N) for _ in range(T)]
    rng = np.random.default_rng(2)
    for step in range(1, 9):
        bags = [[list(rng.integers(0, N, rng.integers(0, 6))) for _ in range(B)] for _ in range(T)]
        idx, off, _ = _bags_to_arrays(bags)
        grad = rng.normal(0, 0.1, (B, T * d)).astype(F)
        out = o.forward(idx, off, B)
        ref = []
        for t in range(T):
            flat = torch.tensor([r for bag in bags[t] for r in bag], dtype=torch.long)
            offs = torch.tensor(np.cumsum([0] + [len(bag) for bag in bags[t]])[:-1], dtype=torch.long)
            w = W[t].clone().requires_grad_(True)
            pooled = torch.nn.functional.embedding_bag(flat, w, offs, mode="sum")
            ref.append(pooled.detach())
            (pooled * torch.tensor(grad[:, t * d:(t + 1) * d])).sum().backward()
            gw = w.grad
            touched = torch.zeros(N, dtype=torch.bool)
            touched[flat] = True
            if opt == orc.SGD:
                W[t] = W[t] - lr * gw
            else:
                G[t] = G[t] + touched * gw.pow(2).mean(1)
                W[t] = W[t] - touched[:, None] * lr * gw / (G[t].sqrt() + eps)[:, None]
        assert np.allclose(out, torch.cat(ref, 1).numpy(), rtol=1e-5, atol=1e-6)
        o.backward(grad, lr, step)
        for t in range(T):
            got = np.stack([o.fetch_value(t, r) for r in range(N)])
            assert np.allclose(got, W[t].numpy(), rtol=2e-5, atol=2e-6)


# ---------------------------- literal single-array emulator (P6, P7) -----
@pytest.mark.parametrize("bits,ways,policy,opt,frac", [
    (8, 2, "lru", "sgd", 0.25), (4, 4, "lfu", "sgd", 0.25), (8, 4, "lfu", "adagrad", 0.25),
    (4, 2, "lru", "adagrad", 0.25), (8, 1, "lru", "sgd", 0.1), (8, 1, "lfu", "sgd", 0.1),
    (8, 2, "lru", "sgd", 0.0), (4, 2, "lfu", "sgd", 0.0), (2, 4, "lfu", "sgd", 0.25), (2, 2, "lru", "adagrad", 0.0),
    (-8, 2, "lru", "sgd", 0.25), (-4, 4, "lfu", "sgd", 0.0),      # negative width: round to nearest while training
    (16, 2, "lru", "sgd", 0.25), (16, 4, "lfu", "adagrad", 0.0), (-16, 2, "lfu", "sgd", 0.25),   # FP16 table
])
def test_two_space_oracle_equals_single_array_emulation(bits, ways, policy, opt, frac):
    nearest = bits < 0
    bits = abs(bits)
    N, d, B, lr, seed = 24, 8, 6, 0.05, 21
    pol = orc.LRU if policy == "lru" else orc.LFU
    op = orc.SGD if opt == "sgd" else orc.ROWWISE_ADAGRAD
    o = orc.Oracle([N], d, bits, frac, ways, pol, optimizer=op, seed=seed)
    e = emu.Emulator(N, d, bits, o.sets(0), ways, policy, optimizer=opt, seed=seed, rounding="nearest" if nearest else "stochastic")
    if nearest:
        o.set_rounding(orc.RTN)
    rng = np.random.default_rng(bits * 7 + ways)
    for r in range(N):
        assert np.array_equal(o.fetch_value(0, r), e.T[r])
    for step in range(1, 8):
        hot = rng.integers(0, N)
        bags = [[int(x) for x in np.where(rng.random(4) < 0.4, hot, rng.integers(0, N, 4))][:rng.integers(0, 5)]
                for _ in range(B)]
        if step == 3:
            bags[0] = [int(hot)] * 40          # a row hot enough to need two tree levels
        idx, off, _ = _bags_to_arrays([bags])
        grad = rng.normal(0, 0.05, (B, d)).astype(F)
        assert np.array_equal(o.forward(idx, off, B), e.forward(bags))
        o.backward(grad, lr, step)
        e.backward(bags, grad, lr, step)
        for r in range(N):
            assert np.array_equal(o.fetch_value(0, r), e.T[r]), (step, r)
        if o.sets(0) > 0:
            tags, _, ts = o.cache(0)
            assert np.array_equal(tags, e.I_C.reshape(-1))
            if policy == "lru":
                assert np.array_equal(ts, e.ts.reshape(-1))
        if policy == "lfu":
            assert [o.cnt(0, r) for r in range(N)] == list(e.cnt)
        if opt == "adagrad":
            assert np.array_equal(np.array([o.adagrad(0, r) for r in range(N)], F), e.G)


# --------------------------------------------- memory accounting (P8) ----
def test_memory_compression_factors_of_the_appendix():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "compression_factor_table.txt")) if not l.startswith("#")]
    N, D = 3_200_000, 128
    checked = 0
    for bits, ratio, factor in rows:
        bits, ratio, factor = int(bits), float(ratio), float(factor)
        o = orc.Oracle([N], D, bits, ratio, 32, orc.LFU)
        m = o.memory_bytes().astype(np.float64)
        got = (m[0] + m[1] + m[2] + m[3]) / m[5]
        o.close()
        checked += 1
        assert abs(got - factor) < 6e-6, (bits, ratio, got, factor)
    assert checked == 10


def test_table1_sizes_fixture():
    sizes = [int(x) for l in open(os.path.join(GOLDEN, "kaggle_table_sizes.txt")) if not l.startswith("#") for x in l.split()]
    assert len(sizes) == 26 and sum(1 for s in sizes if s > 1000) == 15
    assert round(sum(sizes) * 128 / 1e9, 1) == 4.3


# --------------------------------------------------- invariants (P9, P10) -
@pytest.mark.parametrize("policy", [orc.LRU, orc.LFU])
def test_invariants_on_a_skewed_stream(policy):
    from paper_2010_11305_b200 import workloads as wl
    cfg = wl.scaled(wl.config(1), steps=6)
    cfg.policy = policy
    st = wl.Stream(cfg, "cpu")
    o = orc.Oracle(cfg.num_rows, cfg.dim, cfg.bits, cfg.cache_fraction, cfg.ways, policy, seed=cfg.seed)
    n_sets = o.sets(0)
    salt = orc.salt(cfg.seed, 0)
    total = 0
    snapshot = {r: o.row(0, r) for r in range(0, cfg.num_rows[0], 37)}
    touched_or_evicted = set()
    for step in range(1, 7):
        idx, off, grad = (x.numpy() for x in st.batch(step))
        tags_before, _, _ = o.cache(0)
        out1 = o.forward(idx, off, cfg.batch)
        o.backward(grad, cfg.lr, step)
        total += idx.size
        tags, rows, ts = o.cache(0)
        res = tags[tags >= 0]
        assert len(set(res)) == len(res)                                   # a row is cached at most once
        for slot, r in enumerate(tags):
            if r >= 0:
                assert orc.set_index(int(r), salt, n_sets) == slot // cfg.ways   # and only in set h(row)
        assert np.all(ts <= step)
        urows, mult, _ = o.last_unique(0)
        assert mult.sum() == idx.size
        touched_or_evicted |= set(int(r) for r in urows) | (set(tags_before[tags_before >= 0]) - set(res))
        s = o.stats(0)
        assert s[0] == total and s[7] == step and s[4] - s[5] == len(res)  # admissions - evictions = residents
        assert s[2] == s[3] + s[4] + s[6] or cfg.cache_fraction == 0        # unique = hits + admissions + bypasses
        if policy == orc.LFU:
            assert sum(o.cnt(0, int(r)) for r in o.touched(0)) == total
        # the next forward sees exactly what this step committed
        out2 = o.forward(idx, off, cfg.batch)
        want = np.zeros_like(out2)
        pos = 0
        for b in range(cfg.batch):
            for p in range(off[b], off[b + 1]):
                want[b] = (want[b] + o.fetch_value(0, int(idx[p]))).astype(F)
        assert np.array_equal(out2, want)
        assert not np.array_equal(out1, out2)
    for r, (codes, s_, b_) in snapshot.items():
        if r not in touched_or_evicted:
            c2, s2, b2 = o.row(0, r)
            assert np.array_equal(codes, c2) and s_ == s2 and b_ == b2     # untouched rows are bit-unchanged


def test_hit_rates_behave_like_the_paper_says():
    from paper_2010_11305_b200 import workloads as wl
    base = wl.Config("t", [20000], 4, 8, 0.05, 32, orc.LFU, 0, 0.01, 512, ("fixed", 4), [1.05], 40, seed=9)

    def hit_rate(ways, policy, zipf, frac=0.05, steps=40):
        cfg = wl.Config(**{**base.__dict__, "ways": ways, "policy": policy, "zipf": [zipf], "cache_fraction": frac})
        st = wl.Stream(cfg, "cpu")
        o = orc.Oracle(cfg.num_rows, cfg.dim, 8, frac, ways, policy, seed=cfg.seed)
        lookups = hits = 0
        for step in range(1, steps + 1):
            idx, off, grad = (x.numpy() for x in st.batch(step))
            o.forward(idx, off, cfg.batch)
            o.backward(grad, 0.01, step)
            if step == steps // 2:
                lookups, hits = o.stats(0)[0], o.stats(0)[1]
        s = o.stats(0)
        return float(s[1] - hits) / float(s[0] - lookups)

    uni = hit_rate(32, orc.LRU, None)
    assert abs(uni - 0.05) < 0.02                       # uniform stream: hit rate ~ cached fraction
    k = np.arange(1, 20001, dtype=np.float64) ** -1.05
    ideal = k[:992].sum() / k.sum()                     # mass of the 31*32 hottest rows
    lfu32 = hit_rate(32, orc.LFU, 1.05)
    lfu1 = hit_rate(1, orc.LFU, 1.05)
    lru1 = hit_rate(1, orc.LRU, 1.05)
    assert lfu32 <= ideal + 0.02
    assert lfu32 > 0.8 * ideal
    assert lfu32 >= lfu1 >= lru1 - 0.01                 # ordering of the paper's hit-rate table
    assert hit_rate(32, orc.LFU, 1.05, frac=0.2) > lfu32  # larger cache, higher hit rate


def test_nearest_rounding_in_training_loses_small_updates_and_stochastic_does_not():
    """Section 3 "Rounding" and the no-cache accuracy table: with round-to-nearest an update smaller than half a
    quantization step is lost every time, with stochastic rounding it survives on average."""
    d, N = 8, 4
    res = {}
    for mode in (orc.RTN, orc.SR):
        o = orc.Oracle([N], d, 8, 0.0, 8, orc.LRU, seed=2)
        o.set_rounding(mode)
        x0 = o.fetch_value(0, 1).astype(np.float64)
        step_size = float(o.row(0, 1)[1])
        # each update moves the interior columns by a fifth of a quantization step; the columns holding the row's
        # minimum and maximum stay put, so scale and bias do not follow the update
        x0f = x0.astype(F)
        inner = np.ones(d, bool)
        inner[[int(np.argmin(x0f)), int(np.argmax(x0f))]] = False
        g = np.zeros((1, d), F)
        g[0, inner] = 0.2 * step_size
        idx, off, B = _bags_to_arrays([[[1]]])
        for step in range(1, 101):
            o.forward(idx, off, B)
            o.backward(g, 1.0, step)
        res[mode] = ((x0 - o.fetch_value(0, 1).astype(np.float64)) / step_size)[inner]
    assert np.all(np.abs(res[orc.RTN]) < 1.0)             # nothing accumulated: 100 updates of 0.2 steps all rounded away
    assert np.all(res[orc.SR] > 8.0)                      # expectation 20 quantization steps (until a column reaches the minimum)


# --------------------------------------------------------- FP16 table ----
def test_half_conversions_against_numpy_and_bracketing():
    rng = np.random.default_rng(3)
    xs = np.concatenate([rng.normal(0, 1, 4000), rng.normal(0, 1e-4, 2000), rng.normal(0, 3e-7, 2000), rng.uniform(-65504, 65504, 1000),
                         [0.0, -0.0, 65504.0, -65504.0, 2.0 ** -24, 2.0 ** -25, 3 * 2.0 ** -25, 1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11,
                          6.1e-5, 5.96e-8, 2.98e-8]]).astype(F)
    for x in xs:
        rn, rd, ru = (orc.float_to_half(x, m) for m in (0, 1, 2))
        assert rn == int(np.float16(x).view(np.uint16)), x                     # numpy rounds to nearest even
        lo, hi = orc.half_to_float(rd), orc.half_to_float(ru)
        assert lo <= x <= hi
        assert orc.half_to_float(rd) == np.array(rd, np.uint16).view(np.float16).astype(F)
        if lo != hi:                                                            # neighbours: one unit in the last place apart
            assert np.nextafter(np.array(rd, np.uint16).view(np.float16), np.float16(np.inf)).view(np.uint16) == ru or (lo == 0 and hi == 0)
        else:
            assert F(np.float16(x)) == x


def test_half_stochastic_rounding_is_unbiased():
    x = np.array([0.1, -0.3337, 1.0 + 2.0 ** -12, 3.3e-6, 100.123, 0.5], F)
    K = 60000
    acc = np.zeros(len(x))
    for step in range(K):
        h = orc.to_half_row(x, orc.SR, orc.rowkey(1, orc.DOMAIN_SR, 0, 5, step))
        acc += h.view(np.float16).astype(np.float64)
    ulp = np.array([float(np.spacing(np.float16(v))) for v in x])
    assert np.all(np.abs(acc / K - x) <= 4.5 * (np.abs(ulp) / 2) / np.sqrt(K) + 1e-12)
    assert orc.to_half_row(x, orc.RTN)[5] == int(np.float16(0.5).view(np.uint16))       # representable values never move
    assert np.all(orc.to_half_row(np.array([0.5, -2.0, 0.0], F), orc.SR, 77) == np.array([0.5, -2.0, 0.0], np.float16).view(np.uint16))


def test_fp16_table_halves_the_memory():
    # Section 4.3: the compression factor of a non-cached FP16 table is 0.5
    o = orc.Oracle([1000], 128, 16, 0.0, 32, orc.LFU)
    m = o.memory_bytes().astype(np.float64)
    assert (m[0] + m[1] + m[2] + m[3]) / m[5] == 0.5


@pytest.mark.parametrize("policy", [orc.LRU, orc.LFU])
def test_lowest_resident_priority_of_a_full_set_never_falls(policy):
    """Algorithm 2 replaces the resident with the lowest priority value by a row whose value is strictly larger, and
    counts / time stamps only grow: once a set is full, the minimum over its residents is non-decreasing from step to step.
    (The CUDA path records that minimum per set and uses it to bypass hopeless candidates early.)"""
    from paper_2010_11305_b200 import workloads as wl
    cfg = wl.Config(name="floor", num_rows=[800, 120], dim=8, bits=8, cache_fraction=0.1, ways=4, policy=policy, optimizer=wl.SGD,
                    lr=0.05, batch=40, bag=("poisson", 3.0), zipf=[1.1, 0.9], steps=40, seed=9)
    st = wl.Stream(cfg, "cpu")
    o = orc.Oracle(cfg.num_rows, cfg.dim, cfg.bits, cfg.cache_fraction, cfg.ways, policy, seed=cfg.seed)
    prev = [None] * cfg.num_tables
    grew = 0
    for step in range(1, cfg.steps + 1):
        idx, off, grad = st.batch(step)
        o.forward(idx.numpy(), off.numpy(), cfg.batch)
        o.backward(grad.numpy(), cfg.lr, step)
        for t in range(cfg.num_tables):
            tags, _, ts = o.cache(t)
            tags = tags.reshape(-1, cfg.ways)
            if policy == orc.LFU:
                pv = np.array([[o.cnt(t, int(r)) if r >= 0 else -1 for r in row] for row in tags], np.int64)
            else:
                pv = np.where(tags >= 0, ts.reshape(-1, cfg.ways).astype(np.int64), -1)
            low = np.where((tags >= 0).all(1), pv.min(1), -1)          # -1: the set still has an empty way
            if prev[t] is not None:
                full_before = prev[t] >= 0
                assert (low[full_before] >= prev[t][full_before]).all(), (step, t)
                grew += int((low[full_before] > prev[t][full_before]).sum())
            prev[t] = low
    o.close()
    assert grew > 0                                                     # and it did move
