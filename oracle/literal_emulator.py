"""Single-array emulation of the method, after the paper's own CPU experiments.

TEST INFRASTRUCTURE ONLY.  Section 4 of the paper emulates the low-precision
table and its cache with ONE FP32 array per table: rows that are cache
resident keep full precision, every other row is fake-quantized (quantize then
dequantize, Algorithm 1) whenever the method would have stored it in low
precision, and Algorithm 2 decides which is which.  This file restates that
emulation in slow scalar Python so that the two-space C oracle (real codes +
separate FP32 cache) can be compared with it bit for bit on fetched values,
tags and priority values.  It is written independently of the C file: own
hash, own quantizer, own fused multiply-add (exact rational arithmetic).

The conventions the paper leaves open (hash constants, order of I_U, LFU
increment, timestamp unit, summation tree) are the same as in the C oracle;
they are what "parity unpinned" refers to there.
"""
from fractions import Fraction

import numpy as np

F = np.float32
M32 = 0xFFFFFFFF


def mix32(x):
    x &= M32
    x ^= x >> 16
    x = (x * 0x7FEB352D) & M32
    x ^= x >> 15
    x = (x * 0x846CA68B) & M32
    x ^= x >> 16
    return x


def _absorb(h, w):
    return mix32(((h ^ w) + 0x9E3779B9) & M32)


def rowkey(seed, domain, table, row, step):
    h = 0x243F6A88
    for w in (seed & M32, seed >> 32, domain, table, row, step & M32, step >> 32):
        h = _absorb(h, w & M32)
    return h


def uniform(key, column):
    bits = mix32(key ^ ((column * 0x9E3779B9 + 0x7F4A7C15) & M32))
    return F(bits >> 8) * F(2.0 ** -24)


def set_hash(row, table, seed, n_sets):
    salt = 0x13198A2E
    for w in (seed & M32, seed >> 32, table):
        salt = _absorb(salt, w)
    return (mix32(row ^ salt) * n_sets) >> 32


def fma32(a, b, c):
    """Correctly rounded a*b+c in binary32 via exact rationals."""
    exact = Fraction(float(a)) * Fraction(float(b)) + Fraction(float(c))
    guess = F(float(exact))
    best = None
    for cand in (np.nextafter(guess, F(-np.inf)), guess, np.nextafter(guess, F(np.inf))):
        if not np.isfinite(cand):
            continue
        err = abs(Fraction(float(cand)) - exact)
        even = (int(np.array(cand, F).view(np.uint32)) & 1) == 0
        if best is None or err < best[0] or (err == best[0] and even and not best[2]):
            best = (err, cand, even)
    r = best[1]
    if r == 0 and exact == 0:  # sign of an exact zero sum follows IEEE: +0 unless both addends are -0
        prod_neg = (np.signbit(a) != np.signbit(b))
        return F(-0.0) if (prod_neg and np.signbit(c)) else F(0.0)
    return F(r)


def fake_half(r, mode, key):
    """FP16_to_FP32(FP32_to_FP16(x)) per element (Section 4.1), nearest or stochastic between the two FP16 neighbours."""
    out = np.zeros(len(r), F)
    for i, x in enumerate(r):
        v = F(min(max(F(x), F(-65504.0)), F(65504.0)))
        h = np.float16(v)                              # numpy converts with round-to-nearest-even
        if mode == "nearest" or F(h) == v:
            out[i] = F(h)
            continue
        if F(h) > v:
            lo, hi = np.nextafter(h, np.float16(-np.inf)), h
        else:
            lo, hi = h, np.nextafter(h, np.float16(np.inf))
        p = F(F(v - F(lo)) / F(F(hi) - F(lo)))
        out[i] = F(hi) if uniform(key, i) < p else F(lo)
    return out, None, None, None


def fake_quantize(r, bits, mode, key):
    """Algorithm 1: r <- q*s + b with q = round_to_int((r-b)/s), in place semantics (returns a new row)."""
    if bits == 16:
        return fake_half(r, mode, key)
    d = len(r)
    b = F(min(r)) + F(0.0)
    mx = F(max(r))
    qmax = F(2 ** bits - 1)
    s = F((mx - b) / qmax)
    tiny = F(np.finfo(np.float32).tiny)
    inv = F(1.0) / s if s >= tiny else F(0.0)
    if inv == 0:
        s = F(0.0)
    out = np.zeros(d, F)
    codes = np.zeros(d, np.int64)
    for i in range(d):
        y = F((F(r[i]) - b) * inv)
        y = min(max(y, F(0.0)), qmax)
        if mode == "nearest":
            q = int(np.rint(y))
        else:
            f = np.floor(y)
            p = F(y - f)
            q = int(f) + (1 if uniform(key, i) < p else 0)
        codes[i] = q
        out[i] = fma32(F(q), s, b)
    return out, codes, s, b


def tree_sum(terms):
    """Radix-32 tree: up to 32 terms are added left to right; longer lists are cut
    into consecutive chunks of 32 whose sums are reduced by the same rule."""
    if len(terms) <= 32:
        acc = terms[0].copy()
        for t in terms[1:]:
            acc = (acc + t).astype(F)
        return acc
    return tree_sum([tree_sum(terms[i:i + 32]) for i in range(0, len(terms), 32)])


class Emulator:
    """One table, one FP32 array, Algorithm 2 on top."""

    def __init__(self, N, d, bits, n_sets, ways, policy, optimizer="sgd", eps=1e-8, lo=-0.05, hi=0.05, seed=0,
                 table=0, rounding="stochastic"):
        self.rounding = rounding
        self.N, self.d, self.bits, self.n, self.alpha = N, d, bits, n_sets, ways
        self.policy, self.optimizer, self.eps, self.seed, self.table = policy, optimizer, F(eps), seed, table
        self.T = np.zeros((N, d), F)
        for i in range(N):
            k = rowkey(seed, 1, table, i, 0)
            x = np.array([fma32(uniform(k, c), F(hi) - F(lo), F(lo)) for c in range(d)], F)
            self.T[i] = fake_quantize(x, bits, "nearest", 0)[0]
        self.I_C = -np.ones((max(n_sets, 1), ways), np.int64)      # tags
        self.ts = np.zeros((max(n_sets, 1), ways), np.int64)       # LRU: PV of cached rows
        self.cnt = np.zeros(N, np.int64)                           # LFU: PV of every row
        self.G = np.zeros(N, F)

    def h(self, i):
        return set_hash(i, self.table, self.seed, self.n)

    def forward(self, bags):
        """bags: list of lists of row ids -> pooled sums, each starting from +0 and adding in order."""
        out = np.zeros((len(bags), self.d), F)
        for b, bag in enumerate(bags):
            for i in bag:
                if 0 <= i < self.N:
                    out[b] = (out[b] + self.T[i]).astype(F)
        return out

    def _pv_resident(self, s, w):
        j = self.I_C[s, w]
        if j < 0:
            return -1
        return int(self.cnt[j]) if self.policy == "lfu" else int(self.ts[s, w])

    def backward(self, bags, grad_out, lr, step):
        """One update of the cached table (Section 3 "update", Section 3 "Cache Replacement Policy", Section 5.1),
        in four passes over the distinct rows of the batch: merge, priorities, full-precision update, placement."""
        lr = F(lr)
        # merge: one gradient per distinct row, duplicates summed (Section 5.1)
        where = {}
        for b, bag in enumerate(bags):
            for i in bag:
                if 0 <= i < self.N:
                    where.setdefault(i, []).append(b)
        rows = sorted(where)
        merged = {i: tree_sum([np.asarray(grad_out[b], F) for b in where[i]]) for i in rows}
        cached = {i: (self.n > 0 and i in self.I_C[self.h(i)]) for i in rows}
        # priorities: popularity counts every access, recency stamps the cached rows that were used
        for i in rows:
            if self.policy == "lfu":
                self.cnt[i] = min(self.cnt[i] + len(where[i]), M32)
            elif cached[i]:
                s = self.h(i)
                self.ts[s, list(self.I_C[s]).index(i)] = step
        # update: every touched row moves in full precision, wherever it lives
        for i in rows:
            self.T[i] = self._optimizer(i, merged[i], lr)
        # placement: rows that were cached stay as they are; the others, in ascending row id, either take the place of
        # their set's lowest-priority resident (which then drops to low precision) or drop to low precision themselves
        for i in rows:
            if cached[i]:
                continue
            if self.n == 0 or not self._admit(i, step):
                self.T[i] = self._lower(i, step)

    def _optimizer(self, i, g, lr):
        if self.optimizer == "sgd":
            mult = lr
        else:
            sq = []
            for l in range(self.d // 4):
                a = F(g[4 * l] * g[4 * l])
                for e in (1, 2, 3):
                    a = fma32(g[4 * l + e], g[4 * l + e], a)
                sq.append(a)
            stride = len(sq) // 2
            while stride >= 1:
                for l in range(stride):
                    sq[l] = F(sq[l] + sq[l + stride])
                stride //= 2
            self.G[i] = F(self.G[i] + F(sq[0] * (F(1.0) / F(self.d))))
            mult = F(lr / F(np.sqrt(self.G[i]) + self.eps))
        return np.array([fma32(-mult, g[c], self.T[i, c]) for c in range(self.d)], F)

    def _lower(self, i, step):
        """The row as the low-precision table would hold it after this step (Algorithm 1 with this step's random bits)."""
        return fake_quantize(self.T[i], self.bits, self.rounding, rowkey(self.seed, 2, self.table, int(i), step))[0]

    def _admit(self, i, step):
        """Whether row i enters the cache; if so the displaced resident is lowered and i takes its way."""
        s = self.h(i)
        standing = [self._pv_resident(s, w) for w in range(self.alpha)]
        weakest = int(np.argmin(standing))           # first minimum: the lowest way wins a tie, an empty way beats all
        mine = int(self.cnt[i]) if self.policy == "lfu" else step
        direct_mapped_recency = self.alpha == 1 and self.policy == "lru"
        if mine <= standing[weakest] and not direct_mapped_recency:
            return False
        out = self.I_C[s, weakest]
        if out >= 0:
            self.T[out] = self._lower(out, step)
        self.I_C[s, weakest] = i
        if self.policy == "lru":
            self.ts[s, weakest] = step
        return True
