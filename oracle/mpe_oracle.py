"""ctypes view of the CPU oracle (oracle/mpe_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests, by the smoke check and by the
CPU-baseline leg of the benchmark.  Nothing on the product path may use it.
Arrays cross the boundary as numpy arrays; this file holds no arithmetic of
the method.
"""
import ctypes as C

import numpy as np

from . import build as _build

LRU, LFU = 0, 1
SGD, ROWWISE_ADAGRAD = 0, 1
RTN, SR = 0, 1
DOMAIN_INIT, DOMAIN_SR, DOMAIN_FLUSH = 1, 2, 3

_lib = C.CDLL(_build.build())

_u8p = np.ctypeslib.ndpointer(np.uint8, flags="C_CONTIGUOUS")
_i32p = np.ctypeslib.ndpointer(np.int32, flags="C_CONTIGUOUS")
_u32p = np.ctypeslib.ndpointer(np.uint32, flags="C_CONTIGUOUS")
_i64p = np.ctypeslib.ndpointer(np.int64, flags="C_CONTIGUOUS")
_u64p = np.ctypeslib.ndpointer(np.uint64, flags="C_CONTIGUOUS")
_f32p = np.ctypeslib.ndpointer(np.float32, flags="C_CONTIGUOUS")


def _sig(name, restype, *argtypes):
    f = getattr(_lib, name)
    f.restype = restype
    f.argtypes = list(argtypes)
    return f


_mix32 = _sig("orc_mix32", C.c_uint32, C.c_uint32)
_rowkey = _sig("orc_rowkey", C.c_uint32, C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint64)
_draw = _sig("orc_draw", C.c_uint32, C.c_uint32, C.c_uint32)
_uniform = _sig("orc_uniform", C.c_float, C.c_uint32, C.c_uint32)
_salt = _sig("orc_salt", C.c_uint32, C.c_uint64, C.c_uint32)
_set_index = _sig("orc_set_index", C.c_int32, C.c_uint32, C.c_uint32, C.c_int32)
_num_sets = _sig("orc_num_sets", C.c_int32, C.c_int64, C.c_double, C.c_int32)
_quantize = _sig("orc_quantize", None, _f32p, C.c_int32, C.c_int32, C.c_int32, C.c_uint32, _u8p,
                 C.POINTER(C.c_float), C.POINTER(C.c_float))
_dequantize = _sig("orc_dequantize", None, _u8p, C.c_int32, C.c_float, C.c_float, _f32p)
_pack = _sig("orc_pack", None, _u8p, C.c_int32, C.c_int32, _u8p)
_unpack = _sig("orc_unpack", None, _u8p, C.c_int32, C.c_int32, _u8p)
_h2f = _sig("orc_half_to_float", C.c_float, C.c_uint16)
_f2h = _sig("orc_float_to_half", C.c_uint16, C.c_float, C.c_int32)
_to_half_row = _sig("orc_to_half_row", None, _f32p, C.c_int32, C.c_int32, C.c_uint32, np.ctypeslib.ndpointer(np.uint16, flags="C_CONTIGUOUS"))
_init_row = _sig("orc_init_row", None, C.c_uint64, C.c_uint32, C.c_uint32, C.c_int32, C.c_float, C.c_float, _f32p)
_tree_sum = _sig("orc_tree_sum", None, C.POINTER(C.c_void_p), C.c_int64, C.c_int32, _f32p)

_create = _sig("orc_create", C.c_void_p, _i64p, C.c_int32, C.c_int32, C.c_int32, C.c_double, C.c_int32,
               C.c_int32, C.c_int32, C.c_float, C.c_float, C.c_float, C.c_uint64)
_destroy = _sig("orc_destroy", None, C.c_void_p)
_set_mask = _sig("orc_set_table_mask", None, C.c_void_p, C.c_void_p)
_set_rounding = _sig("orc_set_rounding", None, C.c_void_p, C.c_int32)
_forward = _sig("orc_forward", C.c_int, C.c_void_p, _i32p, _i32p, C.c_int32, C.c_int64, _f32p)
_backward = _sig("orc_backward", C.c_int, C.c_void_p, _f32p, C.c_float, C.c_int64)
_flush = _sig("orc_flush", C.c_int, C.c_void_p)
_dropped = _sig("orc_dropped", C.c_int64, C.c_void_p)
_sets = _sig("orc_sets", C.c_int32, C.c_void_p, C.c_int32)
_get_row = _sig("orc_get_row", None, C.c_void_p, C.c_int32, C.c_int64, _u8p, C.POINTER(C.c_float), C.POINTER(C.c_float))
_get_cache = _sig("orc_get_cache", None, C.c_void_p, C.c_int32, _i32p, _f32p, _u32p)
_get_cnt = _sig("orc_get_cnt", C.c_uint32, C.c_void_p, C.c_int32, C.c_int64)
_get_adagrad = _sig("orc_get_adagrad", C.c_float, C.c_void_p, C.c_int32, C.c_int64)
_touched = _sig("orc_touched", C.c_int64, C.c_void_p, C.c_int32, _i64p, C.c_int64)
_stats = _sig("orc_stats", None, C.c_void_p, C.c_int32, _u64p)
_memory = _sig("orc_memory_bytes", None, C.c_void_p, _u64p)
_last_unique = _sig("orc_last_unique", C.c_int64, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64)


def mix32(x):
    return int(_mix32(x & 0xFFFFFFFF))


def rowkey(seed, domain, table, row, step):
    return int(_rowkey(seed, domain, table, row, step))


def draw(key, column):
    return int(_draw(key, column))


def uniform(key, column):
    return float(_uniform(key, column))


def salt(seed, table):
    return int(_salt(seed, table))


def set_index(row, salt_, n_sets):
    return int(_set_index(row, salt_, n_sets))


def num_sets(num_rows, cache_fraction, ways):
    return int(_num_sets(num_rows, cache_fraction, ways))


def quantize(x, bits, mode=RTN, key=0):
    """Row-wise min-max quantization of one row -> (codes[d] uint8, scale, bias)."""
    x = np.ascontiguousarray(x, np.float32)
    q = np.zeros(x.shape[0], np.uint8)
    s, b = C.c_float(), C.c_float()
    _quantize(x, x.shape[0], bits, mode, key, q, C.byref(s), C.byref(b))
    return q, np.float32(s.value), np.float32(b.value)


def dequantize(q, scale, bias):
    q = np.ascontiguousarray(q, np.uint8)
    x = np.zeros(q.shape[0], np.float32)
    _dequantize(q, q.shape[0], float(scale), float(bias), x)
    return x


def pack(q, bits):
    q = np.ascontiguousarray(q, np.uint8)
    out = np.zeros(q.shape[0] * bits // 8, np.uint8)
    _pack(q, q.shape[0], bits, out)
    return out


def unpack(packed, d, bits):
    packed = np.ascontiguousarray(packed, np.uint8)
    out = np.zeros(d, np.uint8)
    _unpack(packed, d, bits, out)
    return out


def half_to_float(h):
    return np.float32(_h2f(int(h)))


def float_to_half(f, direction=0):
    """FP16 bits of f; direction 0 nearest-even, 1 toward -inf, 2 toward +inf."""
    return int(_f2h(float(np.float32(f)), direction))


def to_half_row(x, mode=RTN, key=0):
    x = np.ascontiguousarray(x, np.float32)
    out = np.zeros(x.shape[0], np.uint16)
    _to_half_row(x, x.shape[0], mode, key, out)
    return out


def init_row(seed, table, row, d, lo, hi):
    x = np.zeros(d, np.float32)
    _init_row(seed, table, row, d, lo, hi, x)
    return x


def tree_sum(terms):
    """Radix-32 summation tree over the rows of terms[m, d]."""
    terms = np.ascontiguousarray(terms, np.float32)
    m, d = terms.shape
    ptrs = (C.c_void_p * m)(*[terms.ctypes.data + i * d * 4 for i in range(m)])
    out = np.zeros(d, np.float32)
    _tree_sum(ptrs, m, d, out)
    return out


class OracleError(RuntimeError):
    """A call the oracle refused; `code` is its ORC_ERR_* value."""

    def __init__(self, what, code):
        super().__init__(f"{what} failed: {code}")
        self.code = code


ERR_ARG, ERR_OFFSETS, ERR_SEQUENCE = -1, -2, -3


class Oracle:
    """One embedding collection: T tables sharing dim, precision, cache shape and policy."""

    def __init__(self, num_rows, dim, bits, cache_fraction, ways, policy, optimizer=SGD, eps=1e-8,
                 init_lo=-0.05, init_hi=0.05, seed=0):
        self.num_rows = np.ascontiguousarray(num_rows, np.int64)
        self.T, self.d, self.bits = len(self.num_rows), dim, bits
        self.ways = 32 if ways == 0 else ways
        self.policy, self.optimizer = policy, optimizer
        self._h = _create(self.num_rows, self.T, dim, bits, cache_fraction, ways, policy, optimizer, eps,
                          init_lo, init_hi, seed)
        if not self._h:
            raise ValueError("orc_create rejected the arguments")
        self.batch = 0

    def close(self):
        if self._h:
            _destroy(self._h)
            self._h = None

    def __del__(self):
        if _destroy is not None:        # at interpreter exit the module's names may be gone already
            self.close()

    def set_rounding(self, mode):
        _set_rounding(self._h, mode)

    def set_table_mask(self, mask):
        if mask is None:
            _set_mask(self._h, None)
        else:
            m = np.ascontiguousarray(mask, np.uint8)
            _set_mask(self._h, m.ctypes.data)

    def forward(self, indices, offsets, batch):
        indices = np.ascontiguousarray(indices, np.int32)
        offsets = np.ascontiguousarray(offsets, np.int32)
        out = np.zeros((batch, self.T * self.d), np.float32)
        rc = _forward(self._h, indices if indices.size else np.zeros(1, np.int32), offsets, batch, indices.size, out)
        if rc != 0:
            raise OracleError("orc_forward", rc)
        self.batch = batch
        return out

    def backward(self, grad_out, lr, step):
        g = np.ascontiguousarray(grad_out, np.float32)
        rc = _backward(self._h, g, lr, step)
        if rc != 0:
            raise OracleError("orc_backward", rc)

    def flush(self):
        _flush(self._h)

    def dropped(self):
        return int(_dropped(self._h))

    def sets(self, t):
        return int(_sets(self._h, t))

    def row(self, t, row):
        codes = np.zeros(self.d * self.bits // 8, np.uint8)
        s, b = C.c_float(), C.c_float()
        _get_row(self._h, t, row, codes, C.byref(s), C.byref(b))
        return codes, np.float32(s.value), np.float32(b.value)

    def rows(self, t, rows):
        n = len(rows)
        codes = np.zeros((n, self.d * self.bits // 8), np.uint8)
        scale = np.zeros(n, np.float32)
        bias = np.zeros(n, np.float32)
        for i, r in enumerate(rows):
            codes[i], scale[i], bias[i] = self.row(t, int(r))
        return codes, scale, bias

    def cache(self, t):
        slots = max(self.sets(t) * self.ways, 0)
        tags = np.zeros(max(slots, 1), np.int32)
        rows = np.zeros((max(slots, 1), self.d), np.float32)
        ts = np.zeros(max(slots, 1), np.uint32)
        _get_cache(self._h, t, tags, rows, ts)
        return tags[:slots], rows[:slots], ts[:slots]

    def cnt(self, t, row):
        return int(_get_cnt(self._h, t, row))

    def adagrad(self, t, row):
        return np.float32(_get_adagrad(self._h, t, row))

    def touched(self, t):
        n = int(_touched(self._h, t, np.zeros(1, np.int64), 0))
        rows = np.zeros(max(n, 1), np.int64)
        _touched(self._h, t, rows, n)
        return rows[:n]

    def stats(self, t):
        out = np.zeros(8, np.uint64)
        _stats(self._h, t, out)
        return out

    def memory_bytes(self):
        out = np.zeros(6, np.uint64)
        _memory(self._h, out)
        return out

    def last_unique(self, t):
        n = int(_last_unique(self._h, t, None, None, None, 0))
        rows = np.zeros(max(n, 1), np.int64)
        mult = np.zeros(max(n, 1), np.int32)
        grads = np.zeros((max(n, 1), self.d), np.float32)
        _last_unique(self._h, t, rows.ctypes.data, mult.ctypes.data, grads.ctypes.data, n)
        return rows[:n], mult[:n], grads[:n]

    def fetch_value(self, t, row):
        """FP32 value fetch(T, C, i) would return now (cache row if resident, else dequantized)."""
        tags, rows, _ = self.cache(t)
        hit = np.nonzero(tags == row)[0]
        if hit.size:
            return rows[hit[0]].copy()
        codes, s, b = self.row(t, row)
        if self.bits == 16:
            return codes.view(np.float16).astype(np.float32)
        return dequantize(unpack(codes, self.d, self.bits), s, b)
