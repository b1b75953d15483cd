"""Thin ctypes binding of the C ABI in include/mpe.h.

Argument marshalling only: every function forwards to the entry point of the
same name in libmpe.so.  Device buffers are torch CUDA tensors (torch is used
for device memory and streams, nothing else); host buffers are numpy arrays or
pinned torch CPU tensors.  There is no CPU fallback: if the library is missing
or cannot be loaded, importing this module raises.
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmpe.so")

LRU, LFU = 0, 1
SGD, ROWWISE_ADAGRAD = 0, 1
ROUND_NEAREST, ROUND_STOCHASTIC = 0, 1
TABLE_DEVICE, TABLE_HOST = 0, 1
SELFTEST_LOOK_BACK_TIMEOUT, SELFTEST_RENEW_TAGS = 1, 2
OK, ERR_ARG, ERR_UNSUPPORTED, ERR_CUDA, ERR_SEQUENCE, ERR_INDEX, ERR_OFFSETS, ERR_NOMEM, ERR_TOO_LARGE, ERR_TIMEOUT = 0, -1, -2, -3, -4, -5, -6, -7, -8, -9
STATIC_MAX_INDICES, STATIC_MAX_BAGS, STATIC_MAX_TABLES = 32768, 32768, 64

EXPORTS = [
    "mpe_create", "mpe_create_placed", "mpe_reserve", "mpe_prepare", "mpe_forward", "mpe_forward_static", "mpe_backward", "mpe_set_rounding", "mpe_step_host", "mpe_step_host_submit", "mpe_step_host_wait", "mpe_flush", "mpe_destroy",
    "mpe_last_error", "mpe_stats", "mpe_memory_bytes", "mpe_workspace_bytes", "mpe_selftest", "mpe_cache_geometry", "mpe_step_info", "mpe_export_rows",
    "mpe_export_cache", "mpe_export_aux", "mpe_use_graphs", "mpe_kernel_launches", "mpe_profile", "mpe_profile_read",
    "mpe_forward_routed", "mpe_gather_grad", "mpe_peer_buffer_alloc", "mpe_peer_buffer_open", "mpe_peer_buffer_close", "mpe_peer_buffer_free",
    "mpe_error_string",
]


class TableSpec(C.Structure):
    _fields_ = [("num_rows", C.c_int64), ("dim", C.c_int32)]


def load_library(path: str = LIB_PATH) -> C.CDLL:
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with `python -m paper_2010_11305_b200.build` "
                          "(there is no CPU fallback for this library)")
    return C.CDLL(path)


_lib = load_library()
_vp, _i32, _i64, _u64, _f32, _f64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64, C.c_float, C.c_double
_lib.mpe_create.argtypes = [C.POINTER(_vp), C.POINTER(TableSpec), _i32, _i32, _f64, _i32, _i32, _i32, _f32, _f32, _f32, _u64, _i32]
_lib.mpe_create_placed.argtypes = [C.POINTER(_vp), C.POINTER(TableSpec), _i32, _i32, _f64, _i32, _i32, _i32, _f32, _f32, _f32, _u64, _i32, _i32]
_lib.mpe_reserve.argtypes = [_vp, _i32, _i64]
_lib.mpe_forward.argtypes = [_vp, _vp, _vp, _i32, _i64, _vp, _vp]
_lib.mpe_prepare.argtypes = [_vp, _vp, _vp, _i32, _i64, _vp]
_lib.mpe_forward_static.argtypes = [_vp, _vp, _vp, _i32, _i64, _vp, _vp]
_lib.mpe_backward.argtypes = [_vp, _vp, _f32, _i64]
_lib.mpe_step_host.argtypes = [_vp, _vp, _vp, _i32, _i64, _vp, _vp, _f32, _i64]
_lib.mpe_step_host_submit.argtypes = [_vp, _vp, _vp, _i32, _i64, _vp, _vp, _f32, _i64]
_lib.mpe_step_host_wait.argtypes = [_vp]
_lib.mpe_flush.argtypes = [_vp]
_lib.mpe_destroy.argtypes = [_vp]
_lib.mpe_last_error.argtypes = [_vp, C.POINTER(_i32), C.POINTER(_i64)]
_lib.mpe_stats.argtypes = [_vp, _i32, _vp]
_lib.mpe_memory_bytes.argtypes = [_vp, _vp]
_lib.mpe_workspace_bytes.argtypes = [_vp, _vp]
_lib.mpe_selftest.argtypes = [_vp, C.c_int32]
_lib.mpe_cache_geometry.argtypes = [_vp, _i32, C.POINTER(_i32), C.POINTER(_i32)]
_lib.mpe_step_info.argtypes = [_vp, _vp]
_lib.mpe_export_rows.argtypes = [_vp, _i32, _vp, _i64, _vp, _vp, _vp]
_lib.mpe_export_cache.argtypes = [_vp, _i32, _vp, _vp, _vp]
_lib.mpe_export_aux.argtypes = [_vp, _i32, _vp, _i64, _vp, _vp]
_lib.mpe_use_graphs.argtypes = [_vp, _i32]
_lib.mpe_set_rounding.argtypes = [_vp, _i32]
_lib.mpe_kernel_launches.argtypes = [_vp, C.POINTER(_u64)]
_lib.mpe_profile.argtypes = [_vp, _i32]
_lib.mpe_profile_read.argtypes = [_vp, _i32, _vp, _vp, _vp, C.POINTER(_i32)]
_lib.mpe_forward_routed.argtypes = [_vp, _vp, _vp, _i32, _i64, C.POINTER(_vp), _i32, _i32, _i32, _vp]
_lib.mpe_gather_grad.argtypes = [_vp, C.POINTER(_vp), _i32, _i32, _i32, _i32, _vp, _vp]
_lib.mpe_peer_buffer_alloc.argtypes = [_i32, _i64, C.POINTER(_vp), _vp]
_lib.mpe_peer_buffer_open.argtypes = [_i32, _vp, C.POINTER(_vp)]
_lib.mpe_peer_buffer_close.argtypes = [_i32, _vp]
_lib.mpe_peer_buffer_free.argtypes = [_i32, _vp]
_lib.mpe_error_string.argtypes = [C.c_int]
_lib.mpe_error_string.restype = C.c_char_p
for _n in EXPORTS[:-1]:
    getattr(_lib, _n).restype = C.c_int


class MpeError(RuntimeError):
    def __init__(self, code, where):
        super().__init__(f"{where}: {_lib.mpe_error_string(code).decode()} ({code})")
        self.code = code


def _check(code, where):
    if code != OK:
        raise MpeError(code, where)


def _ptr(x):
    """Address of a torch tensor / numpy array (None -> NULL)."""
    if x is None:
        return None
    if isinstance(x, np.ndarray):
        assert x.flags["C_CONTIGUOUS"]
        return x.ctypes.data
    assert x.is_contiguous()
    return x.data_ptr()


class Mpe:
    """Handle of one embedding collection on one GPU (see include/mpe.h for the semantics)."""

    def __init__(self, num_rows, dim, bits, cache_fraction, ways, policy, optimizer=SGD, eps=1e-8, init_lo=-0.05,
                 init_hi=0.05, seed=0, device=0, table_placement=TABLE_DEVICE):
        self.T, self.dim, self.bits = len(num_rows), dim, bits
        self.num_rows = [int(n) for n in num_rows]
        specs = (TableSpec * self.T)(*[TableSpec(int(n), dim) for n in num_rows])
        h = _vp()
        if table_placement == TABLE_DEVICE:
            _check(_lib.mpe_create(C.byref(h), specs, self.T, bits, cache_fraction, ways, policy, optimizer, eps, init_lo,
                                   init_hi, seed, device), "mpe_create")
        else:
            _check(_lib.mpe_create_placed(C.byref(h), specs, self.T, bits, cache_fraction, ways, policy, optimizer, eps,
                                          init_lo, init_hi, seed, device, table_placement), "mpe_create_placed")
        self._h = h
        self.device = device
        self.ways = self.cache_geometry(0)[1]

    def close(self):
        if getattr(self, "_h", None):
            _lib.mpe_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    # ---- the step -------------------------------------------------------------------------
    def reserve(self, max_batch, max_total_indices):
        _check(_lib.mpe_reserve(self._h, max_batch, max_total_indices), "mpe_reserve")

    def prepare(self, d_indices, d_offsets, batch, stream=None):
        """Sort and de-duplicate the next batch on `stream` while the current step runs; the forward of that batch takes it over."""
        _check(_lib.mpe_prepare(self._h, _ptr(d_indices), _ptr(d_offsets), batch, d_indices.numel(), stream), "mpe_prepare")

    def forward(self, d_indices, d_offsets, batch, d_out, stream=None):
        _check(_lib.mpe_forward(self._h, _ptr(d_indices), _ptr(d_offsets), batch, d_indices.numel(), _ptr(d_out),
                                stream), "mpe_forward")

    def forward_static(self, d_indices, d_offsets, batch, d_out, stream=None):
        """Evaluation forward for callers that must not allocate: its scratch is a fixed array inside the library."""
        _check(_lib.mpe_forward_static(self._h, _ptr(d_indices), _ptr(d_offsets), batch, d_indices.numel(), _ptr(d_out),
                                       stream), "mpe_forward_static")

    def forward_routed(self, d_indices, d_offsets, batch, out_ptrs, tables_global, table_base, stream=None):
        """Forward whose pooled vectors go straight to their owners' buffers; out_ptrs: one device address per rank."""
        arr = (_vp * len(out_ptrs))(*[int(p) for p in out_ptrs])
        _check(_lib.mpe_forward_routed(self._h, _ptr(d_indices), _ptr(d_offsets), batch, d_indices.numel(), arr, len(out_ptrs),
                                       tables_global, table_base, stream), "mpe_forward_routed")

    def gather_grad(self, grad_ptrs, tables_global, table_base, batch, d_grad_local, stream=None):
        """Pull this handle's columns of every rank's gradient buffer into d_grad_local ([batch][tables * dim])."""
        arr = (_vp * len(grad_ptrs))(*[int(p) for p in grad_ptrs])
        _check(_lib.mpe_gather_grad(self._h, arr, len(grad_ptrs), tables_global, table_base, batch, _ptr(d_grad_local), stream),
               "mpe_gather_grad")

    def backward(self, d_grad_out, lr, step):
        _check(_lib.mpe_backward(self._h, _ptr(d_grad_out), lr, step), "mpe_backward")

    def step_host(self, h_indices, h_offsets, batch, h_grad_out, h_out, lr, step):
        n = h_indices.size if isinstance(h_indices, np.ndarray) else h_indices.numel()
        _check(_lib.mpe_step_host(self._h, _ptr(h_indices), _ptr(h_offsets), batch, n, _ptr(h_grad_out), _ptr(h_out),
                                  lr, step), "mpe_step_host")

    def step_host_submit(self, h_indices, h_offsets, batch, h_grad_out, h_out, lr, step):
        """Enqueue one step from host buffers without waiting; the buffers belong to the library until step_host_wait()."""
        n = h_indices.size if isinstance(h_indices, np.ndarray) else h_indices.numel()
        _check(_lib.mpe_step_host_submit(self._h, _ptr(h_indices), _ptr(h_offsets), batch, n, _ptr(h_grad_out), _ptr(h_out),
                                         lr, step), "mpe_step_host_submit")

    def step_host_wait(self):
        _check(_lib.mpe_step_host_wait(self._h), "mpe_step_host_wait")

    def flush(self):
        _check(_lib.mpe_flush(self._h), "mpe_flush")

    # ---- observation ------------------------------------------------------------------------
    def last_error(self):
        code, detail = _i32(), _i64()
        _check(_lib.mpe_last_error(self._h, C.byref(code), C.byref(detail)), "mpe_last_error")
        return code.value, detail.value

    def selftest(self, which):
        _check(_lib.mpe_selftest(self._h, which), "mpe_selftest")

    def stats(self, table):
        out = np.zeros(8, np.uint64)
        _check(_lib.mpe_stats(self._h, table, out.ctypes.data), "mpe_stats")
        return out

    def memory_bytes(self):
        out = np.zeros(6, np.uint64)
        _check(_lib.mpe_memory_bytes(self._h, out.ctypes.data), "mpe_memory_bytes")
        return out

    def workspace_bytes(self):
        """(bytes of the per-step workspace, bytes of the host-step staging buffers)."""
        out = np.zeros(2, np.uint64)
        _check(_lib.mpe_workspace_bytes(self._h, out.ctypes.data), "mpe_workspace_bytes")
        return int(out[0]), int(out[1])

    def cache_geometry(self, table):
        n, w = _i32(), _i32()
        _check(_lib.mpe_cache_geometry(self._h, table, C.byref(n), C.byref(w)), "mpe_cache_geometry")
        return n.value, w.value

    def step_info(self):
        out = np.zeros(6, np.int64)
        _check(_lib.mpe_step_info(self._h, out.ctypes.data), "mpe_step_info")
        return out

    def export_rows(self, table, rows):
        rows = np.ascontiguousarray(rows, np.int64)
        n = rows.size
        codes = np.zeros((n, self.dim * self.bits // 8), np.uint8)
        scale = np.zeros(n, np.float32)
        bias = np.zeros(n, np.float32)
        _check(_lib.mpe_export_rows(self._h, table, rows.ctypes.data, n, codes.ctypes.data, scale.ctypes.data,
                                    bias.ctypes.data), "mpe_export_rows")
        return codes, scale, bias

    def export_cache(self, table):
        n_sets, ways = self.cache_geometry(table)
        slots = n_sets * ways
        tags = np.zeros(max(slots, 1), np.int32)
        rows = np.zeros((max(slots, 1), self.dim), np.float32)
        ts = np.zeros(max(slots, 1), np.uint32)
        _check(_lib.mpe_export_cache(self._h, table, tags.ctypes.data, rows.ctypes.data, ts.ctypes.data), "mpe_export_cache")
        return tags[:slots], rows[:slots], ts[:slots]

    def export_aux(self, table, rows):
        rows = np.ascontiguousarray(rows, np.int64)
        cnt = np.zeros(max(rows.size, 1), np.uint32)
        G = np.zeros(max(rows.size, 1), np.float32)
        _check(_lib.mpe_export_aux(self._h, table, rows.ctypes.data, rows.size, cnt.ctypes.data, G.ctypes.data), "mpe_export_aux")
        return cnt[:rows.size], G[:rows.size]

    def set_rounding(self, mode):
        _check(_lib.mpe_set_rounding(self._h, mode), "mpe_set_rounding")

    def use_graphs(self, enable):
        _check(_lib.mpe_use_graphs(self._h, 1 if enable else 0), "mpe_use_graphs")

    # ---- instrumentation --------------------------------------------------------------------
    def kernel_launches(self):
        c = _u64()
        _check(_lib.mpe_kernel_launches(self._h, C.byref(c)), "mpe_kernel_launches")
        return c.value

    def profile(self, enable):
        _check(_lib.mpe_profile(self._h, 1 if enable else 0), "mpe_profile")

    def profile_read(self, cap=64):
        names = C.create_string_buffer(32 * cap)
        ms = np.zeros(cap, np.float64)
        launches = np.zeros(cap, np.uint64)
        n = _i32()
        _check(_lib.mpe_profile_read(self._h, cap, C.addressof(names), ms.ctypes.data, launches.ctypes.data, C.byref(n)),
               "mpe_profile_read")
        out = {}
        for i in range(n.value):
            name = names.raw[32 * i:32 * i + 32].split(b"\0")[0].decode()
            out[name] = (float(ms[i]), int(launches[i]))
        return out


IPC_HANDLE_BYTES = 64


def peer_buffer_alloc(device, nbytes):
    """(device address, 64-byte handle other processes can open) of a fresh exchange buffer."""
    p, hd = _vp(), C.create_string_buffer(IPC_HANDLE_BYTES)
    _check(_lib.mpe_peer_buffer_alloc(device, nbytes, C.byref(p), hd), "mpe_peer_buffer_alloc")
    return p.value, hd.raw


def peer_buffer_open(device, handle):
    p = _vp()
    _check(_lib.mpe_peer_buffer_open(device, C.create_string_buffer(handle, IPC_HANDLE_BYTES), C.byref(p)), "mpe_peer_buffer_open")
    return p.value


def peer_buffer_close(device, address):
    _check(_lib.mpe_peer_buffer_close(device, address), "mpe_peer_buffer_close")


def peer_buffer_free(device, address):
    _check(_lib.mpe_peer_buffer_free(device, address), "mpe_peer_buffer_free")
