"""ctypes binding of the CPU oracle (test infrastructure only).

Only the tests, the smoke check and the CPU-baseline leg of the benchmark may import this package.
It compiles `tensair_oracle.cpp` with g++ on first use and never touches the CUDA library.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "tensair_oracle.cpp"
_LIB = _HERE / "libtensair_oracle.so"


def build(force: bool = False) -> Path:
    """Compile the oracle into a shared library next to its source."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fopenmp", "-fPIC", "-shared",
                               "-ffp-contract=off", "-o", str(tmp), str(_SRC)])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(str(build()))
        u32, u64, i32, f32, f64, vp = C.c_uint32, C.c_uint64, C.c_int32, C.c_float, C.c_double, C.c_void_p
        P = C.POINTER
        sig = {
            "orc_philox4x32_10": (None, [P(u32), P(u32), P(u32)]),
            "orc_build_alias": (None, [vp, u32, vp, vp]),
            "orc_negative": (u32, [u64, u32, u64, u32, u32, vp, vp, u32]),
            "orc_init_input_table": (None, [u64, u32, u32, vp]),
            "orc_create": (vp, [u32, u32, u32, u32, u32, u32, f32, u32, u64, u32, vp, vp, vp]),
            "orc_destroy": (None, [vp]),
            "orc_set_max_grad_buffer": (None, [vp, u32]),
            "orc_update_sampler": (None, [vp]),
            "orc_get_sampler": (None, [vp, vp, vp, vp]),
            "orc_batch_loss": (f64, [vp, u32, vp, u32, u64]),
            "orc_train_batch": (C.c_int, [vp, u32, vp, u32, u64, P(f64), P(u32)]),
            "orc_train_batch_routed": (C.c_int, [vp, u32, vp, u32, u64, P(f64), P(u32)]),
            "orc_route": (u32, [u64, u32, u32]),
            "orc_apply_messages": (C.c_int, [vp, u32, u64]),
            "orc_drain": (C.c_int, [vp]),
            "orc_read_embeddings": (None, [vp, u32, C.c_int, u32, u32, vp]),
            "orc_write_embeddings": (None, [vp, u32, C.c_int, u32, u32, vp]),
            "orc_last_pairs": (u32, [vp]),
            "orc_read_negatives": (None, [vp, vp]),
            "orc_read_g": (None, [vp, vp]),
            "orc_read_message": (C.c_int64, [vp, u32, u64, vp, vp]),
            "orc_delay": (u32, [vp, u64, u32, u32]),
            "orc_log_size": (u64, [vp, u32]),
            "orc_read_log": (None, [vp, u32, vp]),
            "orc_pending": (u64, [vp, u32]),
            "orc_book_create": (vp, [u32]),
            "orc_book_destroy": (None, [vp]),
            "orc_book_compute": (u64, [vp, u32]),
            "orc_book_apply": (u32, [vp, u32, u64]),
            "orc_book_size": (u32, [vp, u32]),
            "orc_cosine_difference": (None, [vp, vp, u32, u32, vp]),
            "orc_top_drifted": (u32, [vp, u32, u32, vp, vp]),
            "orc_threads": (C.c_int, []),
        }
        for name, (res, args) in sig.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def philox4x32_10(ctr, key):
    c = (C.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in ctr])
    k = (C.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    o = (C.c_uint32 * 4)()
    lib().orc_philox4x32_10(c, k, o)
    return [int(x) for x in o]


def build_alias(counts):
    counts = np.ascontiguousarray(counts, dtype=np.uint64)
    V = counts.size
    thresh = np.empty(V, dtype=np.uint32)
    alias = np.empty(V, dtype=np.uint32)
    lib().orc_build_alias(_ptr(counts), V, _ptr(thresh), _ptr(alias))
    return thresh, alias


def negative(seed, replica, batch_index, p, j, thresh, alias):
    return int(lib().orc_negative(seed, replica, batch_index, p, j, _ptr(thresh), _ptr(alias), thresh.size))


def init_input_table(seed, V, d):
    out = np.empty((V, d), dtype=np.float32)
    lib().orc_init_input_table(seed, V, d, _ptr(out))
    return out


def cosine_difference(a, b):
    """1 - cos(a_r, b_r) per row of two float32 arrays [n, d]."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    b = np.ascontiguousarray(b, dtype=np.float32)
    assert a.shape == b.shape and a.ndim == 2
    out = np.empty(a.shape[0], dtype=np.float32)
    lib().orc_cosine_difference(_ptr(a), _ptr(b), a.shape[0], a.shape[1], _ptr(out))
    return out


def route(seed, W, token) -> int:
    return int(lib().orc_route(seed, W, token))


def top_drifted(diff, k):
    """(ids, values) of the k largest entries of a float32 array, largest first, smaller index first among equals."""
    diff = np.ascontiguousarray(diff, dtype=np.float32)
    ids = np.empty(min(k, diff.size), dtype=np.uint32)
    vals = np.empty(min(k, diff.size), dtype=np.float32)
    m = lib().orc_top_drifted(_ptr(diff), diff.size, k, _ptr(ids), _ptr(vals))
    assert m == ids.size
    return ids, vals


def threads() -> int:
    return int(lib().orc_threads())


class Oracle:
    """The oracle's model replicas, sampler and message exchange."""

    def __init__(self, V, d, window, k, batch, W=1, lr=0.025, max_delay=0, seed=0,
                 counts=None, init_in=None, init_out=None, reduction=0, max_grad_buffer=1):
        self.V, self.d, self.window, self.k, self.batch, self.W = V, d, window, k, batch, W
        self.seed = seed
        if counts is not None:
            counts = np.ascontiguousarray(counts, dtype=np.uint64)
            assert counts.size == V
        if init_in is not None:
            init_in = np.ascontiguousarray(init_in, dtype=np.float32)
            assert init_in.shape == (V, d)
        if init_out is not None:
            init_out = np.ascontiguousarray(init_out, dtype=np.float32)
            assert init_out.shape == (V, d)
        self._h = lib().orc_create(V, d, window, k, batch, W, lr, max_delay, seed, reduction,
                                   _ptr(counts), _ptr(init_in), _ptr(init_out))
        lib().orc_set_max_grad_buffer(self._h, max_grad_buffer)

    def close(self):
        if self._h:
            lib().orc_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def train_batch(self, replica, tokens, batch_index):
        """Returns (status, loss, n_rows)."""
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        loss = C.c_double(0.0)
        nrows = C.c_uint32(0)
        rc = lib().orc_train_batch(self._h, replica, _ptr(tokens), tokens.size, batch_index,
                                   C.byref(loss), C.byref(nrows))
        return rc, loss.value, nrows.value

    def train_batch_routed(self, replica, tokens, batch_index):
        """The replica's share of the batch (centre words routed to it).  Returns (status, loss, n_rows)."""
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        loss = C.c_double(0.0)
        nrows = C.c_uint32(0)
        rc = lib().orc_train_batch_routed(self._h, replica, _ptr(tokens), tokens.size, batch_index,
                                          C.byref(loss), C.byref(nrows))
        return rc, loss.value, nrows.value

    def batch_loss(self, replica, tokens, batch_index):
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        return float(lib().orc_batch_loss(self._h, replica, _ptr(tokens), tokens.size, batch_index))

    def apply_messages(self, replica, step):
        return int(lib().orc_apply_messages(self._h, replica, step))

    def drain(self):
        return int(lib().orc_drain(self._h))

    def update_sampler(self):
        lib().orc_update_sampler(self._h)

    def sampler(self):
        thresh = np.empty(self.V, dtype=np.uint32)
        alias = np.empty(self.V, dtype=np.uint32)
        counts = np.empty(self.V, dtype=np.uint64)
        lib().orc_get_sampler(self._h, _ptr(thresh), _ptr(alias), _ptr(counts))
        return thresh, alias, counts

    def read_embeddings(self, replica, which, row0=0, nrows=None):
        nrows = self.V - row0 if nrows is None else nrows
        out = np.empty((nrows, self.d), dtype=np.float32)
        lib().orc_read_embeddings(self._h, replica, which, row0, nrows, _ptr(out))
        return out

    def write_embeddings(self, replica, which, row0, rows):
        rows = np.ascontiguousarray(rows, dtype=np.float32)
        lib().orc_write_embeddings(self._h, replica, which, row0, rows.shape[0], _ptr(rows))

    def last_pairs(self):
        return int(lib().orc_last_pairs(self._h))

    def read_negatives(self):
        out = np.empty((self.last_pairs(), self.k), dtype=np.uint32)
        lib().orc_read_negatives(self._h, _ptr(out))
        return out

    def read_g(self):
        out = np.empty((self.last_pairs(), self.k + 1), dtype=np.float64)
        lib().orc_read_g(self._h, _ptr(out))
        return out

    def read_message(self, replica, batch_index):
        n = int(lib().orc_read_message(self._h, replica, batch_index, None, None))
        if n < 0:
            return None
        ids = np.empty(n, dtype=np.uint32)
        delta = np.empty((n, self.d), dtype=np.float32)
        lib().orc_read_message(self._h, replica, batch_index, _ptr(ids), _ptr(delta))
        return ids, delta

    def read_message_ids(self, replica, batch_index):
        """The row ids of a held message without its delta rows, or None."""
        n = int(lib().orc_read_message(self._h, replica, batch_index, None, None))
        if n < 0:
            return None
        ids = np.empty(n, dtype=np.uint32)
        lib().orc_read_message(self._h, replica, batch_index, _ptr(ids), None)
        return ids

    def delay(self, step, sender, receiver):
        return int(lib().orc_delay(self._h, step, sender, receiver))

    def delivery_log(self, replica):
        """uint64 array [n, 5]: origin step, sender, due step, applied at, staleness."""
        n = int(lib().orc_log_size(self._h, replica))
        out = np.empty((n, 5), dtype=np.uint64)
        lib().orc_read_log(self._h, replica, _ptr(out))
        return out

    def pending(self, replica):
        return int(lib().orc_pending(self._h, replica))


class StalenessBook:
    """Event-level bookkeeping of the applied-gradient sets G_i (Section 3.1)."""

    def __init__(self, models):
        self._h = lib().orc_book_create(models)

    def compute(self, model):
        return int(lib().orc_book_compute(self._h, model))

    def apply(self, model, grad):
        return int(lib().orc_book_apply(self._h, model, grad))

    def size(self, model):
        return int(lib().orc_book_size(self._h, model))

    def __del__(self):
        try:
            lib().orc_book_destroy(self._h)
        except Exception:
            pass
