"""Thin ctypes binding of libtensair.so: same names as the C ABI, argument marshalling only.

PyTorch is used for device memory and streams; every step of the path runs in the library's kernels.
There is no fallback: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path
from typing import Optional

import numpy as np

import os

_HERE = Path(__file__).resolve().parent
# TENSAIR_CHECKED=1 loads the checked build (every data-dependent index compared with its bound on the device)
CHECKED = os.environ.get("TENSAIR_CHECKED", "0") == "1"
LIB_PATH = _HERE / ("libtensair_checked.so" if CHECKED else "libtensair.so")

SUM, MEAN = 0, 1
OK, EINVAL, ENOMEM, ECUDA, EBADTOKEN, EPENDING, ENOTFOUND, ETIMEOUT, EBOUNDS = 0, -1, -2, -3, -4, -5, -6, -7, -8


class Config(C.Structure):
    _fields_ = [("V", C.c_uint32), ("d", C.c_uint32), ("window", C.c_uint32), ("k", C.c_uint32),
                ("batch", C.c_uint32), ("W", C.c_uint32), ("lr", C.c_float), ("max_grad_buffer", C.c_uint32),
                ("max_delay", C.c_uint32), ("row_stride", C.c_uint32), ("seed", C.c_uint64),
                ("device", C.c_int32), ("reduction", C.c_uint32)]


class Sizes(C.Structure):
    _fields_ = [("tables_bytes", C.c_uint64), ("pool_bytes", C.c_uint64), ("scratch_bytes", C.c_uint64),
                ("row_stride", C.c_uint32), ("max_pairs", C.c_uint32), ("max_rows", C.c_uint32),
                ("reserved", C.c_uint32)]


class Buffers(C.Structure):
    _fields_ = [("tables", C.c_void_p), ("tables_bytes", C.c_uint64), ("pool", C.c_void_p),
                ("pool_bytes", C.c_uint64), ("scratch", C.c_void_p), ("scratch_bytes", C.c_uint64),
                ("stream", C.c_void_p)]


class MsgInfo(C.Structure):
    _fields_ = [("n_rows", C.c_uint32), ("n_in_rows", C.c_uint32), ("n_pairs", C.c_uint32), ("slot", C.c_uint32),
                ("pool_offset", C.c_uint64)]


class MsgView(C.Structure):
    _fields_ = [("ids", C.c_void_p), ("delta", C.c_void_p), ("max_rows", C.c_uint32), ("row_stride", C.c_uint32),
                ("ids_offset", C.c_uint64), ("delta_offset", C.c_uint64), ("header_offset", C.c_uint64)]


class Delivery(C.Structure):
    _fields_ = [("origin_step", C.c_uint64), ("sender", C.c_uint64), ("due_step", C.c_uint64),
                ("applied_at", C.c_uint64), ("staleness", C.c_uint64)]


class KernelTime(C.Structure):
    _fields_ = [("name", C.c_char * 32), ("launches", C.c_uint64), ("total_ms", C.c_double)]


class TensairError(RuntimeError):
    def __init__(self, code: int, what: str, detail: str = ""):
        self.code = code
        super().__init__(f"{what} failed: {code} ({strerror(code)}){': ' + detail if detail else ''}")


# every symbol include/tensair.h declares: name -> (restype, argtypes)
_u32, _u64, _i32, _vp, _int = C.c_uint32, C.c_uint64, C.c_int32, C.c_void_p, C.c_int
_P = C.POINTER
SYMBOLS = {
    "tensair_workspace_bytes": (_int, [_P(Config), _P(Sizes)]),
    "tensair_init": (_int, [_P(Config), _P(Buffers), _vp, _vp, _vp, _P(_vp)]),
    "tensair_workspace_bytes_sharded": (_int, [_P(Config), _u32, _P(Sizes)]),
    "tensair_init_sharded": (_int, [_P(Config), _P(Buffers), _vp, _vp, _vp, _u32, _u32, _P(_vp)]),
    "tensair_message_buffers": (_int, [_vp, _u32, _u64, _P(MsgView)]),
    "tensair_message_rows": (_int, [_vp, _u32, _u64, _P(_u32), _P(_u32)]),
    "tensair_commit_message": (_int, [_vp, _u32, _u64, _u32, _u32]),
    "tensair_commit_message_on": (_int, [_vp, _u32, _u64, _u32, _u32, _vp]),
    "tensair_shadow_apply": (_int, [_vp, _u32, _u64, _int, _P(_u32)]),
    "tensair_destroy": (None, [_vp]),
    "tensair_train_batch": (_int, [_vp, _u32, _vp, _u32, _u64, _P(C.c_double), _P(MsgInfo)]),
    "tensair_train_batch_host": (_int, [_vp, _u32, _vp, _u32, _u64, _P(C.c_double), _P(MsgInfo)]),
    "tensair_train_batch_routed": (_int, [_vp, _u32, _vp, _u32, _u64, _P(C.c_double), _P(MsgInfo)]),
    "tensair_route": (_int, [_u64, _u32, _u32, _vp]),
    "tensair_train_batch_static": (_int, [_vp, _u32, _vp, _u32, _u64, _P(C.c_double), _P(MsgInfo)]),
    "tensair_apply_messages": (_int, [_vp, _u32, _u64, _P(_u32)]),
    "tensair_apply_step": (_int, [_vp, _u64, _P(_u32)]),
    "tensair_drain": (_int, [_vp, _P(_u32)]),
    "tensair_update_sampler": (_int, [_vp]),
    "tensair_read_loss_async": (_int, [_vp, _vp]),
    "tensair_sync": (_int, [_vp]),
    "tensair_read_embeddings": (_int, [_vp, _u32, _int, _u32, _u32, _vp]),
    "tensair_write_embeddings": (_int, [_vp, _u32, _int, _u32, _u32, _vp]),
    "tensair_snapshot_rows": (_int, [_vp, _u32, _int, _u32, _u32, _vp]),
    "tensair_cosine_difference": (_int, [_vp, _u32, _int, _u32, _u32, _vp, _vp]),
    "tensair_top_drifted": (_int, [_vp, _vp, _u32, _u32, _vp, _vp, _vp]),
    "tensair_read_negatives": (_int, [_vp, _vp, _P(_u32)]),
    "tensair_read_scalars": (_int, [_vp, _vp]),
    "tensair_read_message": (_int, [_vp, _u32, _u64, _P(_u32), _vp, _vp]),
    "tensair_read_sampler": (_int, [_vp, _vp, _vp, _vp]),
    "tensair_read_delivery_log": (_int, [_vp, _u32, _u64, _vp, _P(_u64)]),
    "tensair_pending": (_int, [_vp, _u32, _P(_u64)]),
    "tensair_kernel_launches": (_u64, [_vp]),
    "tensair_profile": (_int, [_vp, _int]),
    "tensair_tune": (_int, [C.c_char_p, _int]),
    "tensair_profile_read": (_int, [_vp, _u32, _vp, _P(_u32)]),
    "tensair_strerror": (C.c_char_p, [_int]),
    "tensair_last_error": (C.c_char_p, [_vp]),
    "tensair_error_of_flags": (_int, [_u32]),
    "tensair_checked_build": (_int, []),
    "tensair_raise_error_flags": (_int, [_vp, _u32]),
    "tensair_build_alias_host": (_int, [_vp, _u32, _vp, _vp]),
    "tensair_philox4x32_10": (None, [_P(_u32), _P(_u32), _P(_u32)]),
    "tensair_delay": (_u32, [_u64, _u32, _u64, _u32, _u32]),
    "tensair_schedule_create": (_int, [_u32, _u32, _u64, _P(_vp)]),
    "tensair_schedule_destroy": (None, [_vp]),
    "tensair_schedule_on_train": (_int, [_vp, _u32, _u64]),
    "tensair_schedule_take_due": (_int, [_vp, _u32, _u64, _int, _u64, _vp, _P(_u64)]),
    "tensair_schedule_pending": (_int, [_vp, _u32, _P(_u64)]),
    "tensair_schedule_save": (_int, [_vp, _vp, _u64, _P(_u64)]),
    "tensair_schedule_load": (_int, [_vp, C.c_char_p, _u64]),
    "tensair_save_state": (_int, [_vp, _vp, _u64, _P(_u64)]),
    "tensair_load_state": (_int, [_vp, C.c_char_p, _u64]),
}

_lib = None


def lib():
    """The loaded library.  Raises if it has not been built: there is no other code path."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2211_10280_b200.build"
                               f"{' --bounds' if CHECKED else ''}`")
        L = C.CDLL(str(LIB_PATH))
        for name, (res, args) in SYMBOLS.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
        # launch-shape knobs from the environment: TENSAIR_TUNE="knob=value,knob=value" (see tensair_tune)
        for item in filter(None, os.environ.get("TENSAIR_TUNE", "").split(",")):
            name, value = item.split("=")
            if L.tensair_tune(name.strip().encode(), int(value)) != OK:
                raise RuntimeError(f"TENSAIR_TUNE: unknown knob or bad value in {item!r}")
    return _lib


def _np_ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def strerror(code: int) -> str:
    return lib().tensair_strerror(code).decode()


def _check(rc: int, what: str, ctx=None):
    if rc != OK:
        detail = lib().tensair_last_error(ctx).decode() if ctx else ""
        raise TensairError(rc, what, detail)


# ------------------------------------------------------------------ host-only calls
def tensair_workspace_bytes(cfg: Config) -> Sizes:
    out = Sizes()
    _check(lib().tensair_workspace_bytes(C.byref(cfg), C.byref(out)), "tensair_workspace_bytes")
    return out


def tensair_workspace_bytes_sharded(cfg: Config, world_replicas: int) -> Sizes:
    out = Sizes()
    _check(lib().tensair_workspace_bytes_sharded(C.byref(cfg), world_replicas, C.byref(out)),
           "tensair_workspace_bytes_sharded")
    return out


def tensair_build_alias_host(counts: Optional[np.ndarray], V: int):
    if counts is not None:
        counts = np.ascontiguousarray(counts, dtype=np.uint64)
    thresh = np.empty(V, np.uint32)
    alias = np.empty(V, np.uint32)
    _check(lib().tensair_build_alias_host(_np_ptr(counts), V, _np_ptr(thresh), _np_ptr(alias)), "tensair_build_alias_host")
    return thresh, alias


def tensair_philox4x32_10(counter, key):
    c = (C.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in counter])
    k = (C.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    o = (C.c_uint32 * 4)()
    lib().tensair_philox4x32_10(c, k, o)
    return [int(x) for x in o]


def tensair_error_of_flags(flags: int) -> int:
    return int(lib().tensair_error_of_flags(flags))


def tensair_tune(name: str, value: int):
    _check(lib().tensair_tune(name.encode(), value), "tensair_tune")


def tensair_delay(seed: int, max_delay: int, step: int, sender: int, receiver: int) -> int:
    return int(lib().tensair_delay(seed, max_delay, step, sender, receiver))


def tensair_route(seed: int, W: int, token: int) -> int:
    out = C.c_uint32(0)
    rc = lib().tensair_route(seed, W, token, C.byref(out))
    if rc != OK:
        raise TensairError(rc, "tensair_route")
    return int(out.value)


class Schedule:
    """tensair_schedule_*: the delivery schedule and staleness bookkeeping on their own (no GPU)."""

    def __init__(self, W: int, max_delay: int, seed: int):
        h = C.c_void_p()
        _check(lib().tensair_schedule_create(W, max_delay, seed, C.byref(h)), "tensair_schedule_create")
        self._h = h

    def on_train(self, replica: int, step: int) -> int:
        return int(lib().tensair_schedule_on_train(self._h, replica, step))

    def take_due(self, receiver: int, step: int, drain: bool = False) -> np.ndarray:
        n = C.c_uint64(0)
        cap = 4096
        buf = (Delivery * cap)()
        _check(lib().tensair_schedule_take_due(self._h, receiver, step, int(drain), cap, buf, C.byref(n)),
               "tensair_schedule_take_due")
        assert n.value <= cap
        return np.array([[r.origin_step, r.sender, r.due_step, r.applied_at, r.staleness] for r in buf[:n.value]],
                        dtype=np.uint64).reshape(-1, 5)

    def pending(self, receiver: int) -> int:
        n = C.c_uint64(0)
        _check(lib().tensair_schedule_pending(self._h, receiver, C.byref(n)), "tensair_schedule_pending")
        return int(n.value)

    def save(self) -> bytes:
        n = C.c_uint64(0)
        _check(lib().tensair_schedule_save(self._h, None, 0, C.byref(n)), "tensair_schedule_save")
        buf = C.create_string_buffer(n.value)
        _check(lib().tensair_schedule_save(self._h, buf, n.value, C.byref(n)), "tensair_schedule_save")
        return buf.raw[:n.value]

    def load(self, blob: bytes) -> int:
        return int(lib().tensair_schedule_load(self._h, blob, len(blob)))

    def __del__(self):
        try:
            lib().tensair_schedule_destroy(self._h)
        except Exception:
            pass


# ------------------------------------------------------------------ device context
class Context:
    """Owns the torch allocations a tensair_ctx borrows and forwards calls to the C ABI."""

    def __init__(self, V, d, window, k, batch, W=1, lr=0.025, max_delay=0, seed=0, counts=None,
                 init_in=None, init_out=None, device=0, row_stride=0, stream=None, reduction=SUM,
                 max_grad_buffer=1, world_replicas=None, first_replica=0):
        """W replicas live in this context.  world_replicas (default W) > W makes it one shard of a job whose
        replicas are spread over several processes: see tensair_init_sharded."""
        import torch

        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the SGNS path has no CPU implementation")
        self.torch = torch
        self.device = torch.device("cuda", device)
        self.cfg = Config(V=V, d=d, window=window, k=k, batch=batch, W=W, lr=lr, max_grad_buffer=max_grad_buffer,
                          max_delay=max_delay, row_stride=row_stride, seed=seed, device=device, reduction=reduction)
        self.world_replicas = W if world_replicas is None else world_replicas
        self.first_replica = first_replica
        self.sizes = tensair_workspace_bytes_sharded(self.cfg, self.world_replicas)
        with torch.cuda.device(self.device):
            self.stream = stream if stream is not None else torch.cuda.current_stream()
            self.tables = torch.empty(self.sizes.tables_bytes, dtype=torch.uint8, device=self.device)
            self.pool = torch.empty(self.sizes.pool_bytes, dtype=torch.uint8, device=self.device)
            self.scratch = torch.empty(self.sizes.scratch_bytes, dtype=torch.uint8, device=self.device)
        bufs = Buffers(self.tables.data_ptr(), self.sizes.tables_bytes, self.pool.data_ptr(), self.sizes.pool_bytes,
                       self.scratch.data_ptr(), self.sizes.scratch_bytes, self.stream.cuda_stream)
        if counts is not None:
            counts = np.ascontiguousarray(counts, dtype=np.uint64)
            assert counts.size == V
        if init_in is not None:
            init_in = np.ascontiguousarray(init_in, dtype=np.float32)
            assert init_in.shape == (V, d)
        if init_out is not None:
            init_out = np.ascontiguousarray(init_out, dtype=np.float32)
            assert init_out.shape == (V, d)
        h = C.c_void_p()
        if self.world_replicas == W and first_replica == 0:
            _check(lib().tensair_init(C.byref(self.cfg), C.byref(bufs), _np_ptr(counts), _np_ptr(init_in),
                                      _np_ptr(init_out), C.byref(h)), "tensair_init")
        else:
            _check(lib().tensair_init_sharded(C.byref(self.cfg), C.byref(bufs), _np_ptr(counts), _np_ptr(init_in),
                                              _np_ptr(init_out), first_replica, self.world_replicas, C.byref(h)),
                   "tensair_init_sharded")
        self._h = h
        self._keep = []

    # -- lifetime
    def close(self):
        if getattr(self, "_h", None):
            lib().tensair_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _train(self, fn, name, replica, ptr, n, batch_index, want_loss, want_info):
        loss = C.c_double(0.0)
        info = MsgInfo()
        rc = fn(self._h, replica, ptr, n, batch_index, C.byref(loss) if want_loss else None,
                C.byref(info) if want_info else None)
        _check(rc, name, self._h)
        return (loss.value if want_loss else None), (info if want_info else None)

    def tensair_train_batch(self, replica, tokens_dev, batch_index, want_loss=False, want_info=False):
        """tokens_dev: int32 CUDA tensor.  Returns (loss or None, MsgInfo or None)."""
        assert tokens_dev.is_cuda and tokens_dev.dtype == self.torch.int32 and tokens_dev.is_contiguous()
        return self._train(lib().tensair_train_batch, "tensair_train_batch", replica, tokens_dev.data_ptr(),
                           tokens_dev.numel(), batch_index, want_loss, want_info)

    def tensair_train_batch_routed(self, replica, tokens_dev, batch_index, want_loss=False, want_info=False):
        """The replica's share of a batch all replicas are handed: the pairs whose centre word is routed to it."""
        assert tokens_dev.is_cuda and tokens_dev.dtype == self.torch.int32 and tokens_dev.is_contiguous()
        return self._train(lib().tensair_train_batch_routed, "tensair_train_batch_routed", replica,
                           tokens_dev.data_ptr(), tokens_dev.numel(), batch_index, want_loss, want_info)

    def tensair_train_batch_static(self, replica, tokens_dev, batch_index, want_loss=False, want_info=False):
        """tensair_train_batch with the per-batch working memory taken from the library's built-in array."""
        assert tokens_dev.is_cuda and tokens_dev.dtype == self.torch.int32 and tokens_dev.is_contiguous()
        return self._train(lib().tensair_train_batch_static, "tensair_train_batch_static", replica,
                           tokens_dev.data_ptr(), tokens_dev.numel(), batch_index, want_loss, want_info)

    def tensair_train_batch_host(self, replica, tokens_host, batch_index, want_loss=False, want_info=False):
        """tokens_host: int32 numpy array or CPU tensor (pinned for an asynchronous copy)."""
        if isinstance(tokens_host, np.ndarray):
            assert tokens_host.dtype == np.int32 and tokens_host.flags.c_contiguous
            ptr, n = tokens_host.ctypes.data, tokens_host.size
        else:
            assert (not tokens_host.is_cuda) and tokens_host.dtype == self.torch.int32 and tokens_host.is_contiguous()
            ptr, n = tokens_host.data_ptr(), tokens_host.numel()
        return self._train(lib().tensair_train_batch_host, "tensair_train_batch_host", replica, ptr, n, batch_index,
                           want_loss, want_info)

    def tensair_apply_messages(self, replica, step) -> int:
        n = C.c_uint32(0)
        _check(lib().tensair_apply_messages(self._h, replica, step, C.byref(n)), "tensair_apply_messages", self._h)
        return int(n.value)

    def tensair_apply_step(self, step) -> int:
        """tensair_apply_messages for every replica of the context in one pass; returns the deliveries made."""
        n = C.c_uint32(0)
        _check(lib().tensair_apply_step(self._h, step, C.byref(n)), "tensair_apply_step", self._h)
        return int(n.value)

    def tensair_drain(self) -> int:
        n = C.c_uint32(0)
        _check(lib().tensair_drain(self._h, C.byref(n)), "tensair_drain", self._h)
        return int(n.value)

    # -- messages between processes (sharded jobs)
    def tensair_message_buffers(self, sender, batch_index):
        """(ids, delta): int32 / float32 CUDA tensors that ARE the pool slot of the message of (global sender,
        batch_index), at full capacity ([max_rows] and [max_rows * row_stride])."""
        v = MsgView()
        _check(lib().tensair_message_buffers(self._h, sender, batch_index, C.byref(v)), "tensair_message_buffers", self._h)
        ids = self.pool[v.ids_offset:v.ids_offset + 4 * v.max_rows].view(self.torch.int32)
        delta = self.pool[v.delta_offset:v.delta_offset + 4 * v.max_rows * v.row_stride].view(self.torch.float32)
        assert ids.data_ptr() == v.ids and delta.data_ptr() == v.delta
        return ids, delta

    def tensair_message_rows(self, replica, batch_index):
        """(rows, input rows) of a local replica's message.  Synchronises."""
        n, n_in = C.c_uint32(0), C.c_uint32(0)
        _check(lib().tensair_message_rows(self._h, replica, batch_index, C.byref(n), C.byref(n_in)),
               "tensair_message_rows", self._h)
        return int(n.value), int(n_in.value)

    def tensair_message_header(self, sender, batch_index):
        """int32 CUDA tensor [2] that IS the head of the slot's header: (rows, input rows) of the message, as the
        kernels that built it left them (valid once the stream has passed them)."""
        v = MsgView()
        _check(lib().tensair_message_buffers(self._h, sender, batch_index, C.byref(v)), "tensair_message_buffers", self._h)
        return self.pool[v.header_offset:v.header_offset + 8].view(self.torch.int32)

    def tensair_commit_message(self, sender, batch_index, n_rows, n_in_rows, stream=None):
        """stream: a torch.cuda.Stream on which the slot's header and index are written (default: the context's)."""
        _check(lib().tensair_commit_message_on(self._h, sender, batch_index, n_rows, n_in_rows,
                                               stream.cuda_stream if stream is not None else None),
               "tensair_commit_message_on", self._h)

    def tensair_shadow_apply(self, receiver, step, drain=False) -> int:
        n = C.c_uint32(0)
        _check(lib().tensair_shadow_apply(self._h, receiver, step, int(drain), C.byref(n)), "tensair_shadow_apply", self._h)
        return int(n.value)

    def tensair_save_state(self) -> bytes:
        """The library's part of a run in flight (sampler state, buffered-message counts, delivery schedule)."""
        n = C.c_uint64(0)
        _check(lib().tensair_save_state(self._h, None, 0, C.byref(n)), "tensair_save_state", self._h)
        buf = C.create_string_buffer(n.value)
        _check(lib().tensair_save_state(self._h, buf, n.value, C.byref(n)), "tensair_save_state", self._h)
        return buf.raw[:n.value]

    def tensair_load_state(self, blob: bytes):
        _check(lib().tensair_load_state(self._h, blob, len(blob)), "tensair_load_state", self._h)

    def tensair_update_sampler(self):
        _check(lib().tensair_update_sampler(self._h), "tensair_update_sampler", self._h)

    def tensair_read_loss_async(self, host_ptr: int):
        """Enqueues the copy of the last batch loss into the (pinned) host double at address host_ptr."""
        _check(lib().tensair_read_loss_async(self._h, host_ptr), "tensair_read_loss_async", self._h)

    def tensair_sync(self) -> int:
        """Returns the status (OK, EBADTOKEN, ETIMEOUT or EBOUNDS) instead of raising."""
        return int(lib().tensair_sync(self._h))

    def tensair_raise_error_flags(self, flags: int):
        _check(lib().tensair_raise_error_flags(self._h, flags), "tensair_raise_error_flags", self._h)

    def tensair_last_error(self) -> str:
        return lib().tensair_last_error(self._h).decode()

    def tensair_read_embeddings(self, replica, which, row0=0, nrows=None) -> np.ndarray:
        nrows = self.cfg.V - row0 if nrows is None else nrows
        out = np.empty((nrows, self.cfg.d), np.float32)
        _check(lib().tensair_read_embeddings(self._h, replica, which, row0, nrows, _np_ptr(out)),
               "tensair_read_embeddings", self._h)
        return out

    def tensair_write_embeddings(self, replica, which, row0, rows: np.ndarray):
        rows = np.ascontiguousarray(rows, dtype=np.float32)
        _check(lib().tensair_write_embeddings(self._h, replica, which, row0, rows.shape[0], _np_ptr(rows)),
               "tensair_write_embeddings", self._h)

    def tensair_snapshot_rows(self, replica, which, row0=0, nrows=None):
        """A dense float32 CUDA tensor [nrows, d] holding the rows as they are now."""
        nrows = self.cfg.V - row0 if nrows is None else nrows
        snap = self.torch.empty((nrows, self.cfg.d), dtype=self.torch.float32, device=self.device)
        _check(lib().tensair_snapshot_rows(self._h, replica, which, row0, nrows, snap.data_ptr()),
               "tensair_snapshot_rows", self._h)
        return snap

    def tensair_cosine_difference(self, replica, which, snap, row0=0):
        """float32 CUDA tensor [nrows]: 1 - cos(row now, row in `snap`)."""
        assert snap.is_cuda and snap.dtype == self.torch.float32 and snap.is_contiguous() and snap.shape[1] == self.cfg.d
        out = self.torch.empty(snap.shape[0], dtype=self.torch.float32, device=self.device)
        _check(lib().tensair_cosine_difference(self._h, replica, which, row0, snap.shape[0], snap.data_ptr(),
                                               out.data_ptr()), "tensair_cosine_difference", self._h)
        return out

    def tensair_top_drifted(self, diff, k):
        """(ids int32-viewable uint32 CUDA tensor [m], values float32 CUDA tensor [m]), m = min(k, len(diff))."""
        assert diff.is_cuda and diff.dtype == self.torch.float32 and diff.is_contiguous() and diff.dim() == 1
        ids = self.torch.empty(k, dtype=self.torch.int32, device=self.device)
        vals = self.torch.empty(k, dtype=self.torch.float32, device=self.device)
        m = C.c_uint32(0)
        _check(lib().tensair_top_drifted(self._h, diff.data_ptr(), diff.shape[0], k, ids.data_ptr(), vals.data_ptr(),
                                         C.byref(m)), "tensair_top_drifted", self._h)
        return ids[:m.value], vals[:m.value]

    def tensair_read_negatives(self) -> np.ndarray:
        n = C.c_uint32(0)
        _check(lib().tensair_read_negatives(self._h, None, C.byref(n)), "tensair_read_negatives", self._h)
        out = np.empty((n.value, self.cfg.k), np.uint32)
        _check(lib().tensair_read_negatives(self._h, _np_ptr(out), None), "tensair_read_negatives", self._h)
        return out

    def tensair_read_scalars(self) -> np.ndarray:
        n = C.c_uint32(0)
        _check(lib().tensair_read_negatives(self._h, None, C.byref(n)), "tensair_read_negatives", self._h)
        out = np.empty((n.value, self.cfg.k + 1), np.float64)
        _check(lib().tensair_read_scalars(self._h, _np_ptr(out)), "tensair_read_scalars", self._h)
        return out

    def tensair_read_message(self, replica, batch_index):
        """(ids uint32[n], delta float32[n, d]) or None when the message is no longer held."""
        n = C.c_uint32(0)
        rc = lib().tensair_read_message(self._h, replica, batch_index, C.byref(n), None, None)
        if rc == ENOTFOUND:
            return None
        _check(rc, "tensair_read_message", self._h)
        ids = np.empty(n.value, np.uint32)
        delta = np.empty((n.value, self.cfg.d), np.float32)
        _check(lib().tensair_read_message(self._h, replica, batch_index, None, _np_ptr(ids), _np_ptr(delta)),
               "tensair_read_message", self._h)
        return ids, delta

    def tensair_read_message_ids(self, replica, batch_index):
        """The row ids of a held message (uint32[n]) without its delta rows, or None."""
        n = C.c_uint32(0)
        rc = lib().tensair_read_message(self._h, replica, batch_index, C.byref(n), None, None)
        if rc == ENOTFOUND:
            return None
        _check(rc, "tensair_read_message", self._h)
        ids = np.empty(n.value, np.uint32)
        _check(lib().tensair_read_message(self._h, replica, batch_index, None, _np_ptr(ids), None),
               "tensair_read_message", self._h)
        return ids

    def tensair_read_sampler(self):
        V = self.cfg.V
        thresh, alias, counts = np.empty(V, np.uint32), np.empty(V, np.uint32), np.empty(V, np.uint64)
        _check(lib().tensair_read_sampler(self._h, _np_ptr(thresh), _np_ptr(alias), _np_ptr(counts)),
               "tensair_read_sampler", self._h)
        return thresh, alias, counts

    def tensair_read_delivery_log(self, replica) -> np.ndarray:
        n = C.c_uint64(0)
        _check(lib().tensair_read_delivery_log(self._h, replica, 0, None, C.byref(n)), "tensair_read_delivery_log", self._h)
        buf = (Delivery * max(1, n.value))()
        _check(lib().tensair_read_delivery_log(self._h, replica, n.value, buf, None), "tensair_read_delivery_log", self._h)
        return np.array([[r.origin_step, r.sender, r.due_step, r.applied_at, r.staleness] for r in buf[:n.value]],
                        dtype=np.uint64).reshape(-1, 5)

    def tensair_pending(self, replica) -> int:
        n = C.c_uint64(0)
        _check(lib().tensair_pending(self._h, replica, C.byref(n)), "tensair_pending", self._h)
        return int(n.value)

    def tensair_kernel_launches(self) -> int:
        return int(lib().tensair_kernel_launches(self._h))

    def tensair_profile(self, enable: bool):
        _check(lib().tensair_profile(self._h, int(enable)), "tensair_profile", self._h)

    def tensair_profile_read(self) -> dict:
        """{kernel name: (launches, total milliseconds)} since the previous read."""
        n = C.c_uint32(0)
        buf = (KernelTime * 64)()
        _check(lib().tensair_profile_read(self._h, 64, buf, C.byref(n)), "tensair_profile_read", self._h)
        return {buf[i].name.decode(): (int(buf[i].launches), float(buf[i].total_ms)) for i in range(min(64, n.value))}
