"""Thin ctypes binding of libtpi.so: the same calls as include/tpi.h, argument
marshalling only.  Every step of the decoder path runs inside the CUDA library;
PyTorch appears only in ``Session`` to allocate the two arenas and the streams.

There is no CPU path: if the shared library is missing, importing ``lib()``
raises, and ``load_model`` fails when no CUDA device is present.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Callable, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtpi.so")

TPI_F32, TPI_BF16 = 0, 1
OPT_GRAPH, OPT_PDL, OPT_PROFILE, OPT_TENSOR, OPT_WAIT_DEADLINE_MS, OPT_ROWSHARD_FUSED = 0, 1, 2, 3, 4, 5
(T_EMB, T_HEAD, T_FINAL_NORM, T_ATTN_NORM, T_WQ, T_WK, T_WV, T_WO,
 T_FFN_NORM, T_WGATE, T_WUP, T_WDOWN) = range(12)


class TpiError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"tpi error {code}: {msg}")
        self.code = code


class TpiConfig(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("hidden", C.c_int32), ("n_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("ffn", C.c_int32),
                ("vocab", C.c_int32), ("max_seq", C.c_int32), ("max_prefill", C.c_int32),
                ("rms_eps", C.c_float), ("rope_base", C.c_float), ("dtype", C.c_int32)]


class TpiResources(C.Structure):
    _fields_ = [("dev_arena", C.c_void_p), ("dev_bytes", C.c_size_t),
                ("host_arena", C.c_void_p), ("host_bytes", C.c_size_t),
                ("compute_stream", C.c_void_p), ("copy_stream", C.c_void_p)]


class TpiStats(C.Structure):
    _fields_ = [("last_prefill_ms", C.c_double), ("last_decode_ms", C.c_double),
                ("last_decode_dev_ms", C.c_double), ("weight_bytes_per_token", C.c_uint64),
                ("link_bytes_total", C.c_uint64), ("blocks_loaded", C.c_uint64),
                ("stall_ms_total", C.c_double), ("dominant_kernel_ms", C.c_double),
                ("dominant_kernel_bytes", C.c_uint64), ("dominant_kernel_samples", C.c_uint32),
                ("kernel_launches_last", C.c_int32), ("window_blocks", C.c_int32),
                ("n_shards", C.c_int32), ("position", C.c_int32), ("graph_active", C.c_int32),
                ("window_peak_bytes", C.c_uint64), ("retained_bytes", C.c_uint64),
                ("retained_blocks", C.c_int32), ("reserved_", C.c_int32),
                ("last_prefill_dev_ms", C.c_double), ("last_prefill_enqueue_ms", C.c_double)]

    def as_dict(self) -> dict:
        return {k: getattr(self, k) for k, _ in self._fields_}


FILL_FN = C.CFUNCTYPE(C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_int64, C.c_int64, C.c_void_p)

# every symbol include/tpi.h declares: name -> (restype, argtypes)
SYMBOLS = {
    "tpi_query_arena": (C.c_int, [C.POINTER(TpiConfig), C.c_int, C.c_int, C.c_int,
                                  C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]),
    "tpi_block_bytes": (C.c_int, [C.POINTER(TpiConfig), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]),
    "tpi_load_model": (C.c_int, [C.POINTER(TpiConfig), C.POINTER(TpiResources), FILL_FN, C.c_void_p,
                                 C.c_int, C.c_int, C.POINTER(C.c_void_p)]),
    "tpi_set_shards": (C.c_int, [C.c_void_p, C.c_int]),
    "tpi_set_window": (C.c_int, [C.c_void_p, C.c_int]),
    "tpi_prefill": (C.c_int, [C.c_void_p, C.POINTER(C.c_int32), C.c_int, C.POINTER(C.c_int32),
                              C.POINTER(C.c_float)]),
    "tpi_decode_step": (C.c_int, [C.c_void_p, C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_float)]),
    "tpi_decode_run": (C.c_int, [C.c_void_p, C.c_int32, C.c_int, C.POINTER(C.c_int32)]),
    "tpi_reset": (C.c_int, [C.c_void_p]),
    "tpi_position": (C.c_int, [C.c_void_p]),
    "tpi_get_hidden": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_float)]),
    "tpi_get_kv": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_float),
                             C.POINTER(C.c_float)]),
    "tpi_put_kv": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_float),
                             C.POINTER(C.c_float)]),
    "tpi_set_position": (C.c_int, [C.c_void_p, C.c_int]),
    "tpi_get_stats": (C.c_int, [C.c_void_p, C.POINTER(TpiStats)]),
    "tpi_set_option": (C.c_int, [C.c_void_p, C.c_int, C.c_int]),
    "tpi_ring_trace": (C.c_int, [C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int), C.c_int]),
    "tpi_ring_trace_retained": (C.c_int, [C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int), C.c_int]),
    "tpi_ring_trace_faulty": (C.c_int, [C.c_int] * 7 + [C.POINTER(C.c_int), C.c_int]),
    "tpi_set_retention": (C.c_int, [C.c_void_p, C.c_int]),
    "tpi_set_partition": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]),
    "tpi_scheduler_report": (C.c_int, [C.c_void_p, C.c_void_p]),
    "tpi_scheduler_reset": (C.c_int, [C.c_void_p]),
    "tpi_steady_conditions": (C.c_int, [C.c_double] * 5 + [C.c_int] + [C.POINTER(C.c_int)] * 3),
    "tpi_free": (None, [C.c_void_p]),
    "tpi_strerror": (C.c_char_p, [C.c_int]),
    "tpi_last_error": (C.c_char_p, []),
}

_LIB = None


def lib() -> C.CDLL:
    """Load libtpi.so (built in-tree by ``paper_2410_00531_b200.build``)."""
    global _LIB
    if _LIB is None:
        path = LIB_PATH
        if os.environ.get("TPI_TIMELINE", "0") not in ("", "0"):   # the instrumented twin (see build.py)
            path = os.path.join(_HERE, "libtpi_timeline.so")
        if not os.path.exists(path):   # a fresh checkout: compile it once (nvcc), or fail loudly
            try:
                from . import build as _build
                _build.build()
            except Exception as e:
                raise ImportError(f"{path} is missing and could not be built ({e}): run "
                                  "`python -m paper_2410_00531_b200.build` (this package has no CPU fallback)") from e
        L = C.CDLL(path)
        for name, (res, args) in SYMBOLS.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _LIB = L
    return _LIB


def _check(rc: int) -> int:
    if rc < 0:
        L = lib()
        raise TpiError(rc, f"{L.tpi_strerror(rc).decode()}: {L.tpi_last_error().decode()}")
    return rc


def _fptr(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_float))


# ------------------------------------------------------------------ the calls of tpi.h
def query_arena(cfg: TpiConfig, n_shards_max: int, window_blocks: int, keep_host_images: bool):
    d, h = C.c_size_t(), C.c_size_t()
    _check(lib().tpi_query_arena(C.byref(cfg), n_shards_max, window_blocks, int(keep_host_images),
                                 C.byref(d), C.byref(h)))
    return d.value, h.value


def block_bytes(cfg: TpiConfig):
    a, f = C.c_size_t(), C.c_size_t()
    _check(lib().tpi_block_bytes(C.byref(cfg), C.byref(a), C.byref(f)))
    return a.value, f.value


def load_model(cfg: TpiConfig, res: TpiResources, fill_cb, n_shards: int, window_blocks: int) -> C.c_void_p:
    h = C.c_void_p()
    _check(lib().tpi_load_model(C.byref(cfg), C.byref(res), fill_cb, None, n_shards, window_blocks, C.byref(h)))
    return h


def set_shards(h, n: int) -> None:
    _check(lib().tpi_set_shards(h, n))


def set_window(h, w: int) -> None:
    _check(lib().tpi_set_window(h, w))


def prefill(h, tokens, vocab: int = 0):
    """Returns (first_token, logits or None); logits are fetched when vocab > 0."""
    t = np.ascontiguousarray(tokens, dtype=np.int32)
    out = C.c_int32()
    lg = np.empty(vocab, np.float32) if vocab else None
    _check(lib().tpi_prefill(h, t.ctypes.data_as(C.POINTER(C.c_int32)), t.size, C.byref(out),
                             _fptr(lg) if vocab else None))
    return out.value, lg


def decode_step(h, token_in: int, vocab: int = 0):
    out = C.c_int32()
    lg = np.empty(vocab, np.float32) if vocab else None
    _check(lib().tpi_decode_step(h, int(token_in), C.byref(out), _fptr(lg) if vocab else None))
    return out.value, lg


def decode_run(h, token_in: int, n_steps: int) -> np.ndarray:
    out = np.empty(n_steps, np.int32)
    _check(lib().tpi_decode_run(h, int(token_in), n_steps, out.ctypes.data_as(C.POINTER(C.c_int32))))
    return out


def reset(h) -> None:
    _check(lib().tpi_reset(h))


def position(h) -> int:
    return _check(lib().tpi_position(h))


def set_position(h, p: int) -> None:
    _check(lib().tpi_set_position(h, p))


def get_hidden(h, layer: int, which: int, hidden: int) -> np.ndarray:
    out = np.empty(hidden, np.float32)
    _check(lib().tpi_get_hidden(h, layer, which, _fptr(out)))
    return out


def get_kv(h, layer: int, kv_head: int, pos0: int, n: int, head_dim: int):
    k, v = np.empty((n, head_dim), np.float32), np.empty((n, head_dim), np.float32)
    _check(lib().tpi_get_kv(h, layer, kv_head, pos0, n, _fptr(k), _fptr(v)))
    return k, v


def put_kv(h, layer: int, kv_head: int, pos0: int, k: np.ndarray, v: np.ndarray) -> None:
    k = np.ascontiguousarray(k, np.float32)
    v = np.ascontiguousarray(v, np.float32)
    _check(lib().tpi_put_kv(h, layer, kv_head, pos0, k.shape[0], _fptr(k), _fptr(v)))


def get_stats(h) -> dict:
    s = TpiStats()
    _check(lib().tpi_get_stats(h, C.byref(s)))
    return s.as_dict()


def set_option(h, option: int, value: int) -> None:
    _check(lib().tpi_set_option(h, option, value))


class TpiSchedReport(C.Structure):
    _fields_ = [(n, C.c_double) for n in ("t_attn_ms", "t_ffn_ms", "t_all_reduce_ms", "tau_attn_ms", "tau_ffn_ms",
                                          "stall_ms_total")] + \
               [(n, C.c_uint32) for n in ("n_t_attn", "n_t_ffn", "n_tau_attn", "n_tau_ffn")] + \
               [(n, C.c_int32) for n in ("tight_holds", "loose_holds", "retention_T", "window_blocks",
                                         "retain_every_T", "reserved_")] + \
               [("m_worker_bytes", C.c_uint64), ("window_device_bytes", C.c_uint64)]


def scheduler_report(h) -> dict:
    r = TpiSchedReport()
    _check(lib().tpi_scheduler_report(h, C.byref(r)))
    return {n: getattr(r, n) for n, _ in r._fields_ if n != "reserved_"}


def scheduler_reset(h) -> None:
    _check(lib().tpi_scheduler_reset(h))


def steady_conditions(t_attn, t_ffn, t_all_reduce, tau_attn, tau_ffn, n_layers: int):
    """Returns (tight, loose, retention_T)."""
    a, b, c = C.c_int(), C.c_int(), C.c_int()
    _check(lib().tpi_steady_conditions(t_attn, t_ffn, t_all_reduce, tau_attn, tau_ffn, n_layers,
                                       C.byref(a), C.byref(b), C.byref(c)))
    return bool(a.value), bool(b.value), c.value


def set_partition(h, kv_heads_per_shard, ffn_cols_per_shard) -> None:
    kv = np.ascontiguousarray(kv_heads_per_shard, dtype=np.int32)
    ff = np.ascontiguousarray(ffn_cols_per_shard, dtype=np.int32)
    if kv.shape != ff.shape or kv.ndim != 1:
        raise ValueError("one entry per shard in both lists")
    _check(lib().tpi_set_partition(h, int(kv.size), kv.ctypes.data_as(C.POINTER(C.c_int32)),
                                   ff.ctypes.data_as(C.POINTER(C.c_int32))))


def set_retention(h, ffn_every_T: int) -> None:
    _check(lib().tpi_set_retention(h, ffn_every_T))


def ring_trace(n_blocks: int, w: int, n_exec: int, max_ops: int = 1 << 16, ffn_every_T: int = 0) -> np.ndarray:
    ops = np.zeros((max_ops, 3), np.int32)
    n = _check(lib().tpi_ring_trace_retained(n_blocks, w, n_exec, ffn_every_T,
                                             ops.ctypes.data_as(C.POINTER(C.c_int)), max_ops))
    if n > max_ops:
        raise ValueError("trace buffer too small")
    return ops[:n]


def ring_trace_faulty(n_blocks: int, w: int, n_exec: int, fail_copy: int, fail_status: int, retry: bool,
                      ffn_every_T: int = 0, max_ops: int = 1 << 16) -> np.ndarray:
    """The ring's ordering trace when block copy number `fail_copy` fails once; raises TpiError(fail_status) unless retry."""
    ops = np.zeros((max_ops, 3), np.int32)
    n = _check(lib().tpi_ring_trace_faulty(n_blocks, w, n_exec, ffn_every_T, fail_copy, fail_status, int(retry),
                                           ops.ctypes.data_as(C.POINTER(C.c_int)), max_ops))
    if n > max_ops:
        raise ValueError("trace buffer too small")
    return ops[:n]


def free(h) -> None:
    lib().tpi_free(h)


# ------------------------------------------------------------------ arenas + lifetime
FillFn = Callable[[int, int, int, int, int, int], None]
"""fill(tensor_id, layer, row0, n_rows, dst_address, n_bytes): write the rows in storage dtype."""


def make_config(*, n_layers, hidden, n_heads, n_kv_heads, head_dim, ffn, vocab, max_seq, max_prefill,
                rms_eps=1e-5, rope_base=10000.0, dtype="bf16") -> TpiConfig:
    return TpiConfig(n_layers, hidden, n_heads, n_kv_heads, head_dim, ffn, vocab, max_seq, max_prefill,
                     rms_eps, rope_base, TPI_BF16 if dtype == "bf16" else TPI_F32)


class Session:
    """Owns the arenas (torch tensors), the streams and the model handle."""

    def __init__(self, cfg: TpiConfig, fill: FillFn, n_shards: int, window_blocks: int = 0,
                 keep_host_images: Optional[bool] = None, device: int = 0, other_windows=(),
                 extra_dev_bytes: int = 0):
        """other_windows: window sizes this session may later switch to with set_window
        (the device arena is sized for the largest of them; 0 means fully resident)."""
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2410_00531_b200 needs a CUDA device (sm_100a); there is no CPU path")
        self.cfg = cfg
        self.torch = torch
        torch.cuda.set_device(device)
        if keep_host_images is None:
            keep_host_images = window_blocks > 0
        d_need, h_need = query_arena(cfg, n_shards, window_blocks, keep_host_images)
        for w in other_windows:
            keep_host_images = True
            d_need = max(d_need, query_arena(cfg, n_shards, w, True)[0])
        if keep_host_images:
            h_need = query_arena(cfg, n_shards, window_blocks, True)[1]
        d_need += int(extra_dev_bytes)      # e.g. room for retained blocks (tpi_set_retention)
        self.dev = torch.empty(d_need, dtype=torch.uint8, device=f"cuda:{device}")
        self.host = torch.empty(h_need, dtype=torch.uint8, pin_memory=True)
        self.compute = torch.cuda.Stream(device=device)
        self.copy = torch.cuda.Stream(device=device)
        esz = 2 if cfg.dtype == TPI_BF16 else 4
        rowlen = {T_WO: cfg.n_heads * cfg.head_dim, T_WDOWN: cfg.ffn}

        def _cb(_user, tid, layer, row0, n_rows, dst):
            try:
                fill(tid, layer, row0, n_rows, dst, n_rows * rowlen.get(tid, cfg.hidden) * esz)
                return 0
            except Exception as e:  # surfaced as TPI_ERR_CALLBACK
                self.fill_error = e
                return 1
        self.fill_error = None
        self._cb = FILL_FN(_cb)     # must outlive the model (tpi_set_shards calls it again)
        res = TpiResources(self.dev.data_ptr(), d_need, self.host.data_ptr(), h_need,
                           self.compute.cuda_stream, self.copy.cuda_stream)
        self.h = load_model(cfg, res, self._cb, n_shards, window_blocks)

    def close(self) -> None:
        if getattr(self, "h", None):
            free(self.h)
            self.h = None
        self.dev = self.host = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
