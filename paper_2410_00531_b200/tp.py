"""ctypes binding of include/tpi_tp.h: the decoder step on R ranks, one shard each (argument marshalling only).

``Group`` owns what the C calls borrow: per rank a device arena, a pinned host arena and two streams (torch), on the
rank's device.  Ranks may share a device; the library then orders every exchange with CUDA events."""
from __future__ import annotations

import ctypes as C
from typing import Optional, Sequence

import numpy as np

from .binding import (FILL_FN, T_WDOWN, T_WO, TPI_BF16, TpiConfig, TpiResources, _check, _fptr, lib)

OPT_EVENTS, OPT_WAIT_POLLS, OPT_DROP_PUSH, OPT_PDL, OPT_BATCHED_PROMPT, OPT_GRAPH = 0, 1, 2, 3, 4, 5
_P, _I = C.c_void_p, C.c_int
_I64P = C.POINTER(C.c_int64)
_I32P = C.POINTER(C.c_int32)


def _lists(partition, n_ranks):
    """(kv heads per rank, FFN columns per rank) -> two int32 arrays (kept alive by the caller) or (None, None)."""
    if partition is None:
        return None, None, None
    kv = np.ascontiguousarray(partition[0], dtype=np.int32)
    ff = np.ascontiguousarray(partition[1], dtype=np.int32)
    if kv.shape != (n_ranks,) or ff.shape != (n_ranks,):
        raise ValueError("one entry per rank in both lists")
    return kv.ctypes.data_as(_I32P), ff.ctypes.data_as(_I32P), (kv, ff)


class TpStats(C.Structure):
    _fields_ = [("n_ranks", C.c_int32), ("position", C.c_int32), ("events", C.c_int32), ("kernel_launches_last", C.c_int32),
                ("exchanges_total", C.c_uint64), ("exchange_bytes_per_token", C.c_uint64),
                ("weight_bytes_rank0", C.c_uint64), ("weight_bytes_worker", C.c_uint64), ("last_decode_ms", C.c_double)]


TP_SYMBOLS = {
    "tpi_tp_rank_slice": (_I, [C.POINTER(TpiConfig), _I, _I, _I, _I64P, _I64P, _I64P, _I64P]),
    "tpi_tp_query_arena": (_I, [C.POINTER(TpiConfig), _I, _I, _I, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]),
    "tpi_tp_rank_slice_p": (_I, [C.POINTER(TpiConfig), _I, _I, _I32P, _I32P, _I, _I64P, _I64P, _I64P, _I64P]),
    "tpi_tp_query_arena_p": (_I, [C.POINTER(TpiConfig), _I, _I, _I32P, _I32P, _I, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]),
    "tpi_tp_create_p": (_I, [C.POINTER(TpiConfig), _I, _I32P, _I32P, C.POINTER(TpiResources), C.POINTER(C.c_int), FILL_FN, _P, _I,
                             C.POINTER(_P)]),
    "tpi_tp_create": (_I, [C.POINTER(TpiConfig), _I, C.POINTER(TpiResources), C.POINTER(C.c_int), FILL_FN, _P, _I, C.POINTER(_P)]),
    "tpi_tp_free": (None, [_P]),
    "tpi_tp_prefill": (_I, [_P, C.POINTER(C.c_int32), _I, C.POINTER(C.c_int32), C.POINTER(C.c_float)]),
    "tpi_tp_decode_step": (_I, [_P, C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_float)]),
    "tpi_tp_decode_run": (_I, [_P, C.c_int32, _I, C.POINTER(C.c_int32)]),
    "tpi_tp_reset": (_I, [_P]),
    "tpi_tp_position": (_I, [_P]),
    "tpi_tp_n_ranks": (_I, [_P]),
    "tpi_tp_get_hidden": (_I, [_P, _I, _I, _I, C.POINTER(C.c_float)]),
    "tpi_tp_get_kv": (_I, [_P, _I, _I, _I, _I, C.POINTER(C.c_float), C.POINTER(C.c_float)]),
    "tpi_tp_set_option": (_I, [_P, _I, _I]),
    "tpi_tp_get_stats": (_I, [_P, C.POINTER(TpStats)]),
}
_BOUND = False


def _tp():
    global _BOUND
    L = lib()
    if not _BOUND:
        for name, (res, args) in TP_SYMBOLS.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _BOUND = True
    return L


def rank_slice(cfg: TpiConfig, n_ranks: int, rank: int, tensor_id: int, partition=None):
    """(row0, n_rows, col0, n_cols) of the unsharded tensor that `rank` holds (host arithmetic, no GPU).
    partition: (kv heads per rank, FFN columns per rank) or None for the uniform 1/R."""
    v = [C.c_int64() for _ in range(4)]
    kv, ff, _keep = _lists(partition, n_ranks)
    _check(_tp().tpi_tp_rank_slice_p(C.byref(cfg), n_ranks, rank, kv, ff, tensor_id, *[C.byref(x) for x in v]))
    return tuple(x.value for x in v)


def query_arena(cfg: TpiConfig, n_ranks: int, rank: int, window_blocks: int = 0, partition=None):
    d, h = C.c_size_t(), C.c_size_t()
    kv, ff, _keep = _lists(partition, n_ranks)
    _check(_tp().tpi_tp_query_arena_p(C.byref(cfg), n_ranks, rank, kv, ff, window_blocks, C.byref(d), C.byref(h)))
    return d.value, h.value


class Group:
    """R ranks in this process; `devices` gives each rank's CUDA device (default: all on `device`)."""

    def __init__(self, cfg: TpiConfig, fill, n_ranks: int, window_blocks: int = 0, devices: Optional[Sequence[int]] = None,
                 device: int = 0, partition=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2410_00531_b200 needs a CUDA device (sm_100a); there is no CPU path")
        self.cfg, self.n_ranks, self.torch = cfg, n_ranks, torch
        devs = list(devices) if devices is not None else [device] * n_ranks
        self.dev, self.host, self.streams = [], [], []
        res = (TpiResources * n_ranks)()
        for i in range(n_ranks):
            d_need, h_need = query_arena(cfg, n_ranks, i, window_blocks, partition)
            torch.cuda.set_device(devs[i])
            self.dev.append(torch.empty(d_need, dtype=torch.uint8, device=f"cuda:{devs[i]}"))
            self.host.append(torch.empty(h_need, dtype=torch.uint8, pin_memory=True))
            self.streams.append((torch.cuda.Stream(device=devs[i]), torch.cuda.Stream(device=devs[i])))
            res[i] = TpiResources(self.dev[i].data_ptr(), d_need, self.host[i].data_ptr(), h_need,
                                  self.streams[i][0].cuda_stream, self.streams[i][1].cuda_stream)
        torch.cuda.set_device(devs[0])
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
        self._cb = FILL_FN(_cb)
        h = _P()
        dv = (C.c_int * n_ranks)(*devs)
        kv, ff, _keep = _lists(partition, n_ranks)
        _check(_tp().tpi_tp_create_p(C.byref(cfg), n_ranks, kv, ff, res, dv, self._cb, None, window_blocks, C.byref(h)))
        self.h = h

    def prefill(self, tokens, vocab: int = 0):
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        out = C.c_int32()
        lg = np.empty(vocab, np.float32) if vocab else None
        _check(_tp().tpi_tp_prefill(self.h, t.ctypes.data_as(C.POINTER(C.c_int32)), t.size, C.byref(out), _fptr(lg) if vocab else None))
        return out.value, lg

    def decode_step(self, token_in: int, vocab: int = 0):
        out = C.c_int32()
        lg = np.empty(vocab, np.float32) if vocab else None
        _check(_tp().tpi_tp_decode_step(self.h, int(token_in), C.byref(out), _fptr(lg) if vocab else None))
        return out.value, lg

    def decode_run(self, token_in: int, n_steps: int) -> np.ndarray:
        out = np.empty(n_steps, np.int32)
        _check(_tp().tpi_tp_decode_run(self.h, int(token_in), n_steps, out.ctypes.data_as(C.POINTER(C.c_int32))))
        return out

    def reset(self) -> None:
        _check(_tp().tpi_tp_reset(self.h))

    def position(self) -> int:
        return _check(_tp().tpi_tp_position(self.h))

    def get_hidden(self, rank: int, layer: int, which: int) -> np.ndarray:
        out = np.empty(self.cfg.hidden, np.float32)
        _check(_tp().tpi_tp_get_hidden(self.h, rank, layer, which, _fptr(out)))
        return out

    def get_kv(self, layer: int, kv_head: int, pos0: int, n: int):
        d = self.cfg.head_dim
        k, v = np.empty((n, d), np.float32), np.empty((n, d), np.float32)
        _check(_tp().tpi_tp_get_kv(self.h, layer, kv_head, pos0, n, _fptr(k), _fptr(v)))
        return k, v

    def set_option(self, option: int, value: int) -> None:
        _check(_tp().tpi_tp_set_option(self.h, option, value))

    def stats(self) -> dict:
        s = TpStats()
        _check(_tp().tpi_tp_get_stats(self.h, C.byref(s)))
        return {k: getattr(s, k) for k, _ in s._fields_}

    def close(self) -> None:
        if getattr(self, "h", None):
            _tp().tpi_tp_free(self.h)
            self.h = None
        self.dev = self.host = self.streams = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
