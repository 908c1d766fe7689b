"""ctypes wrapper over ``pdkv_oracle.c`` -- TEST INFRASTRUCTURE, not the product.

The arithmetic lives in the C file (plain nested loops following Sec. 3.5 of
the paper); this module only marshals numpy arrays.  It must never be imported
by the library package: only tests, the smoke check and the benchmark's
CPU-baseline leg use it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pdkv_oracle.c")
_LIB = os.path.join(_HERE, "libpdkv_oracle.so")


def build(force: bool = False) -> str:
    """Compile the C checker with gcc (no CUDA involved)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-Wall", "-Wextra", "-shared",
                               "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


class _Geom(C.Structure):
    _fields_ = [("layout", C.c_int32), ("L", C.c_int32), ("H", C.c_int32),
                ("D", C.c_int32), ("E", C.c_int32), ("B", C.c_int32), ("NB", C.c_int64)]


class _Batch(C.Structure):
    _fields_ = [("n_req", C.c_int32), ("G", C.c_int32),
                ("seq_len", C.c_void_p), ("src_tbl_off", C.c_void_p), ("src_tbl", C.c_void_p),
                ("dst_tbl_off", C.c_void_p), ("dst_tbl", C.c_void_p), ("skip", C.c_void_p)]


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        lib.okv_kept_tokens.restype = C.c_int64
        lib.okv_kept_tokens.argtypes = [C.POINTER(_Batch), C.c_int]
        lib.okv_request_offset.restype = C.c_int64
        lib.okv_request_offset.argtypes = [C.POINTER(_Batch), C.c_int, C.c_int, C.c_int, C.c_int]
        lib.okv_buffer_elems.restype = C.c_int64
        lib.okv_buffer_elems.argtypes = [C.POINTER(_Batch), C.c_int, C.c_int, C.c_int]
        lib.okv_pack.restype = None
        lib.okv_pack.argtypes = [C.POINTER(_Geom), C.c_void_p, C.POINTER(_Batch), C.c_void_p,
                                 C.c_int, C.c_int, C.c_int, C.c_int]
        lib.okv_unpack.restype = None
        lib.okv_unpack.argtypes = [C.POINTER(_Geom), C.c_void_p, C.POINTER(_Batch), C.c_void_p,
                                   C.c_int, C.c_int, C.c_int, C.c_int]
        lib.okv_transfer.restype = None
        lib.okv_transfer.argtypes = [C.POINTER(_Geom), C.c_void_p, C.POINTER(_Geom), C.c_void_p,
                                     C.POINTER(_Batch), C.c_int, C.c_int, C.c_int, C.c_int]
        _lib = lib
    return _lib


def _geom(g) -> _Geom:
    """``g`` is any object with layout/num_layers/... attributes (duck-typed)."""
    return _Geom(g.layout, g.num_layers, g.num_kv_heads, g.head_dim, g.elem_bytes,
                 g.block_tokens, g.num_blocks)


class _BatchRef:
    """Keeps the numpy arrays alive while the C struct points into them."""

    def __init__(self, batch, granule: int):
        self.arrs = [
            np.ascontiguousarray(batch.seq_len, np.int32),
            np.ascontiguousarray(batch.src_tbl_off, np.int64),
            np.ascontiguousarray(batch.src_tbl, np.int32),
            np.ascontiguousarray(batch.dst_tbl_off, np.int64),
            np.ascontiguousarray(batch.dst_tbl, np.int32),
        ]
        skip = batch.dst_skip
        self.skip = None if skip is None else np.ascontiguousarray(skip, np.uint8)
        p = [a.ctypes.data for a in self.arrs]
        self.c = _Batch(len(self.arrs[0]), int(granule), p[0], p[1], p[2], p[3], p[4],
                        None if self.skip is None else self.skip.ctypes.data)


def _bytes_view(a: np.ndarray) -> np.ndarray:
    if not a.flags.c_contiguous:
        raise ValueError("arrays handed to the checker must be contiguous")
    return a.reshape(-1).view(np.uint8)


def _run(fn, n_req, threads, r0, r1):
    r0 = 0 if r0 is None else r0
    r1 = n_req if r1 is None else r1
    if threads <= 1 or r1 - r0 <= 1:
        fn(r0, r1)
        return
    cuts = np.linspace(r0, r1, min(threads, r1 - r0) + 1).astype(int)
    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(lambda i: fn(int(cuts[i]), int(cuts[i + 1])), range(len(cuts) - 1)))


def kept_tokens(batch, granule: int) -> np.ndarray:
    lib, b = _load(), _BatchRef(batch, granule)
    return np.array([lib.okv_kept_tokens(C.byref(b.c), r) for r in range(batch.n_req)], np.int64)


def request_offsets(batch, granule: int, geom) -> np.ndarray:
    """Element offsets off_r of every request in the buffer, plus the total."""
    lib, b = _load(), _BatchRef(batch, granule)
    return np.array([lib.okv_request_offset(C.byref(b.c), geom.num_layers, geom.num_kv_heads,
                                            geom.head_dim, r) for r in range(batch.n_req + 1)],
                    np.int64)


def buffer_elems(batch, granule: int, geom) -> int:
    lib, b = _load(), _BatchRef(batch, granule)
    return int(lib.okv_buffer_elems(C.byref(b.c), geom.num_layers, geom.num_kv_heads,
                                    geom.head_dim))


def pack(src_geom, src_pool: np.ndarray, batch, granule: int, buf: np.ndarray,
         layers=None, requests=(None, None), threads: int = 1) -> None:
    lib, b, g = _load(), _BatchRef(batch, granule), _geom(src_geom)
    l0, l1 = layers if layers is not None else (0, src_geom.num_layers)
    s, d = _bytes_view(src_pool), _bytes_view(buf)
    _run(lambda a, z: lib.okv_pack(C.byref(g), s.ctypes.data, C.byref(b.c), d.ctypes.data,
                                   l0, l1, a, z), batch.n_req, threads, *requests)


def unpack(dst_geom, dst_pool: np.ndarray, batch, buf: np.ndarray,
           layers=None, requests=(None, None), threads: int = 1) -> None:
    lib, b, g = _load(), _BatchRef(batch, dst_geom.block_tokens), _geom(dst_geom)
    l0, l1 = layers if layers is not None else (0, dst_geom.num_layers)
    s, d = _bytes_view(buf), _bytes_view(dst_pool)
    _run(lambda a, z: lib.okv_unpack(C.byref(g), d.ctypes.data, C.byref(b.c), s.ctypes.data,
                                     l0, l1, a, z), batch.n_req, threads, *requests)


def transfer(src_geom, src_pool: np.ndarray, dst_geom, dst_pool: np.ndarray, batch,
             layers=None, requests=(None, None), threads: int = 1) -> None:
    lib, b = _load(), _BatchRef(batch, dst_geom.block_tokens)
    gs, gd = _geom(src_geom), _geom(dst_geom)
    l0, l1 = layers if layers is not None else (0, src_geom.num_layers)
    s, d = _bytes_view(src_pool), _bytes_view(dst_pool)
    _run(lambda a, z: lib.okv_transfer(C.byref(gs), s.ctypes.data, C.byref(gd), d.ctypes.data,
                                       C.byref(b.c), l0, l1, a, z),
         batch.n_req, threads, *requests)
