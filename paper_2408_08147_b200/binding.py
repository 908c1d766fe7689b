"""Thin ctypes binding over ``libpdkv.so`` (argument marshalling only).

Function names mirror ``include/pdkv.h``.  Every step of the path runs inside
the library's CUDA kernels; PyTorch (or any other allocator) is only the source
of device pointers and stream handles.  There is no CPU fallback: if the
library is missing the import of :func:`lib` fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpdkv.so")

PDKV_LAYOUT_BLOCK_MAJOR = 0
PDKV_LAYOUT_LAYER_MAJOR = 1

PDKV_OK = 0
PDKV_ERR_INVALID_ARG = -1
PDKV_ERR_GEOMETRY = -2
PDKV_ERR_TABLE = -3
PDKV_ERR_BUFFER_TOO_SMALL = -4
PDKV_ERR_CUDA = -5
PDKV_ERR_DEVICE_BOUNDS = -6
PDKV_ERR_NOMEM = -7
PDKV_ERR_LIMIT = -8
PDKV_ERR_BUSY = -9
PDKV_NOALLOC_MAX_TILES = 32768

PDKV_OP_PACK = 0
PDKV_OP_UNPACK = 1
PDKV_OP_TRANSFER = 2
PDKV_OP_BLOCKWISE = 3  # only for pdkv_plan_launches

EXPORTS = (
    "pdkv_pool_bytes", "pdkv_pool_create", "pdkv_pool_destroy", "pdkv_plan_create", "pdkv_plan_create_in",
    "pdkv_plan_destroy", "pdkv_plan_buffer", "pdkv_plan_traffic", "pdkv_pack", "pdkv_unpack",
    "pdkv_transfer", "pdkv_transfer_noalloc", "pdkv_transfer_blockwise", "pdkv_plan_launches", "pdkv_plan_tiles",
    "pdkv_plan_status", "pdkv_upload_blocks", "pdkv_download_blocks", "pdkv_plan_block_bytes",
    "pdkv_queue_create", "pdkv_queue_submit", "pdkv_queue_poll", "pdkv_queue_wait", "pdkv_queue_release",
    "pdkv_queue_stats", "pdkv_queue_destroy", "pdkv_tune", "pdkv_tune_get", "pdkv_strerror",
    "pdkv_plan_autotune", "pdkv_plan_shape", "pdkv_plan_set_shape", "pdkv_plan_launch_shape", "pdkv_plan_option",
    "pdkv_sm_partition_create", "pdkv_sm_partition_info", "pdkv_sm_partition_stream", "pdkv_sm_partition_destroy",
    "pdkv_transfer_copies",
)


class pdkv_pool_desc(C.Structure):
    _fields_ = [("layout", C.c_int32), ("num_layers", C.c_int32), ("num_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("elem_bytes", C.c_int32), ("block_tokens", C.c_int32),
                ("num_blocks", C.c_int64)]


class pdkv_batch_desc(C.Structure):
    _fields_ = [("n_req", C.c_int32), ("seq_len", C.c_void_p), ("src_tbl_off", C.c_void_p),
                ("src_tbl", C.c_void_p), ("dst_tbl_off", C.c_void_p), ("dst_tbl", C.c_void_p),
                ("dst_skip", C.c_void_p)]


class pdkv_tile(C.Structure):
    _fields_ = [("src_off", C.c_int64), ("dst_off", C.c_int64), ("ntok", C.c_int32),
                ("n_kept", C.c_int32)]


class pdkv_launch_shape(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("threads", "unroll", "ctas_per_sm", "group_threads", "vec_bytes", "max_ctas",
                                         "lc_skew", "lc_skew_shift", "lc_fastest", "chunked", "src_order", "variant",
                                         "debug_bounds")]


TILE_DTYPE = np.dtype([("src_off", "<i8"), ("dst_off", "<i8"), ("ntok", "<i4"), ("n_kept", "<i4")])


class PdkvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {pdkv_strerror(status)} ({status})")


_lib = None


def lib() -> C.CDLL:
    """Load the shared library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2408_08147_b200.build` "
            "(nvcc, sm_100a). There is no fallback path.")
    L = C.CDLL(LIB_PATH)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    L.pdkv_pool_bytes.restype = C.c_size_t
    L.pdkv_pool_bytes.argtypes = [C.POINTER(pdkv_pool_desc)]
    L.pdkv_pool_create.argtypes = [C.POINTER(pdkv_pool_desc), vp, C.c_size_t, C.c_int, C.POINTER(vp)]
    L.pdkv_pool_destroy.argtypes = [vp]
    L.pdkv_plan_create.argtypes = [vp, vp, i32, C.POINTER(pdkv_batch_desc), vp, C.POINTER(vp)]
    L.pdkv_plan_create_in.argtypes = [vp, vp, i32, C.POINTER(pdkv_batch_desc), vp, C.c_size_t,
                                      C.POINTER(C.c_size_t), vp, C.POINTER(vp)]
    L.pdkv_plan_destroy.argtypes = [vp]
    L.pdkv_plan_buffer.argtypes = [vp, C.POINTER(C.c_size_t), C.POINTER(C.POINTER(i64))]
    L.pdkv_plan_traffic.argtypes = [vp, C.c_int, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
    L.pdkv_pack.argtypes = [vp, vp, C.c_size_t, C.c_int, C.c_int, vp]
    L.pdkv_unpack.argtypes = [vp, vp, C.c_size_t, C.c_int, C.c_int, vp]
    L.pdkv_transfer.argtypes = [vp, C.c_int, C.c_int, vp]
    L.pdkv_transfer_noalloc.argtypes = [vp, vp, C.POINTER(pdkv_batch_desc), C.c_int, C.c_int, vp]
    L.pdkv_transfer_blockwise.argtypes = [vp, vp]
    L.pdkv_plan_launches.argtypes = [vp, C.c_int, C.POINTER(i64)]
    L.pdkv_plan_tiles.argtypes = [vp, C.c_int, C.POINTER(C.POINTER(pdkv_tile)), C.POINTER(i64)]
    L.pdkv_plan_status.argtypes = [vp, vp]
    L.pdkv_upload_blocks.argtypes = [vp, vp, vp]
    L.pdkv_download_blocks.argtypes = [vp, vp, vp]
    L.pdkv_plan_block_bytes.argtypes = [vp, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
    L.pdkv_queue_create.argtypes = [vp, vp, C.c_int, C.c_int, C.POINTER(vp)]
    L.pdkv_queue_submit.argtypes = [vp, C.POINTER(pdkv_batch_desc), vp, vp, vp, C.POINTER(i64)]
    L.pdkv_plan_launch_shape.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.POINTER(pdkv_launch_shape)]
    L.pdkv_plan_option.argtypes = [vp, C.c_char_p, C.POINTER(i64)]
    L.pdkv_sm_partition_create.argtypes = [C.c_int, C.c_int, C.POINTER(vp)]
    L.pdkv_sm_partition_info.argtypes = [vp, C.POINTER(C.c_int), C.POINTER(C.c_int)]
    L.pdkv_sm_partition_stream.argtypes = [vp, C.c_int, C.POINTER(vp)]
    L.pdkv_sm_partition_destroy.argtypes = [vp]
    L.pdkv_transfer_copies.argtypes = [vp, C.c_int, C.c_int, vp]
    L.pdkv_queue_poll.argtypes = [vp, i64, C.POINTER(C.c_int)]
    L.pdkv_queue_wait.argtypes = [vp, i64]
    L.pdkv_queue_release.argtypes = [vp, i64]
    L.pdkv_queue_stats.argtypes = [vp, C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(i64), C.POINTER(i64)]
    L.pdkv_queue_destroy.argtypes = [vp]
    L.pdkv_tune.argtypes = [C.c_char_p, i64]
    L.pdkv_tune_get.argtypes = [C.c_char_p, C.POINTER(i64)]
    L.pdkv_strerror.restype = C.c_char_p
    L.pdkv_strerror.argtypes = [C.c_int]
    for name in EXPORTS:
        if name not in ("pdkv_pool_bytes", "pdkv_strerror"):
            getattr(L, name).restype = C.c_int
    _lib = L
    return L


def _check(status: int, where: str) -> None:
    if status != PDKV_OK:
        raise PdkvError(status, where)


def pdkv_strerror(status: int) -> str:
    return lib().pdkv_strerror(status).decode()


def make_desc(layout, num_layers, num_kv_heads, head_dim, elem_bytes, block_tokens, num_blocks):
    return pdkv_pool_desc(layout, num_layers, num_kv_heads, head_dim, elem_bytes, block_tokens,
                          num_blocks)


def desc_of(geom) -> pdkv_pool_desc:
    """Descriptor from any object carrying the geometry attribute names."""
    return make_desc(geom.layout, geom.num_layers, geom.num_kv_heads, geom.head_dim,
                     geom.elem_bytes, geom.block_tokens, geom.num_blocks)


def pdkv_pool_bytes(desc: pdkv_pool_desc) -> int:
    return int(lib().pdkv_pool_bytes(C.byref(desc)))


def pdkv_pool_create(desc: pdkv_pool_desc, dev_ptr: int, nbytes: int, device: int) -> int:
    out = C.c_void_p()
    _check(lib().pdkv_pool_create(C.byref(desc), C.c_void_p(dev_ptr), nbytes, device,
                                  C.byref(out)), "pdkv_pool_create")
    return out.value


def pdkv_pool_destroy(pool: int) -> None:
    _check(lib().pdkv_pool_destroy(C.c_void_p(pool)), "pdkv_pool_destroy")


class _BatchArrays:
    """Contiguous, correctly typed copies of a batch, alive for one C call."""

    def __init__(self, seq_len, src_tbl_off, src_tbl, dst_tbl_off, dst_tbl, dst_skip):
        def arr(a, dt):
            return None if a is None else np.ascontiguousarray(a, dt)

        self.a = [arr(seq_len, np.int32), arr(src_tbl_off, np.int64), arr(src_tbl, np.int32),
                  arr(dst_tbl_off, np.int64), arr(dst_tbl, np.int32), arr(dst_skip, np.uint8)]
        p = [None if a is None else a.ctypes.data for a in self.a]
        n = 0 if self.a[0] is None else int(self.a[0].shape[0])
        self.desc = pdkv_batch_desc(n, *p)


def pdkv_plan_create(src_pool: Optional[int], dst_pool: Optional[int], skip_granule_tokens: int,
                     seq_len: Sequence[int], src_tbl_off=None, src_tbl=None, dst_tbl_off=None,
                     dst_tbl=None, dst_skip=None, stream: int = 0) -> int:
    b = _BatchArrays(seq_len, src_tbl_off, src_tbl, dst_tbl_off, dst_tbl, dst_skip)
    out = C.c_void_p()
    _check(lib().pdkv_plan_create(C.c_void_p(src_pool), C.c_void_p(dst_pool),
                                  skip_granule_tokens, C.byref(b.desc), C.c_void_p(stream),
                                  C.byref(out)), "pdkv_plan_create")
    return out.value


def pdkv_plan_create_in(src_pool: Optional[int], dst_pool: Optional[int], skip_granule_tokens: int,
                        seq_len, src_tbl_off=None, src_tbl=None, dst_tbl_off=None, dst_tbl=None,
                        dst_skip=None, workspace_ptr: int = 0, workspace_bytes: int = 0, stream: int = 0):
    """Plan whose device arrays live in caller-provided device memory.
    Returns (plan, needed_bytes); raises PdkvError(BUFFER_TOO_SMALL) with
    ``.needed_bytes`` set when the workspace is too small."""
    b = _BatchArrays(seq_len, src_tbl_off, src_tbl, dst_tbl_off, dst_tbl, dst_skip)
    out, need = C.c_void_p(), C.c_size_t()
    rc = lib().pdkv_plan_create_in(C.c_void_p(src_pool), C.c_void_p(dst_pool), skip_granule_tokens,
                                   C.byref(b.desc), C.c_void_p(workspace_ptr), workspace_bytes, C.byref(need),
                                   C.c_void_p(stream), C.byref(out))
    if rc != PDKV_OK:
        err = PdkvError(rc, "pdkv_plan_create_in")
        err.needed_bytes = int(need.value)
        raise err
    return out.value, int(need.value)


def pdkv_plan_autotune(plan: int, buf_ptr: int = 0, buf_bytes: int = 0, stream: int = 0) -> None:
    _check(lib().pdkv_plan_autotune(C.c_void_p(plan), C.c_void_p(buf_ptr), C.c_size_t(buf_bytes),
                                    C.c_void_p(stream)), "pdkv_plan_autotune")


def pdkv_plan_shape(plan: int, op: int):
    """(threads, unroll, ctas_per_sm, lc_skew) the plan uses for ``op``; zeros = the built-in
    shape, lc_skew -1 = by the stride rule."""
    t, u, c, k = C.c_int32(), C.c_int32(), C.c_int32(), C.c_int32()
    _check(lib().pdkv_plan_shape(C.c_void_p(plan), op, C.byref(t), C.byref(u), C.byref(c), C.byref(k)),
           "pdkv_plan_shape")
    return int(t.value), int(u.value), int(c.value), int(k.value)


def pdkv_plan_launch_shape(plan: int, op: int, layer_begin: int, layer_end: int) -> dict:
    """What the plan launches for ``op`` over the layer range, as a dict of the fields of
    ``pdkv_launch_shape``."""
    out = pdkv_launch_shape()
    _check(lib().pdkv_plan_launch_shape(C.c_void_p(plan), op, layer_begin, layer_end, C.byref(out)),
           "pdkv_plan_launch_shape")
    return {k: int(getattr(out, k)) for k, _ in pdkv_launch_shape._fields_}


def pdkv_plan_option(plan: int, key: str) -> int:
    v = C.c_int64()
    _check(lib().pdkv_plan_option(C.c_void_p(plan), key.encode(), C.byref(v)), f"pdkv_plan_option({key})")
    return int(v.value)


def pdkv_plan_set_shape(plan: int, op: int, threads: int, unroll: int, ctas_per_sm: int) -> None:
    _check(lib().pdkv_plan_set_shape(C.c_void_p(plan), op, threads, unroll, ctas_per_sm), "pdkv_plan_set_shape")


def pdkv_plan_destroy(plan: int) -> None:
    _check(lib().pdkv_plan_destroy(C.c_void_p(plan)), "pdkv_plan_destroy")


def pdkv_plan_buffer(plan: int, n_req: Optional[int] = None):
    """Returns (total_bytes, request offsets as int64 array or None)."""
    total = C.c_size_t()
    offs = C.POINTER(C.c_int64)()
    _check(lib().pdkv_plan_buffer(C.c_void_p(plan), C.byref(total), C.byref(offs)),
           "pdkv_plan_buffer")
    arr = None
    if n_req is not None:
        arr = np.ctypeslib.as_array(offs, shape=(n_req + 1,)).copy()
    return int(total.value), arr


def pdkv_plan_traffic(plan: int, op: int):
    r, w = C.c_uint64(), C.c_uint64()
    _check(lib().pdkv_plan_traffic(C.c_void_p(plan), op, C.byref(r), C.byref(w)),
           "pdkv_plan_traffic")
    return int(r.value), int(w.value)


def pdkv_pack(plan: int, buf_ptr: int, buf_bytes: int, layer_begin: int, layer_end: int,
              stream: int = 0) -> None:
    _check(lib().pdkv_pack(C.c_void_p(plan), C.c_void_p(buf_ptr), buf_bytes, layer_begin,
                           layer_end, C.c_void_p(stream)), "pdkv_pack")


def pdkv_unpack(plan: int, buf_ptr: int, buf_bytes: int, layer_begin: int, layer_end: int,
                stream: int = 0) -> None:
    _check(lib().pdkv_unpack(C.c_void_p(plan), C.c_void_p(buf_ptr), buf_bytes, layer_begin,
                             layer_end, C.c_void_p(stream)), "pdkv_unpack")


def pdkv_transfer(plan: int, layer_begin: int, layer_end: int, stream: int = 0) -> None:
    _check(lib().pdkv_transfer(C.c_void_p(plan), layer_begin, layer_end, C.c_void_p(stream)),
           "pdkv_transfer")


def pdkv_transfer_noalloc(src_pool: int, dst_pool: int, seq_len, src_tbl_off, src_tbl, dst_tbl_off,
                          dst_tbl, dst_skip, layer_begin: int, layer_end: int,
                          stream: int = 0) -> None:
    """Fused transfer that allocates no device memory (no plan object): the
    tile list goes into a fixed scratch array inside the library.  For callers
    that may not call cudaMalloc; batches are limited to
    ``PDKV_NOALLOC_MAX_TILES`` tiles, and overlapping calls race on the scratch."""
    b = _BatchArrays(seq_len, src_tbl_off, src_tbl, dst_tbl_off, dst_tbl, dst_skip)
    _check(lib().pdkv_transfer_noalloc(C.c_void_p(src_pool), C.c_void_p(dst_pool), C.byref(b.desc),
                                       layer_begin, layer_end, C.c_void_p(stream)),
           "pdkv_transfer_noalloc")


def pdkv_transfer_copies(plan: int, layer_begin: int, layer_end: int, stream: int = 0) -> None:
    _check(lib().pdkv_transfer_copies(C.c_void_p(plan), layer_begin, layer_end, C.c_void_p(stream)),
           "pdkv_transfer_copies")


def pdkv_sm_partition_create(device: int, transfer_sms: int) -> int:
    out = C.c_void_p()
    _check(lib().pdkv_sm_partition_create(device, transfer_sms, C.byref(out)), "pdkv_sm_partition_create")
    return out.value


def pdkv_sm_partition_info(partition: int):
    """(transfer SMs, compute SMs) as the driver rounded them."""
    a, b = C.c_int(), C.c_int()
    _check(lib().pdkv_sm_partition_info(C.c_void_p(partition), C.byref(a), C.byref(b)), "pdkv_sm_partition_info")
    return a.value, b.value


def pdkv_sm_partition_stream(partition: int, which: int) -> int:
    out = C.c_void_p()
    _check(lib().pdkv_sm_partition_stream(C.c_void_p(partition), which, C.byref(out)), "pdkv_sm_partition_stream")
    return out.value


def pdkv_sm_partition_destroy(partition: int) -> None:
    _check(lib().pdkv_sm_partition_destroy(C.c_void_p(partition)), "pdkv_sm_partition_destroy")


def pdkv_transfer_blockwise(plan: int, stream: int = 0) -> None:
    _check(lib().pdkv_transfer_blockwise(C.c_void_p(plan), C.c_void_p(stream)),
           "pdkv_transfer_blockwise")


def pdkv_plan_launches(plan: int, op: int) -> int:
    n = C.c_int64()
    _check(lib().pdkv_plan_launches(C.c_void_p(plan), op, C.byref(n)), "pdkv_plan_launches")
    return int(n.value)


def pdkv_plan_tiles(plan: int, op: int) -> np.ndarray:
    """Copy of the plan's tile list as a structured numpy array."""
    p = C.POINTER(pdkv_tile)()
    n = C.c_int64()
    _check(lib().pdkv_plan_tiles(C.c_void_p(plan), op, C.byref(p), C.byref(n)), "pdkv_plan_tiles")
    if n.value == 0:
        return np.zeros(0, TILE_DTYPE)
    raw = C.string_at(p, n.value * C.sizeof(pdkv_tile))
    return np.frombuffer(raw, TILE_DTYPE).copy()


def pdkv_plan_status(plan: int, stream: int = 0) -> None:
    _check(lib().pdkv_plan_status(C.c_void_p(plan), C.c_void_p(stream)), "pdkv_plan_status")


def pdkv_upload_blocks(plan: int, host_src_ptr: int, stream: int = 0) -> None:
    _check(lib().pdkv_upload_blocks(C.c_void_p(plan), C.c_void_p(host_src_ptr), C.c_void_p(stream)),
           "pdkv_upload_blocks")


def pdkv_download_blocks(plan: int, host_dst_ptr: int, stream: int = 0) -> None:
    _check(lib().pdkv_download_blocks(C.c_void_p(plan), C.c_void_p(host_dst_ptr), C.c_void_p(stream)),
           "pdkv_download_blocks")


def pdkv_plan_block_bytes(plan: int):
    """(bytes pdkv_upload_blocks copies, bytes pdkv_download_blocks copies)."""
    a, b = C.c_uint64(), C.c_uint64()
    _check(lib().pdkv_plan_block_bytes(C.c_void_p(plan), C.byref(a), C.byref(b)), "pdkv_plan_block_bytes")
    return int(a.value), int(b.value)


def pdkv_queue_create(src_pool: int, dst_pool: int, device: int, capacity: int) -> int:
    out = C.c_void_p()
    _check(lib().pdkv_queue_create(C.c_void_p(src_pool), C.c_void_p(dst_pool), device, capacity,
                                   C.byref(out)), "pdkv_queue_create")
    return out.value


def pdkv_queue_submit(queue: int, seq_len, src_tbl_off, src_tbl, dst_tbl_off, dst_tbl, dst_skip=None,
                      host_src_ptr: Optional[int] = None, host_dst_ptr: Optional[int] = None,
                      wait_event: Optional[int] = None):
    """Returns a ticket, or ``None`` when every receive slot is taken.  ``wait_event`` is a
    ``cudaEvent_t`` handle (e.g. ``torch.cuda.Event.cuda_event``) the slot's stream waits for."""
    b = _BatchArrays(seq_len, src_tbl_off, src_tbl, dst_tbl_off, dst_tbl, dst_skip)
    t = C.c_int64()
    rc = lib().pdkv_queue_submit(C.c_void_p(queue), C.byref(b.desc), C.c_void_p(host_src_ptr),
                                 C.c_void_p(host_dst_ptr), C.c_void_p(wait_event), C.byref(t))
    if rc == PDKV_ERR_BUSY:
        return None
    _check(rc, "pdkv_queue_submit")
    return int(t.value)


def pdkv_queue_poll(queue: int, ticket: int) -> bool:
    d = C.c_int()
    _check(lib().pdkv_queue_poll(C.c_void_p(queue), ticket, C.byref(d)), "pdkv_queue_poll")
    return bool(d.value)


def pdkv_queue_wait(queue: int, ticket: int) -> None:
    _check(lib().pdkv_queue_wait(C.c_void_p(queue), ticket), "pdkv_queue_wait")


def pdkv_queue_release(queue: int, ticket: int) -> None:
    _check(lib().pdkv_queue_release(C.c_void_p(queue), ticket), "pdkv_queue_release")


def pdkv_queue_stats(queue: int):
    """(capacity, in_use, submitted, rejected)."""
    cap, use, sub, rej = C.c_int(), C.c_int(), C.c_int64(), C.c_int64()
    _check(lib().pdkv_queue_stats(C.c_void_p(queue), C.byref(cap), C.byref(use), C.byref(sub),
                                  C.byref(rej)), "pdkv_queue_stats")
    return cap.value, use.value, int(sub.value), int(rej.value)


def pdkv_queue_destroy(queue: int) -> None:
    _check(lib().pdkv_queue_destroy(C.c_void_p(queue)), "pdkv_queue_destroy")


def pdkv_tune(key: str, value: int) -> None:
    _check(lib().pdkv_tune(key.encode(), value), f"pdkv_tune({key})")


def pdkv_tune_get(key: str) -> int:
    v = C.c_int64()
    _check(lib().pdkv_tune_get(key.encode(), C.byref(v)), f"pdkv_tune_get({key})")
    return int(v.value)
