"""Prefill-to-decode transfer between two ranks (one process per GPU).

The sender rank holds the prefill pool, the receiver rank the decode pool
(Sec. 3.5 of the paper; device i of the prefill instance talks only to device i
of the decode instance, so there is no collective, just one pair):

1. *meta exchange* -- the one low-cost exchange that precedes a transfer: the
   receiver tells the sender its block size and which entries of its tables
   are already resident (shared prefixes are not sent), the sender tells the
   receiver the prompt lengths.  After it both sides compute the same buffer
   layout on their own.
2. the sender packs its discrete blocks into the contiguous buffer
   (``pdkv_pack`` through a pack-only plan);
3. the bytes cross *as a whole*: one ``send`` / ``recv`` of the buffer (NCCL
   point-to-point over NVLink between GPUs; gloo between CPU processes in the
   tests).  ``chunk_bytes`` > 0 sends the same bytes in pieces instead -- with
   the size of one prefill block this is the block-by-block transfer the paper
   argues against, kept for comparison;
4. the receiver restores its discrete blocks from the bytes (``pdkv_unpack``
   through an unpack-only plan).

Per-layer trigger (the paper's second mode, same buffer format): with
``layers_per_stage`` > 0 the transfer runs as a pipeline over layer ranges.  The
sender packs layers ``[l, l+k)`` and hands them to the transport while it
already packs the next range; the receiver posts all receives up front and
restores a range as soon as it has arrived, while later ranges are still on the
link.  A layer range of request r is the byte range
``[off_r + l*per_r, off_r + (l+k)*per_r)`` with ``per_r = (off_{r+1} - off_r) / L``
of the contiguous buffer -- an offset and a length, as in Sec. 3.5 -- so a stage
travels as one message per request with kept tokens, issued as one batch of
point-to-point operations.  Nothing else changes: same meta exchange, same
plans, same kernels.

This module only moves metadata and calls ``torch.distributed``; packing and
unpacking are done by whatever the two factories return (on a GPU:
:class:`~paper_2408_08147_b200.session.TransferSession`, i.e. the library's
kernels).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, Optional

import numpy as np


@dataclass
class SenderMeta:
    """What the sender learns from the receiver."""
    skip_granule_tokens: int          # the decode pool's block size
    dst_tbl_off: np.ndarray           # [n_req + 1] int64: where each request's mask entries start
    dst_skip: Optional[np.ndarray]    # uint8 per decode-table entry, None = nothing resident


def _dist():
    import torch.distributed as dist

    return dist


def _send_array(a: np.ndarray, peer: int, device, group) -> None:
    import torch

    t = torch.from_numpy(np.ascontiguousarray(a, np.int64)).to(device)
    _dist().send(t, dst=peer, group=group)


def _recv_array(n: int, peer: int, device, group) -> np.ndarray:
    import torch

    t = torch.empty(n, dtype=torch.int64, device=device)
    _dist().recv(t, src=peer, group=group)
    return t.cpu().numpy()


def _pieces(total: int, chunk_bytes: int):
    if chunk_bytes <= 0 or chunk_bytes >= total:
        return [(0, total)] if total else []
    return [(a, min(total, a + chunk_bytes)) for a in range(0, total, chunk_bytes)]


def layer_stages(num_layers: int, layers_per_stage: int):
    """Layer ranges ``[(l0, l1), ...]`` of the pipeline, in order."""
    k = max(1, int(layers_per_stage))
    return [(l, min(num_layers, l + k)) for l in range(0, num_layers, k)]


def stage_pieces(req_off, num_layers: int, l0: int, l1: int):
    """Byte ranges of layers ``[l0, l1)`` in the contiguous buffer: one ``(begin, end)`` per
    request that has kept tokens, neighbours merged (a whole-model range is one piece)."""
    out = []
    for r in range(len(req_off) - 1):
        per = (int(req_off[r + 1]) - int(req_off[r])) // num_layers
        a, z = int(req_off[r]) + l0 * per, int(req_off[r]) + l1 * per
        if z <= a:
            continue
        if out and out[-1][1] == a:
            out[-1] = (out[-1][0], z)
        else:
            out.append((a, z))
    return out


def _post(kind, buf, pieces, peer, group):
    """One batch of point-to-point operations for the pieces of a stage; returns its work handles."""
    dist = _dist()
    if not pieces:
        return []
    fn = dist.isend if kind == "send" else dist.irecv
    return dist.batch_isend_irecv([dist.P2POp(fn, buf[a:z], peer, group) for a, z in pieces])


def _host_visible(buf) -> bool:
    return not getattr(buf, "is_cuda", False)


def send_kv(seq_len: np.ndarray, make_sender: Callable[[SenderMeta], object],
            new_buffer: Callable[[int], object], peer: int, *, device="cpu", group=None,
            chunk_bytes: int = 0, layers_per_stage: int = 0):
    """Sender side.  ``make_sender(meta)`` returns an object with ``buffer_bytes``
    and ``pack(buf)`` (a pack-only session built from the prefill tables, the
    prompt lengths and the receiver's mask); ``new_buffer(n)`` returns a flat
    uint8 tensor of n bytes on the sender's device.  Returns (bytes sent, the
    sender object, the buffer): the caller keeps both alive until the stream has
    finished with them, then closes the session."""
    n_req = int(len(seq_len))
    head = _recv_array(2, peer, device, group)                 # [block size, number of mask entries or -1]
    G, n_mask = int(head[0]), int(head[1])
    off = _recv_array(n_req + 1, peer, device, group)
    skip = None
    if n_mask >= 0:
        skip = _recv_array(n_mask, peer, device, group).astype(np.uint8)
    _send_array(np.asarray(seq_len, np.int64), peer, device, group)

    sender = make_sender(SenderMeta(G, off.astype(np.int64), skip))
    total = int(sender.buffer_bytes)
    buf = new_buffer(max(total, 16))
    if layers_per_stage > 0:
        # pipeline over layer ranges: pack range s, hand it to the transport, pack range s+1 meanwhile
        L = int(sender.num_layers)
        works = []
        for l0, l1 in layer_stages(L, layers_per_stage):
            sender.pack(buf, (l0, l1))
            if _host_visible(buf):              # the transport reads host memory: the kernel must have finished
                done = getattr(sender, "synchronize", None)
                if done:
                    done()
            works += _post("send", buf, stage_pieces(sender.request_offsets, L, l0, l1), peer, group)
        for wk in works:                        # NCCL: orders the current stream after the sends; gloo: blocks
            wk.wait()
        return total, sender, buf
    sender.pack(buf)
    if not getattr(buf, "is_cuda", False):      # a host buffer (pinned, written by the kernel over PCIe):
        done = getattr(sender, "synchronize", None)   # the transport reads it from the CPU, so wait for the kernel
        if done:
            done()
    for a, z in _pieces(total, chunk_bytes):
        _dist().send(buf[a:z], dst=peer, group=group)
    return total, sender, buf


def recv_kv(dst_tbl_off: np.ndarray, dst_skip: Optional[np.ndarray], skip_granule_tokens: int,
            make_receiver: Callable[[np.ndarray], object], new_buffer: Callable[[int], object],
            peer: int, *, device="cpu", group=None, chunk_bytes: int = 0, layers_per_stage: int = 0):
    """Receiver side.  ``make_receiver(seq_len)`` returns an object with
    ``buffer_bytes`` and ``unpack(buf)`` (an unpack-only session built from the
    decode tables, the mask and the sender's prompt lengths).  ``chunk_bytes``
    and ``layers_per_stage`` must equal the sender's.  Returns (bytes received, the receiver object, the
    buffer); the decode blocks are valid once the receiver's stream has passed
    the unpack, and only then may the session be closed and the buffer reused."""
    n_req = int(len(dst_tbl_off)) - 1
    n_mask = -1 if dst_skip is None else int(len(dst_skip))
    _send_array(np.array([skip_granule_tokens, n_mask], np.int64), peer, device, group)
    _send_array(np.asarray(dst_tbl_off, np.int64), peer, device, group)
    if dst_skip is not None:
        _send_array(np.asarray(dst_skip, np.int64), peer, device, group)
    seq_len = _recv_array(n_req, peer, device, group).astype(np.int32)

    receiver = make_receiver(seq_len)
    total = int(receiver.buffer_bytes)
    buf = new_buffer(max(total, 16))
    if layers_per_stage > 0:
        # every receive is posted before the first unpack, so that the link never waits for a kernel
        L = int(receiver.num_layers)
        stages = layer_stages(L, layers_per_stage)
        posted = [_post("recv", buf, stage_pieces(receiver.request_offsets, L, l0, l1), peer, group)
                  for l0, l1 in stages]
        for (l0, l1), works in zip(stages, posted):
            for wk in works:
                wk.wait()
            receiver.unpack(buf, (l0, l1))      # restores this range while later ranges are still arriving
        return total, receiver, buf
    for a, z in _pieces(total, chunk_bytes):
        _dist().recv(buf[a:z], src=peer, group=group)
    receiver.unpack(buf)
    return total, receiver, buf


# ---------------------------------------------------------------------------
# GPU factories: the library's sessions on torch's current stream, so that
# pack -> send and recv -> unpack are ordered by the stream itself
# ---------------------------------------------------------------------------

def gpu_sender(src_geom, src_t, src_tbl_off, src_tbl, seq_len):
    """``make_sender`` for a prefill pool held in the flat CUDA tensor ``src_t``."""
    import torch

    from . import workloads as W
    from .session import TransferSession

    def make(meta: SenderMeta):
        batch = W.Batch(np.asarray(seq_len, np.int32), src_tbl_off, src_tbl, meta.dst_tbl_off,
                        np.zeros(0, np.int32), meta.dst_skip)
        return TransferSession(src_geom, src_t, None, None, batch, torch.cuda.current_stream().cuda_stream,
                               skip_granule_tokens=meta.skip_granule_tokens)

    return make


def gpu_receiver(dst_geom, dst_t, dst_tbl_off, dst_tbl, dst_skip):
    """``make_receiver`` for a decode pool held in the flat CUDA tensor ``dst_t``."""
    import torch

    from . import workloads as W
    from .session import TransferSession

    def make(seq_len: np.ndarray):
        z64, z32 = np.zeros(len(seq_len) + 1, np.int64), np.zeros(0, np.int32)
        batch = W.Batch(np.asarray(seq_len, np.int32), z64, z32, dst_tbl_off, dst_tbl, dst_skip)
        return TransferSession(None, None, dst_geom, dst_t, batch, torch.cuda.current_stream().cuda_stream)

    return make


def gpu_buffer(device):
    import torch

    return lambda n: torch.empty(n, dtype=torch.uint8, device=device)
