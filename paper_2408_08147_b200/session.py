"""Convenience wrapper that keeps the C handles of one transfer batch together.

It only marshals arguments: device memory comes from torch tensors handed in by
the caller, every byte is moved by the library's kernels.
"""
from __future__ import annotations

from typing import Optional, Tuple

from . import binding as B


class TransferSession:
    """Pools + plan for one batch.

    ``src_t`` / ``dst_t`` are flat torch CUDA tensors (any 1-byte or 2-byte
    dtype) that hold the prefill and decode pools; either may be ``None`` for a
    pack-only or unpack-only session.  ``batch`` carries ``seq_len`` and the
    CSR tables as numpy arrays.
    """

    def __init__(self, src_geom, src_t, dst_geom, dst_t, batch, stream: int = 0,
                 skip_granule_tokens: int = 0, workspace_t=None):
        """``workspace_t``: optional flat torch CUDA tensor that receives the plan's
        device arrays (no cudaMalloc / cudaFree for this session); it must outlive
        the session and not be shared with another live session."""
        self.src_geom, self.dst_geom, self.batch = src_geom, dst_geom, batch
        self.src_t, self.dst_t = src_t, dst_t
        self.stream = stream
        self.src_pool = self.dst_pool = self.plan = None
        try:
            if src_t is not None:
                self.src_pool = B.pdkv_pool_create(B.desc_of(src_geom), src_t.data_ptr(),
                                                   src_t.numel() * src_t.element_size(),
                                                   src_t.device.index or 0)
            if dst_t is not None:
                self.dst_pool = B.pdkv_pool_create(B.desc_of(dst_geom), dst_t.data_ptr(),
                                                   dst_t.numel() * dst_t.element_size(),
                                                   dst_t.device.index or 0)
            tables = (batch.seq_len,
                      batch.src_tbl_off if src_t is not None else None,
                      batch.src_tbl if src_t is not None else None,
                      batch.dst_tbl_off if (dst_t is not None or batch.dst_skip is not None) else None,
                      batch.dst_tbl if dst_t is not None else None,
                      batch.dst_skip)
            if workspace_t is None:
                self.plan = B.pdkv_plan_create(self.src_pool, self.dst_pool, skip_granule_tokens, *tables,
                                               stream=stream)
            else:
                self.plan, _ = B.pdkv_plan_create_in(
                    self.src_pool, self.dst_pool, skip_granule_tokens, *tables,
                    workspace_ptr=workspace_t.data_ptr(),
                    workspace_bytes=workspace_t.numel() * workspace_t.element_size(), stream=stream)
        except Exception:
            self.close()
            raise
        self.buffer_bytes, self.request_offsets = B.pdkv_plan_buffer(self.plan, batch.n_req)
        g = src_geom if src_t is not None else dst_geom
        self.num_layers = g.num_layers

    def _layers(self, layers: Optional[Tuple[int, int]]):
        return (0, self.num_layers) if layers is None else layers

    def pack(self, buf_t, layers=None, stream: Optional[int] = None) -> None:
        l0, l1 = self._layers(layers)
        B.pdkv_pack(self.plan, buf_t.data_ptr(), buf_t.numel() * buf_t.element_size(), l0, l1,
                    self.stream if stream is None else stream)

    def unpack(self, buf_t, layers=None, stream: Optional[int] = None) -> None:
        l0, l1 = self._layers(layers)
        B.pdkv_unpack(self.plan, buf_t.data_ptr(), buf_t.numel() * buf_t.element_size(), l0, l1,
                      self.stream if stream is None else stream)

    def transfer(self, layers=None, stream: Optional[int] = None) -> None:
        l0, l1 = self._layers(layers)
        B.pdkv_transfer(self.plan, l0, l1, self.stream if stream is None else stream)

    def transfer_copies(self, layers=None, stream: Optional[int] = None) -> None:
        """The fused transfer as plain device copies (block-major pools of equal block size only)."""
        l0, l1 = self._layers(layers)
        B.pdkv_transfer_copies(self.plan, l0, l1, self.stream if stream is None else stream)

    def transfer_blockwise(self, stream: Optional[int] = None) -> None:
        B.pdkv_transfer_blockwise(self.plan, self.stream if stream is None else stream)

    def upload_blocks(self, host_src_t, stream: Optional[int] = None) -> None:
        """H2D of the prefill blocks the batch reads, from a host image of the pool."""
        B.pdkv_upload_blocks(self.plan, host_src_t.data_ptr(), self.stream if stream is None else stream)

    def download_blocks(self, host_dst_t, stream: Optional[int] = None) -> None:
        """D2H of the decode blocks the batch writes, into a host image of the pool."""
        B.pdkv_download_blocks(self.plan, host_dst_t.data_ptr(), self.stream if stream is None else stream)

    def block_bytes(self):
        return B.pdkv_plan_block_bytes(self.plan)

    def status(self, stream: Optional[int] = None) -> None:
        B.pdkv_plan_status(self.plan, self.stream if stream is None else stream)

    def autotune(self, buf_t=None, stream: Optional[int] = None):
        """Time candidate launch shapes on this batch and keep the fastest per operation
        (pack and unpack only if ``buf_t`` is given).  Returns the shapes per operation."""
        B.pdkv_plan_autotune(self.plan, buf_t.data_ptr() if buf_t is not None else 0,
                             buf_t.numel() * buf_t.element_size() if buf_t is not None else 0,
                             self.stream if stream is None else stream)
        return {op: B.pdkv_plan_shape(self.plan, op) for op in (B.PDKV_OP_PACK, B.PDKV_OP_UNPACK, B.PDKV_OP_TRANSFER)}

    def synchronize(self, stream: Optional[int] = None) -> None:
        """Wait for the session's stream (and raise if a kernel reported an error)."""
        self.status(stream)

    def traffic(self, op: int):
        return B.pdkv_plan_traffic(self.plan, op)

    def launches(self, op: int) -> int:
        return B.pdkv_plan_launches(self.plan, op)

    def close(self) -> None:
        if self.plan:
            B.pdkv_plan_destroy(self.plan)
            self.plan = None
        for name in ("src_pool", "dst_pool"):
            h = getattr(self, name)
            if h:
                B.pdkv_pool_destroy(h)
                setattr(self, name, None)

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()
