"""Seeded synthetic inputs for the paged-KVCache transfer path.

This module only *draws inputs*: prompt lengths, block tables, skip masks and
KV values.  It performs none of the transfer's index arithmetic, so both the
CUDA path and the CPU checker can be fed from it without sharing any of the
method's code.  The workloads imitate the shapes of Llama-class serving
batches (the production traces behind the paper's evaluation, §4 "Setup", are
not public); only tensor shapes and length distributions are imitated.

Layout names follow the pool descriptions used throughout the library:

* ``BLOCK_MAJOR``  ``[block][layer][K/V][token][head][dim]``
* ``LAYER_MAJOR``  ``[layer][K/V][block][head][token][dim]``
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Optional

import numpy as np

BLOCK_MAJOR = 0
LAYER_MAJOR = 1

BASE_SEED = 20240815

# 16-bit pattern written where the path must neither read nor write: a quiet
# NaN with a payload that rounding a normal draw to bf16 never produces.
SENTINEL_U16 = 0x7FC1

# sub-stream ids
_S_LEN, _S_OCC, _S_PERM_SRC, _S_PERM_DST, _S_SKIP, _S_VAL = range(6)


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, stream])))


@dataclass(frozen=True)
class Geometry:
    """Shape of one paged pool."""

    layout: int
    num_layers: int
    num_kv_heads: int
    head_dim: int
    elem_bytes: int
    block_tokens: int
    num_blocks: int

    def shape(self) -> tuple:
        """Logical array shape of the pool, outermost dimension first."""
        L, H, D, B, NB = (self.num_layers, self.num_kv_heads, self.head_dim,
                          self.block_tokens, self.num_blocks)
        if self.layout == BLOCK_MAJOR:
            return (NB, L, 2, B, H, D)
        return (L, 2, NB, H, B, D)

    def num_elems(self) -> int:
        n = 1
        for s in self.shape():
            n *= s
        return n

    def num_bytes(self) -> int:
        return self.num_elems() * self.elem_bytes

    def token_bytes(self) -> int:
        return 2 * self.num_layers * self.num_kv_heads * self.head_dim * self.elem_bytes


@dataclass
class Batch:
    """One transfer batch: per-request lengths, CSR block tables, skip mask."""

    seq_len: np.ndarray          # int32 [n_req]
    src_tbl_off: np.ndarray      # int64 [n_req+1]
    src_tbl: np.ndarray          # int32
    dst_tbl_off: np.ndarray      # int64 [n_req+1]
    dst_tbl: np.ndarray          # int32
    dst_skip: Optional[np.ndarray] = None   # uint8, parallel to dst_tbl

    @property
    def n_req(self) -> int:
        return int(self.seq_len.shape[0])


@dataclass
class Workload:
    name: str
    seed: int
    src: Geometry
    dst: Geometry
    batch: Batch
    note: str = ""
    src_occupied: np.ndarray = field(default_factory=lambda: np.zeros(0, np.int32))


def _blocks(n_tokens: np.ndarray, block: int) -> np.ndarray:
    return (n_tokens.astype(np.int64) + block - 1) // block


def _csr(counts: np.ndarray) -> np.ndarray:
    off = np.zeros(counts.shape[0] + 1, np.int64)
    np.cumsum(counts, out=off[1:])
    return off


def _tables(rng: np.random.Generator, counts: np.ndarray, num_blocks: int,
            occupied: Optional[np.ndarray] = None):
    """Requests take consecutive runs of a seeded permutation of the free slots."""
    free = np.arange(num_blocks, dtype=np.int32)
    if occupied is not None and occupied.size:
        mask = np.ones(num_blocks, bool)
        mask[occupied] = False
        free = free[mask]
    need = int(counts.sum())
    if need > free.shape[0]:
        raise ValueError(f"pool too small: need {need} blocks, {free.shape[0]} free")
    perm = rng.permutation(free)[:need].astype(np.int32)
    return _csr(counts), perm


def draw_lengths(kind: str, n_req: int, seed: int, **kw) -> np.ndarray:
    rng = _rng(seed, _S_LEN)
    if kind == "uniform":
        lo, hi = kw["lo"], kw["hi"]
        return rng.integers(lo, hi + 1, size=n_req).astype(np.int32)
    if kind == "fixed":
        return np.full(n_req, kw["value"], np.int32)
    if kind == "lognormal":
        z = rng.standard_normal(n_req)
        v = np.rint(np.exp(np.log(kw["median"]) + kw["sigma"] * z))
        return np.clip(v, kw["lo"], kw["hi"]).astype(np.int32)
    raise ValueError(kind)


def build_workload(name: str, seed: int, *, num_layers: int, num_kv_heads: int,
                   head_dim: int, elem_bytes: int, seq_len: np.ndarray,
                   src_layout: int, src_block: int, dst_layout: int, dst_block: int,
                   src_slack: float = 1.0, dst_slack: float = 1.0,
                   src_occupied_frac: float = 0.0, skip_frac: float = 0.0,
                   note: str = "") -> Workload:
    """Assemble pools, tables and skip mask around a drawn length vector.

    ``*_slack`` scales the pool size over the blocks the batch needs;
    ``src_occupied_frac`` marks that share of the prefill pool as held by other
    requests (a fragmented free list); ``skip_frac`` marks about that share of
    each request's *leading* decode blocks as already resident (stochastic
    rounding per request).
    """
    seq_len = np.asarray(seq_len, np.int32)
    n_src = _blocks(seq_len, src_block)
    n_dst = _blocks(seq_len, dst_block)
    need_src, need_dst = int(n_src.sum()), int(n_dst.sum())

    occupied = np.zeros(0, np.int32)
    if src_occupied_frac > 0.0:
        nb_src = int(np.ceil(need_src / (1.0 - src_occupied_frac)))
        n_occ = int(np.floor(src_occupied_frac * nb_src))
        occupied = np.sort(_rng(seed, _S_OCC).permutation(nb_src)[:n_occ]).astype(np.int32)
    else:
        nb_src = max(1, int(np.ceil(src_slack * need_src)))
    nb_dst = max(1, int(np.ceil(dst_slack * need_dst)))

    src_off, src_tbl = _tables(_rng(seed, _S_PERM_SRC), n_src, nb_src, occupied)
    dst_off, dst_tbl = _tables(_rng(seed, _S_PERM_DST), n_dst, nb_dst)

    skip = None
    if skip_frac > 0.0:
        u = _rng(seed, _S_SKIP).random(seq_len.shape[0])
        k = np.floor(skip_frac * n_dst + u).astype(np.int64)
        k = np.minimum(k, n_dst)
        skip = np.zeros(dst_tbl.shape[0], np.uint8)
        for r in range(seq_len.shape[0]):
            skip[dst_off[r]:dst_off[r] + k[r]] = 1

    src = Geometry(src_layout, num_layers, num_kv_heads, head_dim, elem_bytes, src_block, nb_src)
    dst = Geometry(dst_layout, num_layers, num_kv_heads, head_dim, elem_bytes, dst_block, nb_dst)
    return Workload(name, seed, src, dst,
                    Batch(seq_len, src_off, src_tbl, dst_off, dst_tbl, skip),
                    note=note, src_occupied=occupied)


def make_config(idx: int, *, num_layers: Optional[int] = None, n_req: Optional[int] = None,
                src_block: Optional[int] = None, src_layout: Optional[int] = None,
                dst_layout: Optional[int] = None, max_len: Optional[int] = None,
                elem_bytes: Optional[int] = None, num_kv_heads: Optional[int] = None,
                head_dim: Optional[int] = None) -> Workload:
    """The five benchmark workloads (idx 1..5); keyword overrides shrink them.

    1 tiny; 2 8B-shaped uniform, same layout both sides; 3 8B-shaped lognormal
    lengths with re-blocking 16 -> 128; 4 70B-shaped, fragmented prefill pool;
    5 many small requests with resident shared-prefix decode blocks skipped.
    """
    seed = BASE_SEED + idx
    if idx == 1:
        n = n_req or 8
        lens = draw_lengths("uniform", n, seed, lo=1, hi=max_len or 300)
        return build_workload("tiny", seed, num_layers=num_layers or 2, num_kv_heads=num_kv_heads or 4,
                              head_dim=head_dim or 64, elem_bytes=elem_bytes or 2, seq_len=lens,
                              src_layout=BLOCK_MAJOR if src_layout is None else src_layout,
                              src_block=src_block or 16,
                              dst_layout=LAYER_MAJOR if dst_layout is None else dst_layout,
                              dst_block=32, src_slack=1.25, dst_slack=1.25)
    if idx == 2:
        n = n_req or 32
        lens = draw_lengths("fixed", n, seed, value=max_len or 2048)
        lay = BLOCK_MAJOR if src_layout is None else src_layout
        return build_workload("llama3-8b-uniform", seed, num_layers=num_layers or 32,
                              num_kv_heads=num_kv_heads or 8, head_dim=head_dim or 128, elem_bytes=elem_bytes or 2,
                              seq_len=lens,
                              src_layout=lay, src_block=src_block or 128,
                              dst_layout=lay if dst_layout is None else dst_layout,
                              dst_block=128)
    if idx == 3:
        n = n_req or 64
        lens = draw_lengths("lognormal", n, seed, median=1024, sigma=0.8, lo=16,
                            hi=max_len or 8192)
        return build_workload("llama3-8b-lognormal-reblock", seed,
                              num_layers=num_layers or 32, num_kv_heads=num_kv_heads or 8,
                              head_dim=head_dim or 128, elem_bytes=elem_bytes or 2, seq_len=lens,
                              src_layout=BLOCK_MAJOR if src_layout is None else src_layout,
                              src_block=src_block or 16,
                              dst_layout=LAYER_MAJOR if dst_layout is None else dst_layout,
                              dst_block=128)
    if idx == 4:
        n = n_req or 16
        lens = draw_lengths("fixed", n, seed, value=max_len or 4096)
        return build_workload("llama3-70b-fragmented", seed, num_layers=num_layers or 80,
                              num_kv_heads=num_kv_heads or 8, head_dim=head_dim or 128, elem_bytes=elem_bytes or 2,
                              seq_len=lens,
                              src_layout=BLOCK_MAJOR if src_layout is None else src_layout,
                              src_block=src_block or 64,
                              dst_layout=LAYER_MAJOR if dst_layout is None else dst_layout,
                              dst_block=128, src_occupied_frac=0.3)
    if idx == 5:
        n = n_req or 1024
        lens = draw_lengths("uniform", n, seed, lo=64, hi=max_len or 512)
        return build_workload("tidal-small-requests", seed, num_layers=num_layers or 32,
                              num_kv_heads=num_kv_heads or 8, head_dim=head_dim or 128, elem_bytes=elem_bytes or 2,
                              seq_len=lens,
                              src_layout=BLOCK_MAJOR if src_layout is None else src_layout,
                              src_block=src_block or 16,
                              dst_layout=LAYER_MAJOR if dst_layout is None else dst_layout,
                              dst_block=128, skip_frac=0.25)
    raise ValueError(f"no config {idx}")


def with_dst_geometry_of_src(w: Workload) -> Workload:
    """Same batch, but the decode side mirrors the prefill pool and its table."""
    b = replace(w.batch, dst_tbl_off=w.batch.src_tbl_off.copy(),
                dst_tbl=w.batch.src_tbl.copy(), dst_skip=None)
    return replace(w, dst=w.src, batch=b)


# ---------------------------------------------------------------------------
# values
# ---------------------------------------------------------------------------

def normal_bf16_bits(n: int, seed: int) -> np.ndarray:
    """n draws of N(0,1) rounded to bf16 (round-to-nearest-even), as uint16 bits."""
    f = _rng(seed, _S_VAL).standard_normal(n, dtype=np.float32)
    u = f.view(np.uint32)
    u = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return u.astype(np.uint16)


def fill_pool_numpy(geom: Geometry, seed: int) -> np.ndarray:
    """A host pool filled with seeded values, as a flat array of raw elements."""
    n = geom.num_elems()
    if geom.elem_bytes == 2:
        return normal_bf16_bits(n, seed)
    rng = _rng(seed, _S_VAL)
    dt = {1: np.uint8, 4: np.uint32, 8: np.uint64}[geom.elem_bytes]
    return rng.integers(0, np.iinfo(dt).max, size=n, dtype=dt, endpoint=True)


def sentinel_pool_numpy(geom: Geometry) -> np.ndarray:
    dt = {1: np.uint8, 2: np.uint16, 4: np.uint32, 8: np.uint64}[geom.elem_bytes]
    val = {1: 0xA5, 2: SENTINEL_U16, 4: 0x7FC1A5A5, 8: 0x7FF8A5A5A5A5A5A5}[geom.elem_bytes]
    return np.full(geom.num_elems(), val, dt)


def fill_pool_torch(pool, seed: int) -> None:
    """Fill a device pool (a flat torch int16/uint16-compatible tensor) in place.

    Values are N(0,1) in bf16 drawn by torch's generator on the pool's device;
    the same bytes are later copied to the host for the CPU checker, so the two
    sides never need to regenerate them.
    """
    import torch

    g = torch.Generator(device=pool.device)
    g.manual_seed(seed)
    pool.view(torch.bfloat16).normal_(generator=g)


# ---------------------------------------------------------------------------
# sub-problems: a few requests of a large batch with their blocks renumbered
# ---------------------------------------------------------------------------

def compact_subproblem(w: Workload, req_ids):
    """Requests ``req_ids`` of ``w`` as a self-contained workload.

    Block ids are renumbered 0..k-1 in order of first appearance, so the pools
    of the sub-problem hold just the gathered blocks.  Returns the new workload
    and the original prefill / decode block ids in compact order; pair it with
    :func:`gather_blocks` to build the compact pools.  Only bookkeeping happens
    here (no element of KV is touched).
    """
    b = w.batch
    req_ids = [int(r) for r in req_ids]

    def renumber(off, tbl):
        ids, new_tbl, counts, seen = [], [], [], {}
        for r in req_ids:
            ent = tbl[off[r]:off[r + 1]]
            counts.append(len(ent))
            for e in ent:
                e = int(e)
                if e not in seen:
                    seen[e] = len(ids)
                    ids.append(e)
                new_tbl.append(seen[e])
        return (_csr(np.asarray(counts, np.int64)), np.asarray(new_tbl, np.int32),
                np.asarray(ids, np.int64))

    s_off, s_tbl, s_ids = renumber(b.src_tbl_off, b.src_tbl)
    d_off, d_tbl, d_ids = renumber(b.dst_tbl_off, b.dst_tbl)
    skip = None
    if b.dst_skip is not None:
        skip = np.concatenate([b.dst_skip[b.dst_tbl_off[r]:b.dst_tbl_off[r + 1]] for r in req_ids]
                              or [np.zeros(0, np.uint8)]).astype(np.uint8)
    nb = Batch(b.seq_len[req_ids].astype(np.int32), s_off, s_tbl, d_off, d_tbl, skip)
    src = replace(w.src, num_blocks=max(1, len(s_ids)))
    dst = replace(w.dst, num_blocks=max(1, len(d_ids)))
    return Workload(w.name + "-sub", w.seed, src, dst, nb, note=w.note), s_ids, d_ids


def gather_blocks(pool, geom: Geometry, ids):
    """Blocks ``ids`` of a flat pool (torch tensor or numpy array of raw
    elements) as a new flat compact pool, through a reshaped view."""
    n = len(ids)
    if n == 0:
        shape = replace(geom, num_blocks=1).shape()
        return pool[:0].new_zeros(int(np.prod(shape))) if hasattr(pool, "new_zeros") \
            else np.zeros(int(np.prod(shape)), pool.dtype)
    v = pool.reshape(geom.shape())
    if hasattr(pool, "new_zeros"):
        import torch

        idx = torch.as_tensor(np.asarray(ids, np.int64), device=pool.device)
        out = v[idx] if geom.layout == BLOCK_MAJOR else v[:, :, idx]
        return out.contiguous().reshape(-1)
    idx = np.asarray(ids, np.int64)
    out = v[idx] if geom.layout == BLOCK_MAJOR else v[:, :, idx]
    return np.ascontiguousarray(out).reshape(-1)


def slice_batch(b: Batch, r0: int, r1: int) -> Batch:
    """Requests [r0, r1) of a batch as a batch of their own (same block ids)."""
    def cut(off, tbl):
        return (off[r0:r1 + 1] - off[r0]).astype(np.int64), tbl[off[r0]:off[r1]].copy()

    s_off, s_tbl = cut(b.src_tbl_off, b.src_tbl)
    d_off, d_tbl = cut(b.dst_tbl_off, b.dst_tbl)
    skip = None if b.dst_skip is None else b.dst_skip[b.dst_tbl_off[r0]:b.dst_tbl_off[r1]].copy()
    return Batch(b.seq_len[r0:r1].copy(), s_off, s_tbl, d_off, d_tbl, skip)
