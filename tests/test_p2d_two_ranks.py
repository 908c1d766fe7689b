"""The two-rank prefill-to-decode protocol on CPU: two gloo processes, the sender
holding only the prefill pool and its tables, the receiver only the decode pool,
its tables and its resident-block mask.  The meta exchange, the library's
sender-only / receiver-only plans (host-only here: buffer sizes and offsets) and
the byte transport are the real ones; packing and unpacking are done by the CPU
checker, because there is no GPU in these processes.  The receiver's pool must
equal a single-process transfer of the same batch."""
import os
import socket
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FAKE_BASE = 0x7F0000000000  # never dereferenced: dry-run plans make no CUDA call


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, port, idx, kw, chunk_blocks, q, layers_per_stage=0):
    os.environ.update(RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    import torch
    import torch.distributed as dist

    from oracle import pdkv_oracle as O
    from paper_2408_08147_b200 import binding as B
    from paper_2408_08147_b200 import p2d
    from paper_2408_08147_b200 import workloads as W

    dist.init_process_group("gloo", rank=rank, world_size=2)
    B.pdkv_tune("dry_run", 1)
    w = W.make_config(idx, **kw)          # both ranks derive the same synthetic batch; each uses only its half
    b = w.batch
    G = w.dst.block_tokens
    chunk = chunk_blocks * w.src.num_bytes() // w.src.num_blocks
    z32 = np.zeros(0, np.int32)
    new_buffer = lambda n: torch.zeros(n, dtype=torch.uint8)

    if rank == 0:                          # sender: prefill pool, prefill tables, prompt lengths
        src = W.fill_pool_numpy(w.src, w.seed)

        class Sender:
            def __init__(self, meta):
                self.batch = W.Batch(b.seq_len, b.src_tbl_off, b.src_tbl, meta.dst_tbl_off, z32, meta.dst_skip)
                self.G = meta.skip_granule_tokens
                pool = B.pdkv_pool_create(B.desc_of(w.src), FAKE_BASE, w.src.num_bytes(), 0)
                plan = B.pdkv_plan_create(pool, None, self.G, b.seq_len, b.src_tbl_off, b.src_tbl,
                                          meta.dst_tbl_off if meta.dst_skip is not None else None, None, meta.dst_skip)
                self.buffer_bytes, self.request_offsets = B.pdkv_plan_buffer(plan, b.n_req)
                self.num_layers = w.src.num_layers
                B.pdkv_plan_destroy(plan)
                B.pdkv_pool_destroy(pool)

            def pack(self, buf, layers=None):
                assert self.buffer_bytes == O.buffer_elems(self.batch, self.G, w.src) * w.src.elem_bytes
                O.pack(w.src, src, self.batch, self.G, buf.numpy()[:self.buffer_bytes].view(np.uint16), layers=layers)

        sent, _, _ = p2d.send_kv(b.seq_len, Sender, new_buffer, peer=1, chunk_bytes=chunk,
                                 layers_per_stage=layers_per_stage)
        q.put(("sender", sent, True))
    else:                                  # receiver: decode pool, decode tables, resident-block mask
        dst = W.sentinel_pool_numpy(w.dst)

        class Receiver:
            def __init__(self, seq_len):
                assert np.array_equal(seq_len, b.seq_len)
                self.batch = W.Batch(seq_len, np.zeros(b.n_req + 1, np.int64), z32, b.dst_tbl_off, b.dst_tbl, b.dst_skip)
                pool = B.pdkv_pool_create(B.desc_of(w.dst), FAKE_BASE, w.dst.num_bytes(), 0)
                plan = B.pdkv_plan_create(None, pool, G, seq_len, None, None, b.dst_tbl_off, b.dst_tbl, b.dst_skip)
                self.buffer_bytes, self.request_offsets = B.pdkv_plan_buffer(plan, b.n_req)
                self.num_layers = w.dst.num_layers
                B.pdkv_plan_destroy(plan)
                B.pdkv_pool_destroy(pool)

            def unpack(self, buf, layers=None):
                O.unpack(w.dst, dst, self.batch, buf.numpy()[:self.buffer_bytes].view(np.uint16), layers=layers)

        # the buffer starts as sentinel bytes, so a range that is restored before it has arrived shows
        new_buffer = lambda n: torch.full((n,), 0xC1, dtype=torch.uint8)
        got, _, _ = p2d.recv_kv(b.dst_tbl_off, b.dst_skip, G, Receiver, new_buffer, peer=0, chunk_bytes=chunk,
                                layers_per_stage=layers_per_stage)
        want = W.sentinel_pool_numpy(w.dst)
        O.transfer(w.src, W.fill_pool_numpy(w.src, w.seed), w.dst, want, b)
        q.put(("receiver", got, bool(np.array_equal(dst, want))))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("idx,kw,chunk_blocks,layers_per_stage", [
    (3, dict(num_layers=2, n_req=6, max_len=700), 0, 0),   # re-blocking 16 -> 128, the buffer as a whole
    (5, dict(num_layers=2, n_req=24), 0, 0),               # resident blocks: the mask travels in the meta exchange
    (5, dict(num_layers=2, n_req=24), 1, 0),               # the same bytes, one prefill block's worth per message
    (3, dict(num_layers=5, n_req=6, max_len=700), 0, 2),   # per-layer trigger: stages of 2, 2 and 1 layers
    (5, dict(num_layers=3, n_req=24), 0, 1),               # one layer per stage; some requests are fully resident
])
def test_two_rank_transfer_equals_single_process_transfer(idx, kw, chunk_blocks, layers_per_stage):
    import torch.multiprocessing as mp

    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, port, idx, kw, chunk_blocks, q, layers_per_stage)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict()
    for _ in procs:
        who, nbytes, ok = q.get(timeout=180)
        got[who] = (nbytes, ok)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got["sender"][0] == got["receiver"][0] > 0      # both sides computed the same buffer size
    assert got["receiver"][1], "the receiver's decode pool differs from a single-process transfer"


def _gpu_worker(rank, port, idx, kw, q, layers_per_stage=0):
    os.environ.update(RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    import torch
    import torch.distributed as dist

    from oracle import pdkv_oracle as O
    from paper_2408_08147_b200 import p2d
    from paper_2408_08147_b200 import workloads as W

    dist.init_process_group("gloo", rank=rank, world_size=2)
    torch.cuda.set_device(0)
    w = W.make_config(idx, **kw)
    b = w.batch
    pinned = lambda n: torch.zeros(n, dtype=torch.uint8, pin_memory=True)   # the contiguous buffer, in host memory
    if rank == 0:
        src_t = torch.from_numpy(W.fill_pool_numpy(w.src, w.seed).view(np.uint8).copy()).cuda()
        torch.cuda.synchronize()
        sent, sess, _buf = p2d.send_kv(b.seq_len, p2d.gpu_sender(w.src, src_t, b.src_tbl_off, b.src_tbl, b.seq_len),
                                       pinned, peer=1, layers_per_stage=layers_per_stage)
        sess.synchronize()
        sess.close()
        q.put(("sender", sent, True))
    else:
        dst_t = torch.from_numpy(W.sentinel_pool_numpy(w.dst).view(np.uint8).copy()).cuda()
        torch.cuda.synchronize()
        got, sess, _buf = p2d.recv_kv(b.dst_tbl_off, b.dst_skip, w.dst.block_tokens,
                                      p2d.gpu_receiver(w.dst, dst_t, b.dst_tbl_off, b.dst_tbl, b.dst_skip), pinned, peer=0,
                                      layers_per_stage=layers_per_stage)
        sess.synchronize()
        sess.close()
        want = W.sentinel_pool_numpy(w.dst)
        O.transfer(w.src, W.fill_pool_numpy(w.src, w.seed), w.dst, want, b)
        q.put(("receiver", got, bool(np.array_equal(dst_t.cpu().numpy().view(np.uint16), want))))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.gpu
@pytest.mark.parametrize("idx,kw,layers_per_stage", [(3, dict(num_layers=2, n_req=6, max_len=700), 0),
                                                     (5, dict(num_layers=2, n_req=24), 0),
                                                     (3, dict(num_layers=5, n_req=6, max_len=700), 2),
                                                     (5, dict(num_layers=4, n_req=24), 1)])
def test_two_rank_transfer_with_the_library_kernels(idx, kw, layers_per_stage):
    """The same protocol with the library on both ends: two processes that share
    the one GPU (their kernels never wait on each other), the contiguous buffer in
    pinned host memory on each side (the kernels write / read it over PCIe) and
    gloo carrying the bytes between the processes."""
    import torch
    import torch.multiprocessing as mp

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_gpu_worker, args=(r, port, idx, kw, q, layers_per_stage)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict()
    for _ in procs:
        who, nbytes, ok = q.get(timeout=300)
        got[who] = (nbytes, ok)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got["sender"][0] == got["receiver"][0] > 0
    assert got["receiver"][1], "the receiver's decode pool differs from the checker's transfer"


def test_stage_pieces_partition_the_buffer(oracle):
    """The byte ranges a layer stage sends are exactly the layer ranges the checker's pack
    writes for those layers, and over all stages they cover the buffer once."""
    sys.path.insert(0, ROOT)
    from paper_2408_08147_b200 import p2d
    from paper_2408_08147_b200 import workloads as W

    w = W.make_config(5, num_layers=5, n_req=30)
    G, L = w.dst.block_tokens, w.src.num_layers
    E = w.src.elem_bytes
    off = oracle.request_offsets(w.batch, G, w.src) * E
    assert (oracle.kept_tokens(w.batch, G) == 0).any()          # fully resident requests send nothing
    src = W.fill_pool_numpy(w.src, w.seed)
    n = oracle.buffer_elems(w.batch, G, w.src)
    covered = np.zeros(n * E, np.int32)
    assert p2d.layer_stages(L, 2) == [(0, 2), (2, 4), (4, 5)]
    for l0, l1 in p2d.layer_stages(L, 2):
        buf = np.full(n, W.SENTINEL_U16, np.uint16)
        oracle.pack(w.src, src, w.batch, G, buf, layers=(l0, l1))
        written = np.repeat(buf != W.SENTINEL_U16, E)
        mask = np.zeros(n * E, bool)
        for a, z in p2d.stage_pieces(off, L, l0, l1):
            assert z > a
            mask[a:z] = True
            covered[a:z] += 1
        assert np.array_equal(mask, written)
    assert (covered == 1).all()
    assert p2d.stage_pieces(off, L, 0, L) == [(0, n * E)]        # a whole-model stage is one message
