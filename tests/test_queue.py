"""Asynchronous retrieval queue (Sec. 3.5): admission into a small fixed set of
receive slots, completion polling, slot hand-over.  The admission logic runs on
CPU (dry-run plans); the GPU test drives real transfers through the slots and
compares the decode pool with the checker."""
import numpy as np
import pytest

from paper_2408_08147_b200 import binding as B
from paper_2408_08147_b200 import build as pdkv_build
from paper_2408_08147_b200 import workloads as W

FAKE = 0x7F0000000000


def _submit(q, b, **kw):
    return B.pdkv_queue_submit(q, b.seq_len, b.src_tbl_off, b.src_tbl, b.dst_tbl_off, b.dst_tbl, b.dst_skip, **kw)


def test_admission_and_slot_handover_on_cpu():
    pdkv_build.build_library()
    B.pdkv_tune("dry_run", 1)
    try:
        w = W.make_config(1)
        ps = B.pdkv_pool_create(B.desc_of(w.src), FAKE, w.src.num_bytes(), 0)
        pd = B.pdkv_pool_create(B.desc_of(w.dst), FAKE + (1 << 40), w.dst.num_bytes(), 0)
        with pytest.raises(B.PdkvError):
            B.pdkv_queue_create(ps, pd, 0, 0)
        q = B.pdkv_queue_create(ps, pd, 0, 2)
        parts = [W.slice_batch(w.batch, i, i + 2) for i in range(0, 8, 2)]
        t0, t1 = _submit(q, parts[0]), _submit(q, parts[1])
        assert t0 is not None and t1 is not None and t0 != t1
        assert _submit(q, parts[2]) is None                       # both slots taken: refused at once
        assert B.pdkv_queue_stats(q) == (2, 2, 2, 1)
        assert B.pdkv_queue_poll(q, t0)
        B.pdkv_queue_release(q, t0)                               # a completed request frees its slot
        t2 = _submit(q, parts[2])
        assert t2 is not None and t2 not in (t0, t1)
        with pytest.raises(B.PdkvError) as e:
            B.pdkv_queue_release(q, t0)                           # stale ticket
        assert e.value.status == B.PDKV_ERR_INVALID_ARG
        with pytest.raises(B.PdkvError):
            B.pdkv_queue_poll(q, 12345)
        # an invalid batch is rejected and does not consume a slot
        B.pdkv_queue_release(q, t1)
        bad = W.slice_batch(w.batch, 6, 8)
        bad.dst_tbl[0] = w.dst.num_blocks
        with pytest.raises(B.PdkvError) as e:
            _submit(q, bad)
        assert e.value.status == B.PDKV_ERR_TABLE
        assert B.pdkv_queue_stats(q)[1] == 1
        B.pdkv_queue_destroy(q)
        B.pdkv_pool_destroy(ps); B.pdkv_pool_destroy(pd)
    finally:
        B.pdkv_tune("dry_run", 0)


@pytest.mark.gpu
@pytest.mark.parametrize("host_pools", [False, True])
def test_queue_transfers_match_the_checker(oracle, host_pools):
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    B.pdkv_tune("dry_run", 0)
    w = W.make_config(3, num_layers=2, n_req=12, max_len=1200)
    src = W.fill_pool_numpy(w.src, w.seed)
    sent = W.sentinel_pool_numpy(w.dst)
    want = sent.copy()
    oracle.transfer(w.src, src, w.dst, want, w.batch)

    def dev(a):
        return torch.from_numpy(a.view(np.uint8).copy()).cuda()

    if host_pools:
        h_src = torch.from_numpy(src.view(np.uint8).copy()).pin_memory()
        h_dst = torch.from_numpy(sent.view(np.uint8).copy()).pin_memory()
        src_t = torch.zeros(w.src.num_bytes(), dtype=torch.uint8, device="cuda")
        kw = dict(host_src_ptr=h_src.data_ptr(), host_dst_ptr=h_dst.data_ptr())
    else:
        src_t, kw = dev(src), {}
    dst_t = dev(sent)
    torch.cuda.synchronize()
    ps = B.pdkv_pool_create(B.desc_of(w.src), src_t.data_ptr(), src_t.numel(), 0)
    pd = B.pdkv_pool_create(B.desc_of(w.dst), dst_t.data_ptr(), dst_t.numel(), 0)
    q = B.pdkv_queue_create(ps, pd, 0, 3)
    pending, parts = [], [W.slice_batch(w.batch, i, i + 2) for i in range(0, 12, 2)]
    busy_seen = 0
    for part in parts:
        t = _submit(q, part, **kw)
        while t is None:                       # on demand: a finished transfer frees a slot
            busy_seen += 1
            B.pdkv_queue_wait(q, pending[0])
            assert B.pdkv_queue_poll(q, pending[0])
            B.pdkv_queue_release(q, pending.pop(0))
            t = _submit(q, part, **kw)
        pending.append(t)
    for t in pending:
        B.pdkv_queue_release(q, t)             # waits for the transfer if it still runs
    cap, used, sub, rej = B.pdkv_queue_stats(q)
    assert (cap, used, sub) == (3, 0, 6) and rej == busy_seen and busy_seen >= 1
    B.pdkv_queue_destroy(q)
    torch.cuda.synchronize()
    got = h_dst.numpy().view(np.uint16) if host_pools else dst_t.cpu().numpy().view(np.uint16)
    assert np.array_equal(got, want)
    B.pdkv_pool_destroy(ps); B.pdkv_pool_destroy(pd)


@pytest.mark.gpu
def test_submit_waits_for_the_producer_of_the_blocks(oracle):
    """The slot streams run beside the caller's streams.  Here the prefill pool is written on
    another stream, behind a long-running kernel, and nothing synchronises on the host before
    the submit: only the event handed to pdkv_queue_submit orders the transfer after it."""
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    B.pdkv_tune("dry_run", 0)
    w = W.make_config(3, num_layers=2, n_req=6, max_len=800)
    src = W.fill_pool_numpy(w.src, w.seed)
    sent = W.sentinel_pool_numpy(w.dst)
    want = sent.copy()
    oracle.transfer(w.src, src, w.dst, want, w.batch)
    staged = torch.from_numpy(src.view(np.uint8).copy()).cuda()       # the values the producer will write
    src_t = torch.zeros_like(staged)                                   # the pool starts out stale
    dst_t = torch.from_numpy(sent.view(np.uint8).copy()).cuda()
    ballast = torch.empty(1 << 28, dtype=torch.float32, device="cuda")
    ps = B.pdkv_pool_create(B.desc_of(w.src), src_t.data_ptr(), src_t.numel(), 0)
    pd = B.pdkv_pool_create(B.desc_of(w.dst), dst_t.data_ptr(), dst_t.numel(), 0)
    q = B.pdkv_queue_create(ps, pd, 0, 1)
    producer = torch.cuda.Stream()
    ready = torch.cuda.Event()
    torch.cuda.synchronize()
    with torch.cuda.stream(producer):
        for _ in range(20):                    # some milliseconds of work ahead of the pool's fill
            ballast.normal_()
        src_t.copy_(staged)
        ready.record(producer)
    t = _submit(q, w.batch, wait_event=ready.cuda_event)               # no host synchronisation before this
    assert t is not None
    B.pdkv_queue_wait(q, t)
    B.pdkv_queue_release(q, t)
    B.pdkv_queue_destroy(q)
    torch.cuda.synchronize()
    assert np.array_equal(dst_t.cpu().numpy().view(np.uint16), want)
    B.pdkv_pool_destroy(ps); B.pdkv_pool_destroy(pd)
