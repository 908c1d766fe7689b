"""The fused transfer for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is off limits: an inference
engine that already handed every byte of HBM to its own KV block allocator, or
a latency-critical path that cannot take cudaMalloc's device-wide stall.  For
them ``pdkv_transfer_noalloc`` keeps its tile list in a fixed array inside the
library instead of a plan.  This file checks, through the C ABI, that it writes
exactly the bytes ``pdkv_transfer`` writes and exactly the bytes the CPU checker
writes (bit for bit, as all parity tests here), on two different batches back
to back so that the second call has to cope with the first call's leftovers in
the shared scratch; that a batch beyond the stated limit is refused before
anything is enqueued; and that a capturing stream is refused, because the call
stages its tile list from host memory it frees on return.

Collected last on purpose (file name): a run that stops at the first failure
has then already run every other test.
"""
import numpy as np
import pytest

from paper_2408_08147_b200 import binding as B
from paper_2408_08147_b200 import workloads as W

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.from_numpy(a.reshape(-1).view(np.uint8).copy()).cuda()


def _run_both(w, layers, stream):
    """Decode pool images after the plan-based call and after the no-allocation call."""
    src = W.fill_pool_numpy(w.src, w.seed)
    src_t = _dev(src)
    sent = W.sentinel_pool_numpy(w.dst)
    want_t, got_t = _dev(sent), _dev(sent)
    b = w.batch
    ps = B.pdkv_pool_create(B.desc_of(w.src), src_t.data_ptr(), src_t.numel(), 0)
    pd_want = B.pdkv_pool_create(B.desc_of(w.dst), want_t.data_ptr(), want_t.numel(), 0)
    pd_got = B.pdkv_pool_create(B.desc_of(w.dst), got_t.data_ptr(), got_t.numel(), 0)
    torch.cuda.synchronize()
    try:
        plan = B.pdkv_plan_create(ps, pd_want, 0, b.seq_len, b.src_tbl_off, b.src_tbl,
                                  b.dst_tbl_off, b.dst_tbl, b.dst_skip, stream)
        n_tiles = len(B.pdkv_plan_tiles(plan, B.PDKV_OP_TRANSFER))
        B.pdkv_transfer(plan, layers[0], layers[1], stream)
        B.pdkv_plan_destroy(plan)
        B.pdkv_transfer_noalloc(ps, pd_got, b.seq_len, b.src_tbl_off, b.src_tbl, b.dst_tbl_off,
                                b.dst_tbl, b.dst_skip, layers[0], layers[1], stream)
        torch.cuda.synchronize()
    finally:
        for h in (ps, pd_want, pd_got):
            B.pdkv_pool_destroy(h)
    return want_t, got_t, sent, n_tiles, src


def test_noalloc_matches_plan_based_transfer_twice_in_a_row(oracle):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    B.lib()
    B.pdkv_tune("dry_run", 0)
    B.pdkv_tune("tile_bytes", 32768)
    stream = torch.cuda.Stream()
    # call 1: many tiles, re-blocking 16 -> 128, block-major -> layer-major
    first = W.make_config(3, num_layers=2, n_req=10, max_len=1500)
    # call 2: a smaller, different batch (skip mask, other geometry) on the same scratch
    second = W.make_config(5, num_layers=3, n_req=12, src_block=32)
    tiles_seen = []
    for w, layers in ((first, (0, 2)), (second, (1, 3))):
        want_t, got_t, sent, n_tiles, src = _run_both(w, layers, stream.cuda_stream)
        tiles_seen.append(n_tiles)
        assert 0 < n_tiles <= B.PDKV_NOALLOC_MAX_TILES
        assert torch.equal(want_t, got_t)
        assert not torch.equal(got_t, _dev(sent)), "nothing was written"
        checker = sent.copy()                      # not only equal to the other entry point: equal to the checker
        oracle.transfer(w.src, src, w.dst, checker, w.batch, layers=layers)
        assert np.array_equal(got_t.cpu().numpy().view(checker.dtype), checker)
    assert tiles_seen[1] < tiles_seen[0]      # the second call left stale tiles behind it


def test_noalloc_rejects_batches_beyond_the_scratch_limit():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    B.lib()
    B.pdkv_tune("dry_run", 0)
    w = W.make_config(3, num_layers=1, n_req=48)
    assert int(w.batch.seq_len.sum()) > B.PDKV_NOALLOC_MAX_TILES
    src_t = torch.zeros(w.src.num_bytes(), dtype=torch.uint8, device="cuda")
    dst_t = _dev(W.sentinel_pool_numpy(w.dst))
    before = dst_t.clone()
    ps = B.pdkv_pool_create(B.desc_of(w.src), src_t.data_ptr(), src_t.numel(), 0)
    pd = B.pdkv_pool_create(B.desc_of(w.dst), dst_t.data_ptr(), dst_t.numel(), 0)
    b = w.batch
    B.pdkv_tune("tile_bytes", 1)              # one token per tile: more tiles than the scratch holds
    try:
        with pytest.raises(B.PdkvError) as e:
            B.pdkv_transfer_noalloc(ps, pd, b.seq_len, b.src_tbl_off, b.src_tbl, b.dst_tbl_off,
                                    b.dst_tbl, b.dst_skip, 0, 1)
        assert e.value.status == B.PDKV_ERR_LIMIT
        assert "scratch" in str(e.value)
        with pytest.raises(B.PdkvError) as e:
            B.pdkv_transfer_noalloc(ps, pd, b.seq_len, b.src_tbl_off, b.src_tbl, b.dst_tbl_off,
                                    b.dst_tbl, b.dst_skip, 0, 2)    # layer range outside the model
        assert e.value.status in (B.PDKV_ERR_INVALID_ARG, B.PDKV_ERR_LIMIT)
    finally:
        B.pdkv_tune("tile_bytes", 32768)
        B.pdkv_pool_destroy(ps)
        B.pdkv_pool_destroy(pd)
    torch.cuda.synchronize()
    assert torch.equal(dst_t, before)         # refused calls enqueue nothing


def test_noalloc_refuses_a_capturing_stream():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    B.lib()
    B.pdkv_tune("dry_run", 0)
    w = W.make_config(1)
    b = w.batch
    src_t = _dev(W.fill_pool_numpy(w.src, w.seed))
    dst_t = _dev(W.sentinel_pool_numpy(w.dst))
    before = dst_t.clone()
    ps = B.pdkv_pool_create(B.desc_of(w.src), src_t.data_ptr(), src_t.numel(), 0)
    pd = B.pdkv_pool_create(B.desc_of(w.dst), dst_t.data_ptr(), dst_t.numel(), 0)
    args = (ps, pd, b.seq_len, b.src_tbl_off, b.src_tbl, b.dst_tbl_off, b.dst_tbl, b.dst_skip, 0, w.src.num_layers)
    cap = torch.cuda.Stream()
    B.pdkv_transfer_noalloc(*args, cap.cuda_stream)       # first call on the device: set-up, outside capture
    torch.cuda.synchronize()
    dst_t.copy_(before)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    refused = None
    with torch.cuda.graph(graph, stream=cap):
        try:
            B.pdkv_transfer_noalloc(*args, torch.cuda.current_stream().cuda_stream)
        except B.PdkvError as e:
            refused = e.status
    assert refused == B.PDKV_ERR_INVALID_ARG
    graph.replay()                                        # an empty graph: nothing was recorded
    torch.cuda.synchronize()
    assert torch.equal(dst_t, before)
    B.pdkv_pool_destroy(ps)
    B.pdkv_pool_destroy(pd)
