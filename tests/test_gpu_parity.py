"""GPU parity: the CUDA path, called through the C ABI, against the CPU checker,
bit for bit, on the same seeded inputs.  Sizes here finish in seconds on the
checker yet span many tiles, ragged tails, both layouts, skip masks, layer
ranges and the narrow-vector fallbacks."""
import numpy as np
import pytest

from paper_2408_08147_b200 import binding as B
from paper_2408_08147_b200 import workloads as W

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

SENT = W.SENTINEL_U16


@pytest.fixture(scope="module", autouse=True)
def _gpu_lib():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    B.lib()                      # must exist: no fallback
    B.pdkv_tune("dry_run", 0)
    B.pdkv_tune("debug_bounds", 0)
    yield
    B.pdkv_tune("debug_bounds", 0)
    B.pdkv_tune("tile_bytes", 32768)
    B.pdkv_tune("lc_fastest", 0)
    B.pdkv_tune("lc_skew", -1)
    B.pdkv_tune("lc_skew_shift", 0)
    B.pdkv_tune("variant", -1)
    B.pdkv_tune("stages", 3)
    B.pdkv_tune("src_order", -1)


def dev(a: np.ndarray):
    return torch.from_numpy(a.reshape(-1).view(np.uint8).copy()).cuda()


def host(t, dtype=np.uint16):
    return t.cpu().numpy().view(dtype)


def check_all_ops(oracle, w, *, layers=None, elem_dtype=np.uint16, side_stream=False,
                  blockwise=True, bounds=False):
    """Run pack, unpack, fused and block-by-block on the GPU and compare every
    byte (owned and untouched) with the checker."""
    from paper_2408_08147_b200.session import TransferSession

    G = w.dst.block_tokens
    src = W.fill_pool_numpy(w.src, w.seed)
    sent = W.sentinel_pool_numpy(w.dst)
    n_buf = oracle.buffer_elems(w.batch, G, w.src)
    slack = 64

    want_buf = np.full(n_buf + slack, sent[0], elem_dtype)
    oracle.pack(w.src, src, w.batch, G, want_buf, layers=layers)
    full_buf = np.zeros(n_buf + slack, elem_dtype)
    oracle.pack(w.src, src, w.batch, G, full_buf)
    want_dst = sent.copy()
    oracle.unpack(w.dst, want_dst, w.batch, full_buf, layers=layers)

    B.pdkv_tune("debug_bounds", 1 if bounds else 0)
    stream = torch.cuda.Stream() if side_stream else torch.cuda.current_stream()
    src_t, dst_t = dev(src), dev(sent)
    buf_t = dev(np.full(n_buf + slack, sent[0], elem_dtype))
    torch.cuda.synchronize()
    with TransferSession(w.src, src_t, w.dst, dst_t, w.batch, stream.cuda_stream) as s:
        assert s.buffer_bytes == n_buf * w.src.elem_bytes
        s.pack(buf_t, layers)
        s.status()
        assert np.array_equal(host(buf_t, elem_dtype), want_buf), "pack"
        assert np.array_equal(host(src_t, elem_dtype), src), "pack wrote the source pool"

        fb_t = dev(full_buf)
        torch.cuda.synchronize()
        s.unpack(fb_t, layers)
        s.status()
        assert np.array_equal(host(dst_t, elem_dtype), want_dst), "unpack"

        dst_t.copy_(dev(sent))
        torch.cuda.synchronize()
        s.transfer(layers)
        s.status()
        assert np.array_equal(host(dst_t, elem_dtype), want_dst), "fused transfer"

        if blockwise and layers is None:
            dst_t.copy_(dev(sent))
            torch.cuda.synchronize()
            s.transfer_blockwise()
            s.status()
            assert np.array_equal(host(dst_t, elem_dtype), want_dst), "block-by-block baseline"
    B.pdkv_tune("debug_bounds", 0)


def test_config1_tiny_bounds_checked_then_plain(oracle):
    w = W.make_config(1)
    check_all_ops(oracle, w, bounds=True)
    check_all_ops(oracle, w, bounds=False, side_stream=True)
    check_all_ops(oracle, w, layers=(1, 2))


@pytest.mark.parametrize("idx,kw", [
    (2, dict(num_layers=2, n_req=5, max_len=640)),                       # A->A, equal blocks
    (2, dict(num_layers=2, n_req=5, max_len=600, src_layout=W.LAYER_MAJOR)),  # B->B
    (3, dict(num_layers=2, n_req=12, max_len=1500)),                     # 16 -> 128 re-blocking
    (4, dict(num_layers=3, n_req=4, max_len=700)),                       # fragmented pool, 64 -> 128
    (5, dict(num_layers=2, n_req=40)),                                   # skip mask
    (5, dict(num_layers=2, n_req=24, src_block=256)),                    # prefill block > decode block
    (3, dict(num_layers=2, n_req=6, max_len=900, src_layout=W.LAYER_MAJOR,
             dst_layout=W.BLOCK_MAJOR)),                                 # B -> A
    (3, dict(num_layers=2, n_req=10, max_len=1500, head_dim=80)),        # 160-byte rows
    (5, dict(num_layers=2, n_req=30, head_dim=80)),                      # 160-byte rows, skip mask
])
def test_scaled_configs(oracle, idx, kw):
    w = W.make_config(idx, **kw)
    check_all_ops(oracle, w, bounds=True)
    check_all_ops(oracle, w)


@pytest.mark.parametrize("tile_bytes,lc_fastest,lc_skew,shift", [(2048, 1, -1, 0), (16384, 0, -1, 0), (1 << 20, 1, 0, 0),
                                                                 (32768, 0, 8, 2), (4096, 0, 4, 0), (8192, 0, 1024, 3),
                                                                 (32768, 0, 0, 0)])
def test_tile_size_and_work_order_do_not_change_the_result(oracle, tile_bytes, lc_fastest, lc_skew, shift):
    """Tile size, sweep order and strip skew (explicit, automatic = -1, off) only
    reorder the work.  The 5- and 3-layer cases have block strides of 5 and 3 times a
    power of two, for which the automatic skew switches itself on; a skew larger than
    the strips of a call (1024, or 8 on a one-layer range) is cut down to fit."""
    B.pdkv_tune("tile_bytes", tile_bytes)
    B.pdkv_tune("lc_fastest", lc_fastest)
    B.pdkv_tune("lc_skew", lc_skew)
    B.pdkv_tune("lc_skew_shift", shift)
    try:
        check_all_ops(oracle, W.make_config(3, num_layers=2, n_req=8, max_len=1200))
        check_all_ops(oracle, W.make_config(5, num_layers=1, n_req=30, src_block=32))
        check_all_ops(oracle, W.make_config(4, num_layers=5, n_req=3, max_len=500))
        check_all_ops(oracle, W.make_config(4, num_layers=3, n_req=3, max_len=500), layers=(1, 2))
    finally:
        B.pdkv_tune("tile_bytes", 32768)
        B.pdkv_tune("lc_fastest", 0)
        B.pdkv_tune("lc_skew", -1)
        B.pdkv_tune("lc_skew_shift", 0)


@pytest.mark.parametrize("variant", [1, 2, 3])
@pytest.mark.parametrize("stages,tile_bytes,chunked", [(2, 16384, 0), (3, 65536, 0), (4, 32768, 1)])
def test_bulk_copy_variant(oracle, variant, stages, tile_bytes, chunked):
    """Variants 1 and 2 (TMA bulk copies through a shared-memory ring; 2 adds tiled
    tensor-map loads for the token-major -> head-major transpose) and 3 (bulk loads in
    read order into shared memory, coalesced stores in write order) must produce the
    same bytes: flat, head-run and transposing tiles, ragged and zero-fill tiles,
    skip masks."""
    B.pdkv_tune("variant", variant)
    B.pdkv_tune("stages", stages)
    B.pdkv_tune("tile_bytes", tile_bytes)
    B.pdkv_tune("chunked", chunked)
    try:
        check_all_ops(oracle, W.make_config(1))
        check_all_ops(oracle, W.make_config(2, num_layers=2, n_req=5, max_len=640))
        check_all_ops(oracle, W.make_config(2, num_layers=2, n_req=4, max_len=600, src_layout=W.LAYER_MAJOR))
        check_all_ops(oracle, W.make_config(3, num_layers=2, n_req=10, max_len=1500), side_stream=True)
        check_all_ops(oracle, W.make_config(5, num_layers=2, n_req=30), layers=(1, 2))
        check_all_ops(oracle, W.make_config(3, num_layers=2, n_req=6, max_len=900, src_layout=W.LAYER_MAJOR,
                                            dst_layout=W.BLOCK_MAJOR))
        # odd block sizes and head counts, 16-byte rows
        lens = np.array([0, 37, 5, 90], np.int32)
        w = W.build_workload("odd", 7, num_layers=2, num_kv_heads=3, head_dim=8, elem_bytes=2, seq_len=lens,
                             src_layout=W.BLOCK_MAJOR, src_block=7, dst_layout=W.LAYER_MAJOR, dst_block=5,
                             src_slack=1.3, dst_slack=1.3)
        check_all_ops(oracle, w)
        # 160-byte rows (80 bf16) and 1-byte elements with 80-byte rows, both directions of the transpose
        for lay in ((W.BLOCK_MAJOR, W.LAYER_MAJOR), (W.LAYER_MAJOR, W.BLOCK_MAJOR)):
            check_all_ops(oracle, W.make_config(3, num_layers=2, n_req=6, max_len=700, head_dim=80, src_layout=lay[0],
                                                dst_layout=lay[1]))
        check_all_ops(oracle, W.make_config(5, num_layers=2, n_req=20, head_dim=80, elem_bytes=1), elem_dtype=np.uint8)
    finally:
        B.pdkv_tune("variant", -1)
        B.pdkv_tune("stages", 3)
        B.pdkv_tune("tile_bytes", 32768)
        B.pdkv_tune("chunked", 0)


@pytest.mark.parametrize("src_order", [0, 1, -1])
def test_row_order_inside_a_tile_does_not_change_the_result(oracle, src_order):
    """Rows of a transposing tile are walked in the order of the side written (0), of the side
    read (1), or chosen by the row size (-1: read order for 160-byte rows, write order for 256)."""
    B.pdkv_tune("src_order", src_order)
    try:
        for D in (80, 128, 24):
            check_all_ops(oracle, W.make_config(3, num_layers=2, n_req=6, max_len=800, head_dim=D))
            check_all_ops(oracle, W.make_config(3, num_layers=2, n_req=5, max_len=600, head_dim=D,
                                                src_layout=W.LAYER_MAJOR, dst_layout=W.BLOCK_MAJOR))
        check_all_ops(oracle, W.make_config(5, num_layers=2, n_req=24, head_dim=80), layers=(1, 2))
    finally:
        B.pdkv_tune("src_order", -1)


@pytest.mark.parametrize("seed", range(16))
def test_random_small_geometries(oracle, seed):
    """Odd block sizes, non-power-of-two heads, rows narrower than 16 bytes,
    1-, 4- and 8-byte elements, random skip masks, zero-length requests."""
    rng = np.random.default_rng(9000 + seed)
    E = int(rng.choice([1, 2, 2, 4, 8]))
    D = int(rng.choice([1, 2, 4, 8, 24, 64]))
    lens = rng.integers(0, 90, size=int(rng.integers(1, 7))).astype(np.int32)
    w = W.build_workload("rnd", int(rng.integers(1 << 30)), num_layers=int(rng.integers(1, 4)),
                         num_kv_heads=int(rng.integers(1, 6)), head_dim=D, elem_bytes=E,
                         seq_len=lens, src_layout=int(rng.integers(2)),
                         src_block=int(rng.choice([1, 3, 7, 16, 48])),
                         dst_layout=int(rng.integers(2)),
                         dst_block=int(rng.choice([2, 5, 16, 32, 64])),
                         src_slack=1.4, dst_slack=1.4)
    if seed % 2 and w.batch.dst_tbl.size:
        w.batch.dst_skip = (rng.random(w.batch.dst_tbl.size) < 0.3).astype(np.uint8)
    dt = {1: np.uint8, 2: np.uint16, 4: np.uint32, 8: np.uint64}[E]
    L = w.src.num_layers
    layers = None if seed % 3 else (L - 1, L)
    check_all_ops(oracle, w, elem_dtype=dt, layers=layers, bounds=True)
    check_all_ops(oracle, w, elem_dtype=dt, layers=layers)


def test_empty_and_degenerate_batches(oracle):
    from paper_2408_08147_b200.session import TransferSession

    g_src = W.Geometry(W.BLOCK_MAJOR, 2, 2, 16, 2, 4, 6)
    g_dst = W.Geometry(W.LAYER_MAJOR, 2, 2, 16, 2, 8, 4)
    sent_t = dev(W.sentinel_pool_numpy(g_dst))
    src_t = dev(W.fill_pool_numpy(g_src, 1))
    z64, z32 = np.zeros(1, np.int64), np.zeros(0, np.int32)
    # no requests at all
    empty = W.Batch(z32, z64, z32, z64, z32)
    dst_t = sent_t.clone()
    with TransferSession(g_src, src_t, g_dst, dst_t, empty) as s:
        assert s.buffer_bytes == 0
        buf_t = torch.zeros(16, dtype=torch.uint8, device="cuda")
        s.pack(buf_t); s.unpack(buf_t); s.transfer(); s.transfer_blockwise(); s.status()
        assert s.launches(B.PDKV_OP_TRANSFER) == 0
    assert torch.equal(dst_t, sent_t)
    # zero-length requests and a request whose blocks are all resident
    lens = np.array([0, 8, 0], np.int32)
    bt = W.Batch(lens, np.array([0, 0, 2, 2], np.int64), np.array([1, 4], np.int32),
                 np.array([0, 0, 1, 1], np.int64), np.array([2], np.int32),
                 np.array([1], np.uint8))
    with TransferSession(g_src, src_t, g_dst, dst_t, bt) as s:
        assert s.buffer_bytes == 0
        s.transfer(); s.transfer_blockwise(); s.status()
    assert torch.equal(dst_t, sent_t)
    # a whole-model call with an empty layer range does nothing
    bt.dst_skip = None
    with TransferSession(g_src, src_t, g_dst, dst_t, bt) as s:
        s.transfer((1, 1)); s.status()
        assert torch.equal(dst_t, sent_t)
        s.transfer()
        want = W.sentinel_pool_numpy(g_dst)
        oracle.transfer(g_src, host(src_t), g_dst, want, bt)
        assert np.array_equal(host(dst_t), want)


def test_per_layer_calls_equal_whole_model(oracle):
    """Sec. 3.5: per-layer or whole-model transfer differ only in offset and
    length; issuing the layers one by one must give the same bytes."""
    from paper_2408_08147_b200.session import TransferSession

    w = W.make_config(3, num_layers=4, n_req=5, max_len=500)
    src = W.fill_pool_numpy(w.src, w.seed)
    sent = W.sentinel_pool_numpy(w.dst)
    want = sent.copy()
    oracle.transfer(w.src, src, w.dst, want, w.batch)
    src_t, dst_t = dev(src), dev(sent)
    with TransferSession(w.src, src_t, w.dst, dst_t, w.batch) as s:
        buf_t = torch.zeros(s.buffer_bytes, dtype=torch.uint8, device="cuda")
        streams = [torch.cuda.Stream() for _ in range(2)]
        torch.cuda.synchronize()
        for l in range(4):                      # layers alternate between two streams
            st = streams[l % 2]
            s.pack(buf_t, (l, l + 1), st.cuda_stream)
            s.unpack(buf_t, (l, l + 1), st.cuda_stream)
        torch.cuda.synchronize()
        assert np.array_equal(host(dst_t), want)
        dst_t.copy_(dev(sent))
        torch.cuda.synchronize()
        for l in reversed(range(4)):
            s.transfer((l, l + 1))
        s.status()
        assert np.array_equal(host(dst_t), want)


@pytest.mark.parametrize("idx,kw", [(5, dict(num_layers=2, n_req=30, src_block=32)),
                                    (3, dict(num_layers=2, n_req=6, max_len=700, src_layout=W.LAYER_MAJOR,
                                             dst_layout=W.BLOCK_MAJOR)),
                                    (4, dict(num_layers=2, n_req=3, max_len=500))])
def test_host_resident_pools(oracle, idx, kw):
    """Upload the referenced prefill blocks from a host image, transfer, download
    the written decode blocks: the host decode image must equal the checker's,
    and nothing else may move in either direction."""
    from paper_2408_08147_b200.session import TransferSession

    w = W.make_config(idx, **kw)
    src = W.fill_pool_numpy(w.src, w.seed)
    sent = W.sentinel_pool_numpy(w.dst)
    want = sent.copy()
    oracle.transfer(w.src, src, w.dst, want, w.batch)
    h_src = torch.from_numpy(src.view(np.uint8).copy()).pin_memory()
    h_dst = torch.from_numpy(sent.view(np.uint8).copy()).pin_memory()
    src_t = torch.full((w.src.num_bytes(),), 0x5A, dtype=torch.uint8, device="cuda")
    dst_t = dev(sent)
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    with TransferSession(w.src, src_t, w.dst, dst_t, w.batch, stream.cuda_stream) as s:
        up, down = s.block_bytes()
        s.upload_blocks(h_src)
        s.transfer()
        s.download_blocks(h_dst)
        s.status()
    assert np.array_equal(h_dst.numpy().view(np.uint16), want)
    # device prefill pool: uploaded blocks equal the host image, all others keep the 0x5A fill
    got_src = src_t.cpu().numpy()
    same = got_src == src.view(np.uint8)
    untouched = got_src == 0x5A
    assert (same | untouched).all()
    not_uploaded = w.src.num_bytes() - up          # bytes of blocks the batch does not read
    assert not_uploaded * 0.98 <= int((~same).sum()) <= not_uploaded   # (1/256 of the fill matches by chance)
    assert up <= w.src.num_bytes() and down <= w.dst.num_bytes()
    if w.src_occupied.size or w.batch.dst_skip is not None:
        assert up < w.src.num_bytes()


def test_per_layer_calls_replayed_from_a_cuda_graph(oracle):
    """pack / unpack / transfer only enqueue kernels (no allocation, copy or
    synchronisation), so a per-layer sequence can be captured once and replayed."""
    from paper_2408_08147_b200.session import TransferSession

    w = W.make_config(3, num_layers=4, n_req=6, max_len=700)
    src = W.fill_pool_numpy(w.src, w.seed)
    sent = W.sentinel_pool_numpy(w.dst)
    want = sent.copy()
    oracle.transfer(w.src, src, w.dst, want, w.batch)
    src_t, dst_t = dev(src), dev(sent)
    cap = torch.cuda.Stream()
    torch.cuda.synchronize()
    with TransferSession(w.src, src_t, w.dst, dst_t, w.batch, cap.cuda_stream) as s:
        buf_t = torch.zeros(s.buffer_bytes, dtype=torch.uint8, device="cuda")
        s.transfer((0, 1))                      # warm-up outside capture (module load, attributes)
        s.pack(buf_t, (0, 1)); s.unpack(buf_t, (0, 1))
        torch.cuda.synchronize()
        dst_t.copy_(dev(sent))
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=cap):
            st = torch.cuda.current_stream().cuda_stream
            for l in range(2):
                s.transfer((l, l + 1), st)
            for l in range(2, 4):
                s.pack(buf_t, (l, l + 1), st)
                s.unpack(buf_t, (l, l + 1), st)
        torch.cuda.synchronize()
        assert np.array_equal(host(dst_t), sent), "capture must not execute anything"
        graph.replay()
        torch.cuda.synchronize()
        assert np.array_equal(host(dst_t), want)
        dst_t.copy_(dev(sent))
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        assert np.array_equal(host(dst_t), want)


def test_bounds_checked_kernels_refuse_and_skip(oracle):
    """With the range check on and both sides declared 4 KiB shorter than they are,
    accesses into the last 4 KiB are refused: they are skipped (the sentinel
    survives), everything else is copied, and the plan reports the refusal."""
    from paper_2408_08147_b200.session import TransferSession

    w = W.make_config(2, num_layers=2, n_req=2, max_len=256)      # block-major both sides, every block used
    src = W.fill_pool_numpy(w.src, w.seed)
    sent = W.sentinel_pool_numpy(w.dst)
    want = sent.copy()
    oracle.transfer(w.src, src, w.dst, want, w.batch)
    src_t, dst_t = dev(src), dev(sent)
    torch.cuda.synchronize()
    B.pdkv_tune("debug_bounds", 1)
    B.pdkv_tune("debug_shrink", 4096)
    try:
        with TransferSession(w.src, src_t, w.dst, dst_t, w.batch) as s:
            s.transfer()
            with pytest.raises(B.PdkvError) as e:
                s.status()
            assert e.value.status == B.PDKV_ERR_DEVICE_BOUNDS and "refused" in str(e.value)
        # Both pools are [block][layer][K/V][token][head][dim] with 2 KiB per token, so the last
        # 4 KiB of a pool are tokens 126..127 of its last block's last (layer, V) strip.  Refused:
        # the writes into the decode pool's tail, and the reads of the prefill pool's tail (whose
        # destination is found through the tables; same block size on both sides).
        expect = want.copy().reshape(w.dst.shape())
        L, NB = w.dst.num_layers, w.dst.num_blocks
        expect[NB - 1, L - 1, 1, 126:128] = SENT
        pos = int(np.flatnonzero(w.batch.src_tbl == w.src.num_blocks - 1)[0])
        expect[int(w.batch.dst_tbl[pos]), L - 1, 1, 126:128] = SENT
        assert np.array_equal(host(dst_t), expect.reshape(-1))
        # a clean run on the same plan data clears nothing by itself: a fresh plan reports OK
        B.pdkv_tune("debug_shrink", 0)
        dst_t.copy_(dev(sent)); torch.cuda.synchronize()
        with TransferSession(w.src, src_t, w.dst, dst_t, w.batch) as s:
            s.transfer(); s.status()
        assert np.array_equal(host(dst_t), want)
    finally:
        B.pdkv_tune("debug_bounds", 0)
        B.pdkv_tune("debug_shrink", 0)


@pytest.mark.parametrize("idx,kw", [(3, dict(num_layers=2, n_req=8, max_len=900)), (5, dict(num_layers=2, n_req=30))])
def test_sender_only_and_receiver_only_plans(oracle, idx, kw):
    """The two halves as separate devices would run them (Sec. 3.5): the sender
    holds only the prefill pool and a pack-only plan, the receiver only the decode
    pool and an unpack-only plan; the buffer travels as one copy in between.  (Here
    both halves run on the same GPU; the buffer copy stands in for the link.)"""
    from paper_2408_08147_b200.session import TransferSession

    w = W.make_config(idx, **kw)
    G = w.dst.block_tokens
    src = W.fill_pool_numpy(w.src, w.seed)
    sent = W.sentinel_pool_numpy(w.dst)
    want = sent.copy()
    oracle.transfer(w.src, src, w.dst, want, w.batch)
    src_t, dst_t = dev(src), dev(sent)
    torch.cuda.synchronize()
    sender = TransferSession(w.src, src_t, None, None, w.batch, skip_granule_tokens=G)
    receiver = TransferSession(None, None, w.dst, dst_t, w.batch)
    try:
        assert sender.buffer_bytes == receiver.buffer_bytes == oracle.buffer_elems(w.batch, G, w.src) * 2
        assert np.array_equal(sender.request_offsets, receiver.request_offsets)
        send_buf = torch.zeros(sender.buffer_bytes, dtype=torch.uint8, device="cuda")
        recv_buf = torch.empty_like(send_buf)
        L = w.src.num_layers
        for l in range(L):                                  # per-layer trigger: offset and length per layer
            sender.pack(send_buf, (l, l + 1))
        recv_buf.copy_(send_buf)                            # the whole buffer in one copy (Sec. 3.5)
        receiver.unpack(recv_buf)
        torch.cuda.synchronize()
        assert np.array_equal(host(dst_t), want)
        with pytest.raises(B.PdkvError):
            sender.transfer()
        with pytest.raises(B.PdkvError):
            receiver.pack(send_buf)
    finally:
        sender.close()
        receiver.close()


def test_plan_in_caller_workspace(oracle):
    """pdkv_plan_create_in keeps the plan's device arrays in memory the caller
    owns: too small a workspace is refused with the needed size, a sufficient one
    gives the same bytes as an allocating plan, and the workspace can be reused."""
    w = W.make_config(3, num_layers=2, n_req=8, max_len=900)
    b = w.batch
    src = W.fill_pool_numpy(w.src, w.seed)
    sent = W.sentinel_pool_numpy(w.dst)
    want = sent.copy()
    oracle.transfer(w.src, src, w.dst, want, b)
    src_t, dst_t = dev(src), dev(sent)
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    ps = B.pdkv_pool_create(B.desc_of(w.src), src_t.data_ptr(), src_t.numel(), 0)
    pd = B.pdkv_pool_create(B.desc_of(w.dst), dst_t.data_ptr(), dst_t.numel(), 0)
    args = (ps, pd, 0, b.seq_len, b.src_tbl_off, b.src_tbl, b.dst_tbl_off, b.dst_tbl, b.dst_skip)
    with pytest.raises(B.PdkvError) as e:
        B.pdkv_plan_create_in(*args, workspace_ptr=ws.data_ptr(), workspace_bytes=512)
    assert e.value.status == B.PDKV_ERR_BUFFER_TOO_SMALL and e.value.needed_bytes > 512
    for _ in range(2):                                   # the same workspace, two plans in a row
        plan, need = B.pdkv_plan_create_in(*args, workspace_ptr=ws.data_ptr(), workspace_bytes=ws.numel())
        assert need == e.value.needed_bytes
        B.pdkv_transfer(plan, 0, w.src.num_layers)
        B.pdkv_plan_status(plan)
        assert np.array_equal(host(dst_t), want)
        B.pdkv_plan_destroy(plan)
        dst_t.copy_(dev(sent)); torch.cuda.synchronize()
    B.pdkv_pool_destroy(ps); B.pdkv_pool_destroy(pd)


def test_pinned_and_autotuned_launch_shapes(oracle):
    """Per-plan launch shapes (set by hand, or found by pdkv_plan_autotune) change how
    the work is spread over threads, never the bytes; shapes found for a geometry
    are handed to later plans of that geometry unless "autotune_reuse" is off."""
    from paper_2408_08147_b200.session import TransferSession

    lens = np.array([700, 33, 1500, 16, 260], np.int32)
    w = W.build_workload("rows-of-160-bytes", 11, num_layers=2, num_kv_heads=8, head_dim=80, elem_bytes=2,
                         seq_len=lens, src_layout=W.BLOCK_MAJOR, src_block=16, dst_layout=W.LAYER_MAJOR,
                         dst_block=128, src_slack=1.2, dst_slack=1.2)
    G = w.dst.block_tokens
    src = W.fill_pool_numpy(w.src, w.seed)
    sent = W.sentinel_pool_numpy(w.dst)
    want_dst = sent.copy()
    oracle.transfer(w.src, src, w.dst, want_dst, w.batch)
    want_buf = np.zeros(oracle.buffer_elems(w.batch, G, w.src), np.uint16)
    oracle.pack(w.src, src, w.batch, G, want_buf)
    src_t, dst_t = dev(src), dev(sent)
    torch.cuda.synchronize()
    ops = (B.PDKV_OP_PACK, B.PDKV_OP_UNPACK, B.PDKV_OP_TRANSFER)
    try:
        with TransferSession(w.src, src_t, w.dst, dst_t, w.batch) as s:
            buf_t = torch.zeros(s.buffer_bytes, dtype=torch.uint8, device="cuda")
            for shape in [(640, 1, 2), (160, 4, 3), (96, 2, 8), (1024, 1, 1), (256, 8, 1)]:
                for op in ops:
                    B.pdkv_plan_set_shape(s.plan, op, *shape)
                buf_t.zero_()
                dst_t.copy_(dev(sent))
                torch.cuda.synchronize()
                s.pack(buf_t); s.unpack(buf_t); s.status()
                assert np.array_equal(host(buf_t), want_buf), f"pack with shape {shape}"
                assert np.array_equal(host(dst_t), want_dst), f"unpack with shape {shape}"
                dst_t.copy_(dev(sent))
                torch.cuda.synchronize()
                s.transfer(); s.status()
                assert np.array_equal(host(dst_t), want_dst), f"transfer with shape {shape}"
            for op in ops:
                B.pdkv_plan_set_shape(s.plan, op, 0, 0, 0)
            buf_t.zero_()
            dst_t.copy_(dev(sent))
            torch.cuda.synchronize()
            found = s.autotune(buf_t)
            s.status()
            for op, (threads, unroll, ctas, skew) in found.items():
                assert (threads, unroll, ctas) == (0, 0, 0) or (threads % 32 == 0 and unroll in (1, 2, 4) and ctas >= 1)
                assert skew in (-1, 0, 16)
            # autotuning runs the real operations: buffer and decode pool hold the batch afterwards
            assert np.array_equal(host(buf_t), want_buf)
            assert np.array_equal(host(dst_t), want_dst)
            dst_t.copy_(dev(sent))
            torch.cuda.synchronize()
            s.transfer(); s.status()
            assert np.array_equal(host(dst_t), want_dst), f"transfer with the shapes found: {found}"
            with TransferSession(w.src, src_t, w.dst, dst_t, w.batch) as again:      # same geometry: shapes handed on
                assert {op: B.pdkv_plan_shape(again.plan, op) for op in ops} == found
            B.pdkv_tune("autotune_reuse", 0)
            with TransferSession(w.src, src_t, w.dst, dst_t, w.batch) as fresh:
                assert all(B.pdkv_plan_shape(fresh.plan, op) == (0, 0, 0, -1) for op in ops)
    finally:
        B.pdkv_tune("autotune_reuse", 1)


def test_transfer_as_plain_device_copies(oracle):
    """Block-major pools with equal blocks: the fused transfer issued as device copies (one per
    block and layer range, 2-D copies and memsets for partial blocks) writes the same bytes;
    other geometries are refused."""
    from paper_2408_08147_b200.session import TransferSession

    for kw, layers in ((dict(num_layers=3, n_req=5, max_len=640), None), (dict(num_layers=4, n_req=4, max_len=333), (1, 3))):
        w = W.make_config(2, **kw)
        w.batch.seq_len[:] = np.array([kw["max_len"], 1, 129, 300, 256][:w.batch.n_req], np.int32)   # ragged tails
        src = W.fill_pool_numpy(w.src, w.seed)
        sent = W.sentinel_pool_numpy(w.dst)
        want = sent.copy()
        oracle.transfer(w.src, src, w.dst, want, w.batch, layers=layers)
        src_t, dst_t = dev(src), dev(sent)
        torch.cuda.synchronize()
        with TransferSession(w.src, src_t, w.dst, dst_t, w.batch) as s:
            s.transfer_copies(layers)
            s.status()
        assert np.array_equal(host(dst_t), want)
    w = W.make_config(3, num_layers=2, n_req=3, max_len=300)            # re-blocking: not expressible as block copies
    src_t, dst_t = dev(W.fill_pool_numpy(w.src, w.seed)), dev(W.sentinel_pool_numpy(w.dst))
    with TransferSession(w.src, src_t, w.dst, dst_t, w.batch) as s:
        with pytest.raises(B.PdkvError) as e:
            s.transfer_copies()
        assert e.value.status == B.PDKV_ERR_GEOMETRY


@pytest.mark.parametrize("partition_sms", [0, 16])
def test_per_layer_transfer_beside_a_compute_kernel(oracle, partition_sms):
    """Sec. 3.5, per-layer trigger: layer l is transferred on a side stream while the main
    stream computes (a matrix product stands in for layer l+1).  The decode pool must still
    be bit-exact -- also when the transfer runs on an SM partition of its own."""
    from paper_2408_08147_b200.session import TransferSession

    w = W.make_config(3, num_layers=6, n_req=8, max_len=1200)
    src = W.fill_pool_numpy(w.src, w.seed)
    sent = W.sentinel_pool_numpy(w.dst)
    want = sent.copy()
    oracle.transfer(w.src, src, w.dst, want, w.batch)
    src_t, dst_t = dev(src), dev(sent)
    a = torch.randn(2048, 2048, device="cuda", dtype=torch.bfloat16)
    c = torch.empty_like(a)
    part = None
    if partition_sms:
        try:
            part = B.pdkv_sm_partition_create(0, partition_sms)
        except B.PdkvError as e:
            pytest.skip(f"no SM partition on this driver: {e}")
        t_sms, c_sms = B.pdkv_sm_partition_info(part)
        assert t_sms >= partition_sms and c_sms > 0
        total = torch.cuda.get_device_properties(0).multi_processor_count
        assert t_sms + c_sms <= total
        side = torch.cuda.ExternalStream(B.pdkv_sm_partition_stream(part, 0))
        main = torch.cuda.ExternalStream(B.pdkv_sm_partition_stream(part, 1))
    else:
        main, side = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    try:
        with TransferSession(w.src, src_t, w.dst, dst_t, w.batch, side.cuda_stream) as s:
            for l in range(w.src.num_layers):
                with torch.cuda.stream(main):
                    for _ in range(4):
                        torch.matmul(a, a, out=c)
                    ev = torch.cuda.Event()
                    ev.record(main)
                side.wait_event(ev)
                s.transfer((l, l + 1), side.cuda_stream)
            torch.cuda.synchronize()
            s.status()
        assert np.array_equal(host(dst_t), want)
    finally:
        if part:
            torch.cuda.synchronize()
            del main, side
            B.pdkv_sm_partition_destroy(part)


def test_address_coded_values_name_where_a_row_came_from(oracle):
    """Every source element carries its own logical coordinate (request, token, layer, K/V,
    head, dim) as a unique 16-bit code, so a misplaced row would not only differ from the
    checker: the decoded value says which coordinate landed in its place.  The decode pool is
    also read back through reshape / index / transpose views (no offset formula) and must
    list the codes of every request in coordinate order."""
    from paper_2408_08147_b200.session import TransferSession

    L, H, D = 2, 2, 8
    lens = np.array([150, 1, 97, 0, 260], np.int32)
    assert int(lens.sum()) * 2 * L * H * D < 65535
    w = W.build_workload("coded", 99, num_layers=L, num_kv_heads=H, head_dim=D, elem_bytes=2, seq_len=lens,
                         src_layout=W.BLOCK_MAJOR, src_block=16, dst_layout=W.LAYER_MAJOR, dst_block=32,
                         src_slack=1.3, dst_slack=1.3)
    b = w.batch
    per_tok = 2 * L * H * D
    first_tok = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)

    def decode(code):
        i = int(code) - 1
        g, rest = divmod(i, per_tok)
        r = int(np.searchsorted(first_tok, g, side="right") - 1)
        l, rest = divmod(rest, 2 * H * D)
        c, rest = divmod(rest, H * D)
        h, d = divmod(rest, D)
        return dict(r=r, t=g - int(first_tok[r]), l=l, c=c, h=h, d=d)

    src6 = np.full(w.src.shape(), SENT, np.uint16)                 # [NB][L][2][B][H][D]
    Bp = w.src.block_tokens
    for r in range(b.n_req):
        for t in range(int(lens[r])):
            blk = int(b.src_tbl[b.src_tbl_off[r] + t // Bp])
            base = (int(first_tok[r]) + t) * per_tok + 1
            src6[blk, :, :, t % Bp] = (base + np.arange(per_tok)).reshape(L, 2, H, D)
    src = src6.reshape(-1)
    sent = W.sentinel_pool_numpy(w.dst)
    want = sent.copy()
    oracle.transfer(w.src, src, w.dst, want, b)
    src_t, dst_t = dev(src), dev(sent)
    torch.cuda.synchronize()
    with TransferSession(w.src, src_t, w.dst, dst_t, b) as s:
        buf_t = torch.zeros(s.buffer_bytes, dtype=torch.uint8, device="cuda")
        s.pack(buf_t)
        s.status()
        packed = host(buf_t)
        s.transfer()
        s.status()
    got = host(dst_t)
    bad = np.flatnonzero(got != want)
    if bad.size:
        i = int(bad[0])
        here = "pad or untouched" if want[i] in (0, SENT) else decode(want[i])
        there = "zero or sentinel" if got[i] in (0, SENT) else decode(got[i])
        pytest.fail(f"{bad.size} decode-pool elements differ; element {i} should hold {here} but holds {there}")
    # the contiguous buffer is the coordinates in order: request, layer, K/V, token, head, dim
    want_buf = np.concatenate([((int(first_tok[r]) + np.arange(int(lens[r])))[None, None, :, None] * per_tok + 1 +
                                (np.arange(L)[:, None, None, None] * 2 + np.arange(2)[None, :, None, None]) * H * D +
                                np.arange(H * D)[None, None, None, :]).reshape(-1) for r in range(b.n_req)])
    assert np.array_equal(packed, want_buf.astype(np.uint16))
    # decode pool through views: [L][2][NB][H][B][D] -> per request [L][2][token][H][D]
    d6 = got.reshape(w.dst.shape())
    Bd = w.dst.block_tokens
    for r in range(b.n_req):
        n = int(lens[r])
        if n == 0:
            continue
        ids = b.dst_tbl[b.dst_tbl_off[r]:b.dst_tbl_off[r] + -(-n // Bd)].astype(np.int64)
        x = d6[:, :, ids].transpose(0, 1, 2, 4, 3, 5).reshape(L, 2, -1, H, D)       # tokens of the request in order
        codes = x[:, :, :n].transpose(2, 0, 1, 3, 4).reshape(n, per_tok).astype(np.int64)
        expect = (int(first_tok[r]) + np.arange(n))[:, None] * per_tok + 1 + np.arange(per_tok)[None, :]
        assert np.array_equal(codes, expect), f"request {r}: first wrong element holds {decode(codes[codes != expect][0])}"
        assert (x[:, :, n:] == 0).all()                                             # tail slots of the last block
