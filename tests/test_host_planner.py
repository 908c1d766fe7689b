"""Host-side logic of the library, no GPU needed: exported symbols, argument
validation, buffer offsets, traffic accounting, and the tile lists (executed by
a small numpy interpreter and compared with the CPU checker)."""
import os
import re

import numpy as np
import pytest

from paper_2408_08147_b200 import binding as B
from paper_2408_08147_b200 import build as pdkv_build
from paper_2408_08147_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SENT = W.SENTINEL_U16
FAKE_BASE = 0x7F0000000000  # never dereferenced: dry-run plans make no CUDA call


@pytest.fixture(scope="module", autouse=True)
def built():
    pdkv_build.build_library()
    B.pdkv_tune("dry_run", 1)
    yield
    B.pdkv_tune("dry_run", 0)
    B.pdkv_tune("tile_bytes", 32768)


def test_library_exports_every_declared_symbol():
    with open(os.path.join(ROOT, "include", "pdkv.h")) as f:
        text = f.read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(pdkv_[a-z_]+)\s*\(", text))
    assert {"pdkv_pool_create", "pdkv_pack", "pdkv_unpack", "pdkv_transfer"} <= declared
    lib = B.lib()
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in pdkv.h but not exported"
    assert declared == set(B.EXPORTS)


def _pools(w):
    ps = B.pdkv_pool_create(B.desc_of(w.src), FAKE_BASE, w.src.num_bytes(), 0)
    pd = B.pdkv_pool_create(B.desc_of(w.dst), FAKE_BASE + (1 << 40), w.dst.num_bytes(), 0)
    return ps, pd


def _plan(w, ps, pd, **over):
    b = w.batch
    kw = dict(seq_len=b.seq_len, src_tbl_off=b.src_tbl_off, src_tbl=b.src_tbl,
              dst_tbl_off=b.dst_tbl_off, dst_tbl=b.dst_tbl, dst_skip=b.dst_skip)
    kw.update(over)
    return B.pdkv_plan_create(ps, pd, w.dst.block_tokens, **kw)


def test_pool_validation():
    good = B.make_desc(0, 2, 4, 64, 2, 16, 10)
    assert B.pdkv_pool_bytes(good) == 10 * 2 * 2 * 16 * 4 * 64 * 2
    for bad in [B.make_desc(2, 2, 4, 64, 2, 16, 10), B.make_desc(0, 0, 4, 64, 2, 16, 10),
                B.make_desc(0, 2, 4, 64, 3, 16, 10), B.make_desc(0, 2, 4, 64, 2, 0, 10),
                B.make_desc(0, 2, 4, 64, 2, 16, 0), B.make_desc(0, 2, -1, 64, 2, 16, 10)]:
        assert B.pdkv_pool_bytes(bad) == 0
        with pytest.raises(B.PdkvError) as e:
            B.pdkv_pool_create(bad, FAKE_BASE, 1 << 30, 0)
        assert e.value.status == B.PDKV_ERR_GEOMETRY
    with pytest.raises(B.PdkvError) as e:
        B.pdkv_pool_create(good, FAKE_BASE + 8, 1 << 30, 0)       # misaligned
    assert e.value.status == B.PDKV_ERR_INVALID_ARG
    with pytest.raises(B.PdkvError) as e:
        B.pdkv_pool_create(good, FAKE_BASE, B.pdkv_pool_bytes(good) - 1, 0)  # too small
    assert e.value.status == B.PDKV_ERR_INVALID_ARG
    with pytest.raises(B.PdkvError) as e:
        B.pdkv_pool_create(good, 0, 1 << 30, 0)
    assert e.value.status == B.PDKV_ERR_INVALID_ARG


def test_plan_validation_errors():
    w = W.make_config(1)
    ps, pd = _pools(w)
    b = w.batch

    def status(**over):
        with pytest.raises(B.PdkvError) as e:
            _plan(w, ps, pd, **over)
        return e.value.status

    t = b.src_tbl.copy(); t[3] = w.src.num_blocks
    assert status(src_tbl=t) == B.PDKV_ERR_TABLE
    t = b.src_tbl.copy(); t[0] = -1
    assert status(src_tbl=t) == B.PDKV_ERR_TABLE
    t = b.dst_tbl.copy(); t[1] = t[0]
    assert status(dst_tbl=t) == B.PDKV_ERR_TABLE                   # two writers for one block
    off = b.src_tbl_off.copy(); off[1:] -= 1
    off[1] = max(off[1], 0)
    assert status(src_tbl_off=off) == B.PDKV_ERR_TABLE             # a table is too short
    off = b.dst_tbl_off.copy(); off[2] = off[1] - 1
    assert status(dst_tbl_off=off) == B.PDKV_ERR_TABLE             # not monotone
    ln = b.seq_len.copy(); ln[0] = -5
    assert status(seq_len=ln) == B.PDKV_ERR_INVALID_ARG
    assert status(src_tbl=None) == B.PDKV_ERR_INVALID_ARG
    # duplicate prefill blocks are legal (shared prefix on the sender)
    t = b.src_tbl.copy(); t[1] = t[0]
    B.pdkv_plan_destroy(_plan(w, ps, pd, src_tbl=t))
    # geometry mismatch between the two pools
    other = B.pdkv_pool_create(B.make_desc(1, 3, 4, 64, 2, 32, w.dst.num_blocks), FAKE_BASE,
                               1 << 40, 0)
    with pytest.raises(B.PdkvError) as e:
        _plan(w, ps, other)
    assert e.value.status == B.PDKV_ERR_GEOMETRY
    # overlapping pools (in-place re-blocking) are refused
    near = B.pdkv_pool_create(B.desc_of(w.dst), FAKE_BASE + 4096, w.dst.num_bytes(), 0)
    with pytest.raises(B.PdkvError) as e:
        _plan(w, ps, near)
    assert e.value.status == B.PDKV_ERR_INVALID_ARG
    B.pdkv_pool_destroy(near)
    # skip granule must be the decode block
    with pytest.raises(B.PdkvError) as e:
        B.pdkv_plan_create(ps, pd, 16, b.seq_len, b.src_tbl_off, b.src_tbl, b.dst_tbl_off, b.dst_tbl)
    assert e.value.status == B.PDKV_ERR_INVALID_ARG
    with pytest.raises(B.PdkvError) as e:
        B.pdkv_plan_create(None, None, 0, b.seq_len)
    assert e.value.status == B.PDKV_ERR_INVALID_ARG
    for p in (ps, pd, other):
        B.pdkv_pool_destroy(p)


def test_launch_argument_errors_and_dry_run_refusal():
    w = W.make_config(1)
    ps, pd = _pools(w)
    plan = _plan(w, ps, pd)
    total, _ = B.pdkv_plan_buffer(plan)
    for fn, args in [(B.pdkv_pack, (plan, FAKE_BASE, total, 0, 3)),
                     (B.pdkv_pack, (plan, FAKE_BASE, total, -1, 1)),
                     (B.pdkv_unpack, (plan, FAKE_BASE, total, 2, 1)),
                     (B.pdkv_pack, (plan, FAKE_BASE + 4, total, 0, 2)),
                     (B.pdkv_transfer, (plan, 0, 5))]:
        with pytest.raises(B.PdkvError) as e:
            fn(*args)
        assert e.value.status == B.PDKV_ERR_INVALID_ARG
    with pytest.raises(B.PdkvError) as e:
        B.pdkv_pack(plan, FAKE_BASE, total - 1, 0, 2)
    assert e.value.status == B.PDKV_ERR_BUFFER_TOO_SMALL
    with pytest.raises(B.PdkvError) as e:               # buffer inside the decode pool
        B.pdkv_unpack(plan, FAKE_BASE + (1 << 40) + 256, total, 0, 2)
    assert e.value.status == B.PDKV_ERR_INVALID_ARG
    # a dry-run plan owns no device arrays: launching is refused, not attempted
    for fn, args in [(B.pdkv_pack, (plan, FAKE_BASE, total, 0, 2)),
                     (B.pdkv_transfer, (plan, 0, 2)), (B.pdkv_transfer_blockwise, (plan,)),
                     (B.pdkv_plan_status, (plan,))]:
        with pytest.raises(B.PdkvError) as e:
            fn(*args)
        assert e.value.status == B.PDKV_ERR_INVALID_ARG
    # pack-only plans cannot unpack
    ponly = B.pdkv_plan_create(ps, None, 32, w.batch.seq_len, w.batch.src_tbl_off, w.batch.src_tbl)
    with pytest.raises(B.PdkvError) as e:
        B.pdkv_unpack(ponly, FAKE_BASE, total, 0, 2)
    assert e.value.status == B.PDKV_ERR_INVALID_ARG
    assert B.pdkv_plan_buffer(ponly)[0] == total
    for p in (plan, ponly):
        B.pdkv_plan_destroy(p)
    B.pdkv_pool_destroy(ps); B.pdkv_pool_destroy(pd)
    assert "table" in B.pdkv_strerror(B.PDKV_ERR_TABLE)
    with pytest.raises(B.PdkvError):
        B.pdkv_tune("no_such_key", 1)
    with pytest.raises(B.PdkvError):
        B.pdkv_tune("threads", 33)
    B.pdkv_tune("threads", 0)


# --------------------------------------------------------------------------
# tile lists, executed in numpy
# --------------------------------------------------------------------------

def _side(geom):
    row = geom.head_dim * geom.elem_bytes
    hrow = row * geom.num_kv_heads
    if geom.layout == W.BLOCK_MAJOR:
        return geom.block_tokens * hrow, hrow, row
    return geom.num_blocks * geom.num_kv_heads * geom.block_tokens * row, row, geom.block_tokens * row


def run_tiles(tiles, src_bytes, src_side, dst_bytes, dst_side, geom, layers):
    """Apply a tile list the way the header documents it; also proves that no
    destination byte is written twice."""
    row = geom.head_dim * geom.elem_bytes
    hrow = row * geom.num_kv_heads
    written = np.zeros(dst_bytes.shape[0], bool)
    for t in tiles:
        for lc in range(2 * layers[0], 2 * layers[1]):
            s_lc, s_tok, s_head = src_side if src_side else (t["n_kept"] * hrow, hrow, row)
            d_lc, d_tok, d_head = dst_side if dst_side else (t["n_kept"] * hrow, hrow, row)
            for tk in range(t["ntok"]):
                for h in range(geom.num_kv_heads):
                    d = t["dst_off"] + lc * d_lc + tk * d_tok + h * d_head
                    assert not written[d:d + row].any()
                    written[d:d + row] = True
                    if t["src_off"] < 0:
                        dst_bytes[d:d + row] = 0
                    else:
                        s = t["src_off"] + lc * s_lc + tk * s_tok + h * s_head
                        dst_bytes[d:d + row] = src_bytes[s:s + row]
    return written


def _random_workload(rng, skip):
    L = int(rng.integers(1, 3)); H = int(rng.integers(1, 4)); D = int(rng.choice([4, 8, 16]))
    lens = rng.integers(0, 40, size=int(rng.integers(1, 5))).astype(np.int32)
    w = W.build_workload("t", int(rng.integers(1 << 30)), num_layers=L, num_kv_heads=H,
                         head_dim=D, elem_bytes=2, seq_len=lens,
                         src_layout=int(rng.integers(2)), src_block=int(rng.choice([1, 3, 4, 8, 16])),
                         dst_layout=int(rng.integers(2)), dst_block=int(rng.choice([2, 4, 5, 8, 32])),
                         src_slack=1.3, dst_slack=1.3)
    if skip and w.batch.dst_tbl.size:
        w.batch.dst_skip = (rng.random(w.batch.dst_tbl.size) < 0.35).astype(np.uint8)
    return w


@pytest.mark.parametrize("seed", range(24))
def test_tile_lists_reproduce_the_checker(oracle, seed):
    rng = np.random.default_rng(4242 + seed)
    w = _random_workload(rng, skip=bool(seed % 2))
    B.pdkv_tune("tile_bytes", int(rng.choice([64, 256, 4096, 65536])))
    ps, pd = _pools(w)
    plan = _plan(w, ps, pd)
    G = w.dst.block_tokens
    g = w.src
    layers = (0, g.num_layers) if seed % 3 else (g.num_layers - 1, g.num_layers)

    src = W.fill_pool_numpy(w.src, w.seed)
    n_buf = oracle.buffer_elems(w.batch, G, w.src)
    total, offs = B.pdkv_plan_buffer(plan, w.batch.n_req)
    assert total == n_buf * 2
    assert np.array_equal(offs, oracle.request_offsets(w.batch, G, w.src) * 2)

    want_buf = np.full(n_buf, SENT, np.uint16)
    oracle.pack(w.src, src, w.batch, G, want_buf, layers=layers)
    got_buf = np.full(n_buf, SENT, np.uint16)
    run_tiles(B.pdkv_plan_tiles(plan, B.PDKV_OP_PACK), src.view(np.uint8), _side(w.src),
              got_buf.view(np.uint8), None, g, layers)
    assert np.array_equal(got_buf, want_buf)

    full_buf = np.zeros(n_buf, np.uint16)
    oracle.pack(w.src, src, w.batch, G, full_buf)
    want_dst = W.sentinel_pool_numpy(w.dst)
    oracle.unpack(w.dst, want_dst, w.batch, full_buf, layers=layers)
    got_dst = W.sentinel_pool_numpy(w.dst)
    run_tiles(B.pdkv_plan_tiles(plan, B.PDKV_OP_UNPACK), full_buf.view(np.uint8), None,
              got_dst.view(np.uint8), _side(w.dst), g, layers)
    assert np.array_equal(got_dst, want_dst)

    got_dst = W.sentinel_pool_numpy(w.dst)
    written = run_tiles(B.pdkv_plan_tiles(plan, B.PDKV_OP_TRANSFER), src.view(np.uint8),
                        _side(w.src), got_dst.view(np.uint8), _side(w.dst), g, layers)
    assert np.array_equal(got_dst, want_dst)

    if layers == (0, g.num_layers):
        rd, wr = B.pdkv_plan_traffic(plan, B.PDKV_OP_TRANSFER)
        assert rd == total and wr == int(written.sum())
        assert B.pdkv_plan_traffic(plan, B.PDKV_OP_PACK) == (total, total)
    B.pdkv_plan_destroy(plan)
    B.pdkv_pool_destroy(ps); B.pdkv_pool_destroy(pd)


def test_tiles_respect_size_cap_and_block_boundaries():
    w = W.make_config(3, num_layers=2, n_req=6, max_len=700)
    B.pdkv_tune("tile_bytes", 16384)
    ps, pd = _pools(w)
    plan = _plan(w, ps, pd)
    hrow = w.src.num_kv_heads * w.src.head_dim * w.src.elem_bytes
    for op in (B.PDKV_OP_PACK, B.PDKV_OP_UNPACK, B.PDKV_OP_TRANSFER):
        tiles = B.pdkv_plan_tiles(plan, op)
        assert tiles["ntok"].min() >= 1 and tiles["ntok"].max() * hrow <= 16384
        copy = tiles[tiles["src_off"] >= 0]
        assert copy["ntok"].sum() == w.batch.seq_len.sum()
    n_blocks = int((-(-w.batch.seq_len.astype(np.int64) // 16)).sum())
    assert B.pdkv_plan_launches(plan, B.PDKV_OP_BLOCKWISE) == n_blocks
    assert B.pdkv_plan_launches(plan, B.PDKV_OP_TRANSFER) == 1
    B.pdkv_plan_destroy(plan)
    B.pdkv_pool_destroy(ps); B.pdkv_pool_destroy(pd)


def test_block_bytes_count_referenced_and_written_blocks():
    w = W.make_config(5, num_layers=2, n_req=60, src_block=32)
    ps, pd = _pools(w)
    plan = _plan(w, ps, pd)
    b = w.batch
    src_ids, dst_ids = set(), set()
    for r in range(b.n_req):
        for t in range(int(b.seq_len[r])):
            e = b.dst_tbl_off[r] + t // w.dst.block_tokens
            if b.dst_skip[e]:
                continue
            dst_ids.add(int(b.dst_tbl[e]))
            src_ids.add(int(b.src_tbl[b.src_tbl_off[r] + t // w.src.block_tokens]))
    blk_src = w.src.num_bytes() // w.src.num_blocks
    blk_dst = w.dst.num_bytes() // w.dst.num_blocks
    assert B.pdkv_plan_block_bytes(plan) == (len(src_ids) * blk_src, len(dst_ids) * blk_dst)
    assert len(src_ids) < w.src.num_blocks            # resident prefixes are not uploaded
    B.pdkv_plan_destroy(plan)
    B.pdkv_pool_destroy(ps); B.pdkv_pool_destroy(pd)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    """There is no CPU fallback: without the built library the binding raises."""
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "libpdkv_absent.so"))
    with pytest.raises(ImportError):
        B.lib()
    with pytest.raises(ImportError):
        B.pdkv_pool_bytes(B.make_desc(0, 1, 1, 8, 2, 4, 2))


def test_workspace_plans_report_their_size():
    w = W.make_config(3, num_layers=2, n_req=6, max_len=700)
    ps, pd = _pools(w)
    b = w.batch
    plan, need = B.pdkv_plan_create_in(ps, pd, 0, b.seq_len, b.src_tbl_off, b.src_tbl, b.dst_tbl_off, b.dst_tbl,
                                       b.dst_skip)
    tiles = sum(len(B.pdkv_plan_tiles(plan, op)) for op in range(3))
    assert need == 256 + 24 * tiles
    B.pdkv_plan_destroy(plan)
    B.pdkv_pool_destroy(ps); B.pdkv_pool_destroy(pd)


def test_tile_offsets_in_petabyte_pools_need_64_bits():
    """Offsets are 64-bit end to end: pools far beyond any GPU (dry-run plans only)
    give tile offsets equal to exact Python integer arithmetic."""
    L, H, D, E, Bp, Bd = 80, 8, 128, 2, 64, 128
    nb_src, nb_dst = 50_000_000, 30_000_000
    gs = W.Geometry(W.BLOCK_MAJOR, L, H, D, E, Bp, nb_src)
    gd = W.Geometry(W.LAYER_MAJOR, L, H, D, E, Bd, nb_dst)
    assert gs.num_bytes() > 2 ** 49
    lens = np.array([200, 64, 129], np.int32)
    n_s = -(-lens.astype(np.int64) // Bp); n_d = -(-lens.astype(np.int64) // Bd)
    rng = np.random.default_rng(5)
    src_tbl = rng.choice(np.arange(nb_src - 1000, nb_src), size=int(n_s.sum()), replace=False).astype(np.int32)
    dst_tbl = rng.choice(np.arange(nb_dst - 1000, nb_dst), size=int(n_d.sum()), replace=False).astype(np.int32)
    off_s = np.concatenate([[0], np.cumsum(n_s)]).astype(np.int64)
    off_d = np.concatenate([[0], np.cumsum(n_d)]).astype(np.int64)
    ps = B.pdkv_pool_create(B.desc_of(gs), FAKE_BASE, gs.num_bytes(), 0)
    pd = B.pdkv_pool_create(B.desc_of(gd), 0x100000000000000, gd.num_bytes(), 0)
    B.pdkv_tune("tile_bytes", 32768)
    plan = B.pdkv_plan_create(ps, pd, 0, lens, off_s, src_tbl, off_d, dst_tbl)
    row, hrow = D * E, H * D * E
    tiles = B.pdkv_plan_tiles(plan, B.PDKV_OP_TRANSFER)
    copy = tiles[tiles["src_off"] >= 0]
    want = []
    for r in range(3):
        t = 0
        while t < lens[r]:
            end = min(int(lens[r]), (t // Bp + 1) * Bp, (t // Bd + 1) * Bd, t + 32768 // hrow)
            bs, bd = int(src_tbl[off_s[r] + t // Bp]), int(dst_tbl[off_d[r] + t // Bd])
            want.append((bs * (2 * L * Bp * hrow) + (t % Bp) * hrow, bd * (H * Bd * row) + (t % Bd) * row, end - t))
            t = end
    got = [(int(a), int(b), int(c)) for a, b, c in zip(copy["src_off"], copy["dst_off"], copy["ntok"])]
    assert got == want and max(a for a, _, _ in got) > 2 ** 49
    B.pdkv_plan_destroy(plan)
    B.pdkv_pool_destroy(ps); B.pdkv_pool_destroy(pd)


def test_launch_shapes_of_a_plan():
    w = W.make_config(3, num_layers=2, n_req=3, max_len=300)
    ps, pd = _pools(w)
    plan = _plan(w, ps, pd)
    try:
        for op in (B.PDKV_OP_PACK, B.PDKV_OP_UNPACK, B.PDKV_OP_TRANSFER):
            assert B.pdkv_plan_shape(plan, op) == (0, 0, 0, -1)      # built-in choice, skew by the stride rule
        B.pdkv_plan_set_shape(plan, B.PDKV_OP_TRANSFER, 384, 2, 3)
        assert B.pdkv_plan_shape(plan, B.PDKV_OP_TRANSFER) == (384, 2, 3, -1)
        assert B.pdkv_plan_shape(plan, B.PDKV_OP_PACK) == (0, 0, 0, -1)
        for bad in [(100, 1, 2), (2048, 1, 2), (256, 3, 2), (256, 4, 0), (0, 4, 2)]:
            with pytest.raises(B.PdkvError) as e:
                B.pdkv_plan_set_shape(plan, B.PDKV_OP_PACK, *bad)
            assert e.value.status == B.PDKV_ERR_INVALID_ARG
        B.pdkv_plan_set_shape(plan, B.PDKV_OP_TRANSFER, 0, 0, 0)
        assert B.pdkv_plan_shape(plan, B.PDKV_OP_TRANSFER) == (0, 0, 0, -1)
        with pytest.raises(B.PdkvError) as e:                         # a host-only plan cannot be timed
            B.pdkv_plan_autotune(plan)
        assert e.value.status == B.PDKV_ERR_INVALID_ARG
    finally:
        B.pdkv_plan_destroy(plan)
        B.pdkv_pool_destroy(ps)
        B.pdkv_pool_destroy(pd)


def test_plans_keep_the_tunables_they_were_created_with():
    """A plan copies the launch tunables when it is created: two plans made under different
    settings keep launching differently after the settings are put back, and a later
    pdkv_tune() changes neither."""
    w = W.make_config(3, num_layers=4, n_req=6, max_len=900)
    ps, pd = _pools(w)
    names = ("threads", "unroll", "ctas_per_sm", "lc_skew", "max_ctas", "debug_bounds", "src_order")
    before = {k: B.pdkv_tune_get(k) for k in names}
    try:
        default_plan = _plan(w, ps, pd)
        for k, v in dict(threads=128, unroll=2, ctas_per_sm=5, lc_skew=8, max_ctas=64, debug_bounds=1,
                         src_order=1).items():
            B.pdkv_tune(k, v)
        tuned_plan = _plan(w, ps, pd)
    finally:
        for k, v in before.items():
            B.pdkv_tune(k, v)
    L = w.src.num_layers
    a = B.pdkv_plan_launch_shape(default_plan, B.PDKV_OP_TRANSFER, 0, L)
    b = B.pdkv_plan_launch_shape(tuned_plan, B.PDKV_OP_TRANSFER, 0, L)
    # block-major 16-token blocks -> layer-major: a row-permuting copy of 256-byte rows
    assert (a["threads"], a["unroll"], a["ctas_per_sm"], a["max_ctas"], a["debug_bounds"]) == (256, 4, 2, 0, 0)
    assert a["vec_bytes"] == 32 and a["src_order"] == 0 and a["lc_skew"] == 0
    assert (b["threads"], b["unroll"], b["ctas_per_sm"], b["lc_skew"], b["max_ctas"], b["debug_bounds"],
            b["src_order"]) == (128, 2, 5, 8, 64, 1, 1)
    assert B.pdkv_plan_option(tuned_plan, "threads") == 128 and B.pdkv_plan_option(default_plan, "threads") == 0
    B.pdkv_tune("threads", 64)                  # later changes reach neither plan
    try:
        assert B.pdkv_plan_launch_shape(default_plan, B.PDKV_OP_TRANSFER, 0, L) == a
        assert B.pdkv_plan_launch_shape(tuned_plan, B.PDKV_OP_TRANSFER, 0, L) == b
    finally:
        B.pdkv_tune("threads", before["threads"])
    # a skew never exceeds the strips of the call: one layer has two
    assert B.pdkv_plan_launch_shape(tuned_plan, B.PDKV_OP_TRANSFER, 1, 2)["lc_skew"] == 2
    with pytest.raises(B.PdkvError):
        B.pdkv_plan_launch_shape(tuned_plan, B.PDKV_OP_TRANSFER, 0, L + 1)
    with pytest.raises(B.PdkvError):
        B.pdkv_plan_option(tuned_plan, "no_such_key")
    for p in (default_plan, tuned_plan):
        B.pdkv_plan_destroy(p)
    B.pdkv_pool_destroy(ps); B.pdkv_pool_destroy(pd)


def test_chooser_classes_of_copy():
    """The built-in launch choice per class of copy, read back without a GPU: flat copies,
    row-permuting copies, the 70B-shaped stride that switches the strip skew on, rows that
    are not whole 64-byte sector pairs (walked in read order), small tiles (thread groups)."""
    def shapes(w):
        ps, pd = _pools(w)
        plan = _plan(w, ps, pd)
        out = [B.pdkv_plan_launch_shape(plan, op, 0, w.src.num_layers) for op in range(3)]
        B.pdkv_plan_destroy(plan); B.pdkv_pool_destroy(ps); B.pdkv_pool_destroy(pd)
        return out

    pack, unpack, fused = shapes(W.make_config(2, n_req=2))                   # block-major both sides: flat
    assert all((s["threads"], s["unroll"], s["group_threads"]) == (512, 1, 512) for s in (pack, unpack, fused))
    assert all(s["lc_skew"] == 0 and s["src_order"] == 0 for s in (pack, unpack, fused))
    pack, unpack, fused = shapes(W.make_config(4, n_req=2))                   # 80 layers x 64 tokens: 5 x 4 MiB blocks
    assert (pack["threads"], pack["unroll"]) == (512, 1) and (fused["threads"], fused["unroll"]) == (256, 4)
    assert pack["lc_skew"] == 16 and fused["lc_skew"] == 16 and unpack["lc_skew"] == 0
    assert pack["lc_skew_shift"] == 2                                          # four 32 KiB tiles per 128 KiB strip
    pack, unpack, fused = shapes(W.make_config(3, n_req=4, head_dim=80))      # 160-byte rows
    assert pack["src_order"] == 0 and unpack["src_order"] == 1 and fused["src_order"] == 1
    assert all(s["vec_bytes"] == 32 for s in (pack, unpack, fused))
    # 27.5 KiB tiles out of the buffer: staged transpose; 20 KiB tiles out of 16-token blocks: staged transpose
    # with the strips of one block on consecutive CTAs (and therefore no strip skew)
    assert (pack["variant"], unpack["variant"], fused["variant"]) == (0, 3, 3)
    assert (unpack["lc_fastest"], fused["lc_fastest"], fused["lc_skew"]) == (0, 1, 0)
    pack, unpack, fused = shapes(W.make_config(4, n_req=2, head_dim=96))      # 192-byte rows, tiles of 24 KiB and more
    assert (pack["variant"], unpack["variant"], fused["variant"]) == (0, 3, 3)
    pack, unpack, fused = shapes(W.make_config(4, n_req=2))                   # 256-byte rows: register copy, write order
    assert (pack["variant"], unpack["variant"], fused["variant"]) == (0, 0, 0) and fused["src_order"] == 0
    pack, unpack, fused = shapes(W.make_config(3, n_req=4, elem_bytes=1))     # 128-byte rows; fused tiles of 16 KiB
    assert (fused["threads"], fused["unroll"], fused["ctas_per_sm"], fused["group_threads"], fused["src_order"]) == (256, 2, 3, 256, 1)
    assert (unpack["threads"], unpack["unroll"], unpack["ctas_per_sm"], unpack["src_order"]) == (256, 4, 2, 0)   # 32 KiB tiles
    assert (pack["threads"], pack["unroll"], pack["ctas_per_sm"]) == (256, 2, 3)                                 # flat, 16 KiB tiles
    pack, unpack, fused = shapes(W.make_config(4, n_req=2, elem_bytes=1))     # 128-byte rows in full tiles: write order
    assert unpack["src_order"] == 0 and fused["src_order"] == 0 and fused["ctas_per_sm"] == 2
    pack, unpack, fused = shapes(W.make_config(3, n_req=4, num_kv_heads=1))   # 4 KiB tiles: groups of threads
    assert fused["group_threads"] < fused["threads"] and fused["group_threads"] % 32 == 0
