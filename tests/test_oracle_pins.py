"""Pins for the CPU checker: it is compared with things other than itself.

* literals worked out by hand from the layout definitions (tests/golden/),
* a second statement of the same maps through numpy reshape / fancy indexing /
  transpose (no offset formula),
* brute-force enumeration of every logical coordinate on tiny inputs with
  address-coded values,
* identities: round trip, fused == unpack after pack, per-layer == whole model
  (Sec. 3.5: a layer is just another offset and length), memcpy special case,
  token and checksum conservation.
"""
import os

import numpy as np
import pytest

from paper_2408_08147_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_worked_offsets.txt")
SENT = W.SENTINEL_U16


# --------------------------------------------------------------------------
# helpers that restate the layouts through numpy views only
# --------------------------------------------------------------------------

def token_major(geom, pool, tbl, length):
    """[L][2][len][H][D] view of one request's tokens, via reshape + transpose."""
    p = pool.reshape(geom.shape())
    B = geom.block_tokens
    nb = -(-length // B)
    tbl = np.asarray(tbl[:nb], np.int64)
    L, H, D = geom.num_layers, geom.num_kv_heads, geom.head_dim
    if geom.layout == W.BLOCK_MAJOR:
        x = p[tbl]                                  # [nb][L][2][B][H][D]
        x = x.transpose(1, 2, 0, 3, 4, 5)           # [L][2][nb][B][H][D]
    else:
        x = p[:, :, tbl]                            # [L][2][nb][H][B][D]
        x = x.transpose(0, 1, 2, 4, 3, 5)           # [L][2][nb][B][H][D]
    return x.reshape(L, 2, nb * B, H, D)[:, :, :length]


def kept_mask(batch, r, granule):
    n = int(batch.seq_len[r])
    if batch.dst_skip is None:
        return np.ones(n, bool)
    ent = np.arange(n) // granule
    return batch.dst_skip[batch.dst_tbl_off[r] + ent] == 0


def numpy_pack(w, src_pool):
    out = []
    for r in range(w.batch.n_req):
        tbl = w.batch.src_tbl[w.batch.src_tbl_off[r]:w.batch.src_tbl_off[r + 1]]
        x = token_major(w.src, src_pool, tbl, int(w.batch.seq_len[r]))
        out.append(x[:, :, kept_mask(w.batch, r, w.dst.block_tokens)].reshape(-1))
    return np.concatenate(out) if out else np.zeros(0, src_pool.dtype)


def numpy_scatter(w, src_pool, dst_init):
    """Expected decode pool, built block by block with numpy assignment."""
    g = w.dst
    dst = dst_init.copy().reshape(g.shape())
    B, L, H, D = g.block_tokens, g.num_layers, g.num_kv_heads, g.head_dim
    for r in range(w.batch.n_req):
        n = int(w.batch.seq_len[r])
        nb = -(-n // B)
        stbl = w.batch.src_tbl[w.batch.src_tbl_off[r]:w.batch.src_tbl_off[r + 1]]
        x = token_major(w.src, src_pool, stbl, n)
        pad = np.zeros((L, 2, nb * B, H, D), src_pool.dtype)
        pad[:, :, :n] = x
        pad = pad.reshape(L, 2, nb, B, H, D)
        for j in range(nb):
            e = w.batch.dst_tbl_off[r] + j
            if w.batch.dst_skip is not None and w.batch.dst_skip[e]:
                continue
            b = int(w.batch.dst_tbl[e])
            blk = pad[:, :, j]                       # [L][2][B][H][D]
            if g.layout == W.BLOCK_MAJOR:
                dst[b] = blk
            else:
                dst[:, :, b] = blk.transpose(0, 1, 3, 2, 4)
    return dst.reshape(-1)


def tiny_workload(rng, *, skip=False):
    L = int(rng.integers(1, 4))
    H = int(rng.integers(1, 4))
    D = int(rng.choice([8, 16]))
    bp = int(rng.choice([1, 2, 3, 4, 8]))
    bd = int(rng.choice([1, 2, 3, 4, 8]))
    n_req = int(rng.integers(1, 5))
    lens = rng.integers(0, 20, size=n_req).astype(np.int32)
    w = W.build_workload("t", int(rng.integers(1 << 30)), num_layers=L, num_kv_heads=H,
                         head_dim=D, elem_bytes=2, seq_len=lens,
                         src_layout=int(rng.integers(2)), src_block=bp,
                         dst_layout=int(rng.integers(2)), dst_block=bd,
                         src_slack=1.5, dst_slack=1.5)
    if skip and w.batch.dst_tbl.size:
        w.batch.dst_skip = (rng.random(w.batch.dst_tbl.size) < 0.4).astype(np.uint8)
    return w


# --------------------------------------------------------------------------
# 1. hand-worked literals
# --------------------------------------------------------------------------

def _golden_rows():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                rows.append([int(v) for v in line.split()])
    return rows


def test_hand_worked_offsets(oracle):
    src_g = W.Geometry(W.BLOCK_MAJOR, 2, 2, 4, 2, 2, 5)
    dst_g = W.Geometry(W.LAYER_MAJOR, 2, 2, 4, 2, 4, 3)
    batch = W.Batch(np.array([5], np.int32), np.array([0, 3], np.int64),
                    np.array([3, 0, 4], np.int32), np.array([0, 2], np.int64),
                    np.array([2, 1], np.int32))
    assert src_g.num_elems() == 320 and dst_g.num_elems() == 384
    assert oracle.buffer_elems(batch, 4, src_g) == 160
    src = np.arange(320, dtype=np.uint16) + 1000       # value = source element + 1000
    buf = np.full(200, SENT, np.uint16)
    oracle.pack(src_g, src, batch, 4, buf)
    dst = np.full(384, SENT, np.uint16)
    oracle.unpack(dst_g, dst, batch, buf)
    dst2 = np.full(384, SENT, np.uint16)
    oracle.transfer(src_g, src, dst_g, dst2, batch)
    rows = _golden_rows()
    assert len(rows) >= 4
    for l, c, t, h, d, s_el, b_el, d_el in rows:
        assert buf[b_el] == 1000 + s_el
        assert dst[d_el] == 1000 + s_el
        assert dst2[d_el] == 1000 + s_el
    assert (buf[160:] == SENT).all()
    d6 = dst.reshape(dst_g.shape())                     # [L][2][NB][H][B][D]
    assert (d6[:, :, 1, :, 1:, :] == 0).all()           # tail slots of the last block
    assert (d6[:, :, 1, :, 0, :] != 0).all() and (d6[:, :, 1, :, 0, :] != SENT).all()
    assert (d6[:, :, 0] == SENT).all()                  # block 0 is in no table
    assert np.array_equal(dst, dst2)


# --------------------------------------------------------------------------
# 2. numpy restatement (library reshape / index / transpose)
# --------------------------------------------------------------------------

@pytest.mark.parametrize("seed", range(30))
@pytest.mark.parametrize("skip", [False, True])
def test_against_numpy_views(oracle, seed, skip):
    rng = np.random.default_rng(1000 + seed)
    w = tiny_workload(rng, skip=skip)
    src = W.fill_pool_numpy(w.src, w.seed)
    G = w.dst.block_tokens
    want_buf = numpy_pack(w, src)
    n_buf = oracle.buffer_elems(w.batch, G, w.src)
    assert n_buf == want_buf.size
    buf = np.full(n_buf + 7, SENT, np.uint16)
    oracle.pack(w.src, src, w.batch, G, buf)
    assert np.array_equal(buf[:n_buf], want_buf)
    assert (buf[n_buf:] == SENT).all()

    dst0 = W.sentinel_pool_numpy(w.dst)
    want_dst = numpy_scatter(w, src, dst0)
    got = dst0.copy()
    oracle.unpack(w.dst, got, w.batch, buf)
    assert np.array_equal(got, want_dst)
    got2 = dst0.copy()
    oracle.transfer(w.src, src, w.dst, got2, w.batch)
    assert np.array_equal(got2, want_dst)


def test_config1_against_numpy_views(oracle):
    w = W.make_config(1)
    src = W.fill_pool_numpy(w.src, w.seed)
    buf = np.zeros(oracle.buffer_elems(w.batch, 32, w.src), np.uint16)
    oracle.pack(w.src, src, w.batch, 32, buf)
    assert np.array_equal(buf, numpy_pack(w, src))
    dst0 = W.sentinel_pool_numpy(w.dst)
    got = dst0.copy()
    oracle.transfer(w.src, src, w.dst, got, w.batch, threads=4)
    assert np.array_equal(got, numpy_scatter(w, src, dst0))


# --------------------------------------------------------------------------
# 3. brute force over every logical coordinate, address-coded values
# --------------------------------------------------------------------------

def _code(r, l, c, t, h, d):
    return (r * 7919 + l * 1543 + c * 769 + t * 193 + h * 53 + d * 11 + 1) % 32749 + 1


@pytest.mark.parametrize("seed", range(12))
def test_brute_force_enumeration(oracle, seed):
    rng = np.random.default_rng(77 + seed)
    w = tiny_workload(rng, skip=bool(seed % 2))
    sg, dg, bt = w.src, w.dst, w.batch
    src6 = np.full(sg.shape(), SENT, np.uint16)

    def idx(g, b, l, c, tt, h, d):
        return (b, l, c, tt, h, d) if g.layout == W.BLOCK_MAJOR else (l, c, b, h, tt, d)

    coords = []
    for r in range(bt.n_req):
        for t in range(int(bt.seq_len[r])):
            bs = int(bt.src_tbl[bt.src_tbl_off[r] + t // sg.block_tokens])
            for l in range(sg.num_layers):
                for c in range(2):
                    for h in range(sg.num_kv_heads):
                        for d in range(sg.head_dim):
                            src6[idx(sg, bs, l, c, t % sg.block_tokens, h, d)] = _code(r, l, c, t, h, d)
                            coords.append((r, l, c, t, h, d))
    src = src6.reshape(-1)
    dst = W.sentinel_pool_numpy(dg)
    oracle.transfer(sg, src, dg, dst, bt)
    d6 = dst.reshape(dg.shape())
    reached = np.zeros(dg.shape(), bool)
    n_kept = 0
    for (r, l, c, t, h, d) in coords:
        e = bt.dst_tbl_off[r] + t // dg.block_tokens
        if bt.dst_skip is not None and bt.dst_skip[e]:
            continue
        i = idx(dg, int(bt.dst_tbl[e]), l, c, t % dg.block_tokens, h, d)
        assert d6[i] == _code(r, l, c, t, h, d)
        reached[i] = True
        n_kept += 1
    assert reached.sum() == n_kept                       # one writer per element
    # everything not reached is either a zeroed tail slot or untouched sentinel
    rest = d6[~reached]
    assert np.isin(rest, [0, SENT]).all()
    n_zero = 0
    for r in range(bt.n_req):
        n = int(bt.seq_len[r])
        nb = -(-n // dg.block_tokens)
        if nb and not (bt.dst_skip is not None and bt.dst_skip[bt.dst_tbl_off[r] + nb - 1]):
            n_zero += (nb * dg.block_tokens - n) * 2 * dg.num_layers * dg.num_kv_heads * dg.head_dim
    assert (rest == 0).sum() == n_zero

    # the buffer holds exactly the kept coordinates, in [l][c][t][h][d] order per request
    G = dg.block_tokens
    buf = np.full(oracle.buffer_elems(bt, G, sg), SENT, np.uint16)
    oracle.pack(sg, src, bt, G, buf)
    want = []
    for r in range(bt.n_req):
        for l in range(sg.num_layers):
            for c in range(2):
                for t in range(int(bt.seq_len[r])):
                    if bt.dst_skip is not None and bt.dst_skip[bt.dst_tbl_off[r] + t // G]:
                        continue
                    for h in range(sg.num_kv_heads):
                        for d in range(sg.head_dim):
                            want.append(_code(r, l, c, t, h, d))
    assert buf.tolist() == want


# --------------------------------------------------------------------------
# 4..7 identities
# --------------------------------------------------------------------------

@pytest.mark.parametrize("seed", range(10))
def test_round_trip_and_fused_identity(oracle, seed):
    rng = np.random.default_rng(500 + seed)
    w = tiny_workload(rng, skip=bool(seed % 2))
    G = w.dst.block_tokens
    src = W.fill_pool_numpy(w.src, w.seed)
    n = oracle.buffer_elems(w.batch, G, w.src)
    buf = np.zeros(n, np.uint16)
    oracle.pack(w.src, src, w.batch, G, buf)
    dst = W.sentinel_pool_numpy(w.dst)
    oracle.unpack(w.dst, dst, w.batch, buf)
    fused = W.sentinel_pool_numpy(w.dst)
    oracle.transfer(w.src, src, w.dst, fused, w.batch)
    assert np.array_equal(dst, fused)
    # pack the decode pool again through its own table: same bytes come back
    back = W.Batch(w.batch.seq_len, w.batch.dst_tbl_off, w.batch.dst_tbl,
                   w.batch.dst_tbl_off, w.batch.dst_tbl, w.batch.dst_skip)
    buf2 = np.zeros(n, np.uint16)
    oracle.pack(w.dst, dst, back, G, buf2)
    assert np.array_equal(buf, buf2)
    # token conservation
    kept = oracle.kept_tokens(w.batch, G)
    assert n == kept.sum() * 2 * w.src.num_layers * w.src.num_kv_heads * w.src.head_dim
    skipped = w.batch.seq_len.sum() - kept.sum()
    assert skipped >= 0
    if w.batch.dst_skip is None:
        assert skipped == 0
    # checksum conservation: buffer and owned decode region carry the same values
    owned = dst[(dst != SENT)]
    assert int(buf.astype(np.uint64).sum()) == int(owned.astype(np.uint64).sum())


@pytest.mark.parametrize("seed", range(6))
def test_same_geometry_gives_back_source(oracle, seed):
    rng = np.random.default_rng(900 + seed)
    w = W.with_dst_geometry_of_src(tiny_workload(rng))
    src = W.fill_pool_numpy(w.src, w.seed)
    G = w.dst.block_tokens
    buf = np.zeros(oracle.buffer_elems(w.batch, G, w.src), np.uint16)
    oracle.pack(w.src, src, w.batch, G, buf)
    dst = W.sentinel_pool_numpy(w.dst)
    oracle.unpack(w.dst, dst, w.batch, buf)
    for r in range(w.batch.n_req):
        tbl = w.batch.src_tbl[w.batch.src_tbl_off[r]:w.batch.src_tbl_off[r + 1]]
        n = int(w.batch.seq_len[r])
        assert np.array_equal(token_major(w.src, src, tbl, n), token_major(w.dst, dst, tbl, n))


def test_memcpy_special_case(oracle):
    # block-major on both sides, equal block size, identity tables, full blocks
    lens = np.array([8, 16, 4], np.int32)
    g = W.Geometry(W.BLOCK_MAJOR, 3, 2, 8, 2, 4, 7)
    off = np.array([0, 2, 6, 7], np.int64)
    tbl = np.arange(7, dtype=np.int32)
    bt = W.Batch(lens, off, tbl, off, tbl)
    src = W.fill_pool_numpy(g, 3)
    dst = W.sentinel_pool_numpy(g)
    oracle.transfer(g, src, g, dst, bt)
    assert dst.tobytes() == src.tobytes()


@pytest.mark.parametrize("seed", range(6))
def test_per_layer_equals_whole_model(oracle, seed):
    rng = np.random.default_rng(300 + seed)
    w = tiny_workload(rng, skip=bool(seed % 2))
    G = w.dst.block_tokens
    src = W.fill_pool_numpy(w.src, w.seed)
    n = oracle.buffer_elems(w.batch, G, w.src)
    whole = np.full(n, SENT, np.uint16)
    oracle.pack(w.src, src, w.batch, G, whole)
    piece = np.full(n, SENT, np.uint16)
    offs = oracle.request_offsets(w.batch, G, w.src)
    kept = oracle.kept_tokens(w.batch, G)
    HD = w.src.num_kv_heads * w.src.head_dim
    for l in range(w.src.num_layers):
        before = piece.copy()
        oracle.pack(w.src, src, w.batch, G, piece, layers=(l, l + 1))
        changed = np.flatnonzero(before != piece)
        # layer l of request r occupies [off_r + l*2*n_r*H*D, + 2*n_r*H*D)
        ok = np.zeros(n, bool)
        for r in range(w.batch.n_req):
            a = offs[r] + l * 2 * kept[r] * HD
            ok[a:a + 2 * kept[r] * HD] = True
        assert ok[changed].all()
    assert np.array_equal(whole, piece)
    d_whole = W.sentinel_pool_numpy(w.dst)
    oracle.unpack(w.dst, d_whole, w.batch, whole)
    d_piece = W.sentinel_pool_numpy(w.dst)
    for l in range(w.dst.num_layers):
        oracle.unpack(w.dst, d_piece, w.batch, whole, layers=(l, l + 1))
    assert np.array_equal(d_whole, d_piece)


def subranges_agree_with_numpy(o, w, src, l0, l1, r0, r1) -> bool:
    """Layer range [l0,l1) and request range [r0,r1) of pack, unpack and the fused transfer
    against the numpy restatement: exactly those layers of exactly those requests move, at
    the offsets of a whole call; everything else keeps the sentinel."""
    G = w.dst.block_tokens
    L, HD = w.src.num_layers, w.src.num_kv_heads * w.src.head_dim
    want_buf_all = numpy_pack(w, src)
    n = want_buf_all.size
    # per-request extents of the buffer from the numpy statement alone
    sizes = [int(kept_mask(w.batch, r, G).sum()) * 2 * L * HD for r in range(w.batch.n_req)]
    starts = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    want_buf = np.full(n, SENT, np.uint16)
    for r in range(r0, r1):
        per_layer = sizes[r] // L
        a = starts[r] + l0 * per_layer
        want_buf[a:a + (l1 - l0) * per_layer] = want_buf_all[a:a + (l1 - l0) * per_layer]
    got_buf = np.full(n, SENT, np.uint16)
    o.pack(w.src, src, w.batch, G, got_buf, layers=(l0, l1), requests=(r0, r1))
    if not np.array_equal(got_buf, want_buf):
        return False
    # decode pool: the chosen requests alone, through the numpy scatter, then only the chosen layers
    d0 = W.sentinel_pool_numpy(w.dst)
    part = W.Workload(w.name, w.seed, w.src, w.dst, W.slice_batch(w.batch, r0, r1))
    full = numpy_scatter(part, src, d0).reshape(w.dst.shape())
    want = d0.copy().reshape(w.dst.shape())
    if w.dst.layout == W.BLOCK_MAJOR:
        want[:, l0:l1] = full[:, l0:l1]
    else:
        want[l0:l1] = full[l0:l1]
    want = want.reshape(-1)
    got = d0.copy()
    o.unpack(w.dst, got, w.batch, want_buf_all, layers=(l0, l1), requests=(r0, r1))
    if not np.array_equal(got, want):
        return False
    got = d0.copy()
    o.transfer(w.src, src, w.dst, got, w.batch, layers=(l0, l1), requests=(r0, r1))
    return bool(np.array_equal(got, want))


@pytest.mark.parametrize("seed", range(16))
def test_layer_and_request_subranges_against_numpy(oracle, seed):
    rng = np.random.default_rng(4200 + seed)
    w = tiny_workload(rng, skip=bool(seed % 2))
    src = W.fill_pool_numpy(w.src, w.seed)
    L, R = w.src.num_layers, w.batch.n_req
    l0 = int(rng.integers(0, L))
    l1 = int(rng.integers(l0, L + 1))
    r0 = int(rng.integers(0, R))
    r1 = int(rng.integers(r0, R + 1))
    assert subranges_agree_with_numpy(oracle, w, src, l0, l1, r0, r1)
    assert subranges_agree_with_numpy(oracle, w, src, 0, L, 0, R)
    if L > 1 and R > 1:
        assert subranges_agree_with_numpy(oracle, w, src, L - 1, L, R - 1, R)


def test_threads_and_request_ranges_agree(oracle):
    w = W.make_config(5, num_layers=2, n_req=24)
    src = W.fill_pool_numpy(w.src, w.seed)
    a = W.sentinel_pool_numpy(w.dst)
    b = a.copy()
    oracle.transfer(w.src, src, w.dst, a, w.batch)
    oracle.transfer(w.src, src, w.dst, b, w.batch, threads=5)
    assert np.array_equal(a, b)
    assert w.batch.dst_skip is not None and w.batch.dst_skip.any()


def test_source_tail_and_foreign_blocks_never_read(oracle):
    # paint everything the path must not read with the sentinel; no sentinel may
    # reach the buffer
    w = W.make_config(4, num_layers=1, n_req=3, max_len=100)
    src = W.sentinel_pool_numpy(w.src)
    s6 = src.reshape(w.src.shape())
    vals = W.normal_bf16_bits(src.size, 5).reshape(w.src.shape())
    B = w.src.block_tokens
    for r in range(w.batch.n_req):
        n = int(w.batch.seq_len[r])
        for j in range(-(-n // B)):
            b = int(w.batch.src_tbl[w.batch.src_tbl_off[r] + j])
            k = min(B, n - j * B)
            s6[b, :, :, :k] = vals[b, :, :, :k]
    assert w.src_occupied.size > 0
    buf = np.zeros(oracle.buffer_elems(w.batch, w.dst.block_tokens, w.src), np.uint16)
    oracle.pack(w.src, src, w.batch, w.dst.block_tokens, buf)
    assert (buf != SENT).all()
