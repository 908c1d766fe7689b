"""The synthetic input recipe: determinism, sizes and distributions of the five
benchmark workloads (no GPU, no transfer arithmetic)."""
import numpy as np

from paper_2408_08147_b200 import workloads as W

GIB = 1 << 30


def test_generators_are_deterministic():
    for i in range(1, 6):
        a, b = W.make_config(i), W.make_config(i)
        assert a.src == b.src and a.dst == b.dst
        for f in ("seq_len", "src_tbl_off", "src_tbl", "dst_tbl_off", "dst_tbl"):
            assert np.array_equal(getattr(a.batch, f), getattr(b.batch, f))
    assert np.array_equal(W.normal_bf16_bits(1000, 7), W.normal_bf16_bits(1000, 7))
    assert not np.array_equal(W.normal_bf16_bits(1000, 7), W.normal_bf16_bits(1000, 8))


def test_tables_are_permutations_of_free_slots():
    for i in range(1, 6):
        w = W.make_config(i)
        b = w.batch
        for tbl, off, geom in ((b.src_tbl, b.src_tbl_off, w.src), (b.dst_tbl, b.dst_tbl_off, w.dst)):
            assert len(np.unique(tbl)) == len(tbl) and tbl.min() >= 0 and tbl.max() < geom.num_blocks
            need = -(-b.seq_len.astype(np.int64) // geom.block_tokens)
            assert np.array_equal(np.diff(off), need)
        assert not np.array_equal(b.src_tbl, np.sort(b.src_tbl))          # scattered, not identity
        assert not np.intersect1d(b.src_tbl, w.src_occupied).size          # occupied slots are never handed out


def test_config_shapes_and_sizes():
    c2 = W.make_config(2)
    assert (c2.src.num_layers, c2.src.num_kv_heads, c2.src.head_dim, c2.src.elem_bytes) == (32, 8, 128, 2)
    assert c2.batch.n_req == 32 and (c2.batch.seq_len == 2048).all()
    assert c2.src.num_bytes() == 8 * GIB and c2.dst.num_bytes() == 8 * GIB and c2.src.layout == c2.dst.layout
    assert c2.src.token_bytes() == 128 * 1024

    c3 = W.make_config(3)
    assert c3.batch.n_req == 64 and c3.src.block_tokens == 16 and c3.dst.block_tokens == 128
    assert c3.batch.seq_len.min() >= 16 and c3.batch.seq_len.max() <= 8192
    assert c3.src.layout == W.BLOCK_MAJOR and c3.dst.layout == W.LAYER_MAJOR
    big = W.draw_lengths("lognormal", 20000, 1, median=1024, sigma=0.8, lo=16, hi=8192)
    assert 980 < np.median(big) < 1070
    assert 0.77 < np.log(big[(big > 16) & (big < 8192)]).std() < 0.83

    c4 = W.make_config(4)
    assert c4.src.num_layers == 80 and c4.batch.n_req == 16 and (c4.batch.seq_len == 4096).all()
    assert c4.src.block_tokens == 64 and c4.dst.block_tokens == 128
    assert c4.src.num_blocks == 1463 and c4.src_occupied.size == 438 and c4.dst.num_blocks == 512
    assert c4.dst.num_bytes() == 20 * GIB and c4.src.num_elems() > 2 ** 32
    assert c4.src.token_bytes() == 320 * 1024

    c5 = W.make_config(5)
    assert c5.batch.n_req == 1024 and c5.batch.seq_len.min() >= 64 and c5.batch.seq_len.max() <= 512
    assert 270 < c5.batch.seq_len.mean() < 306
    for bp in (16, 32, 64, 128, 256):
        assert W.make_config(5, src_block=bp).src.block_tokens == bp


def test_skip_mask_marks_a_quarter_of_leading_decode_blocks():
    w = W.make_config(5)
    b = w.batch
    assert b.dst_skip is not None and 0.22 < b.dst_skip.mean() < 0.28
    for r in range(b.n_req):
        s = b.dst_skip[b.dst_tbl_off[r]:b.dst_tbl_off[r + 1]]
        k = int(s.sum())
        assert (s[:k] == 1).all() and (s[k:] == 0).all()                  # leading blocks only


def test_values_look_like_bf16_normal_draws_and_never_hit_the_sentinel():
    bits = W.normal_bf16_bits(200000, 3)
    f = (bits.astype(np.uint32) << 16).view(np.float32)
    assert abs(f.mean()) < 0.01 and 0.98 < f.std() < 1.02
    assert not (bits == W.SENTINEL_U16).any()
    assert np.isnan((np.array([W.SENTINEL_U16], np.uint32) << 16).view(np.float32)).all()


def test_subproblem_helpers_keep_requests_intact():
    w = W.make_config(5, num_layers=1, n_req=40)
    sub, s_ids, d_ids = W.compact_subproblem(w, [3, 4, 17])
    assert np.array_equal(sub.batch.seq_len, w.batch.seq_len[[3, 4, 17]])
    assert np.array_equal(s_ids[sub.batch.src_tbl], np.concatenate(
        [w.batch.src_tbl[w.batch.src_tbl_off[r]:w.batch.src_tbl_off[r + 1]] for r in (3, 4, 17)]))
    assert sub.src.num_blocks == len(s_ids) and sub.dst.num_blocks == len(d_ids)
    part = W.slice_batch(w.batch, 5, 9)
    assert part.n_req == 4 and part.src_tbl_off[0] == 0
    assert np.array_equal(part.dst_tbl, w.batch.dst_tbl[w.batch.dst_tbl_off[5]:w.batch.dst_tbl_off[9]])
