"""The pins must notice plausible mistakes in the CPU checker.  Each case
plants one mistake in a *copy* of the checker's C source (a swapped stride, a
dropped factor, an off-by-one, a wrong table index), builds it, and runs the
same battery of independent checks the real checker passes: hand-worked
literals, the numpy reshape/transpose restatement, and the per-layer identity.
Every mutant has to fail the battery; the unmodified copy has to pass."""
import importlib.util
import os
import shutil
import subprocess
import sys

import numpy as np
import pytest

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
from paper_2408_08147_b200 import workloads as W
from test_oracle_pins import _golden_rows, numpy_pack, numpy_scatter, subranges_agree_with_numpy, tiny_workload

ORACLE_DIR = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "oracle")
SENT = W.SENTINEL_U16

MUTATIONS = {
    "block-major: token and head strides swapped":
        ("return ((((b * g->L + l) * 2 + c) * g->B + tt) * g->H + h) * g->D + d;",
         "return ((((b * g->L + l) * 2 + c) * g->H + h) * g->B + tt) * g->D + d;"),
    "layer-major: token and head strides swapped":
        ("return ((((l * 2 + c) * g->NB + b) * g->H + h) * g->B + tt) * g->D + d;",
         "return ((((l * 2 + c) * g->NB + b) * g->B + tt) * g->H + h) * g->D + d;"),
    "layer-major: K/V outside the layer":
        ("return ((((l * 2 + c) * g->NB + b)", "return ((((c * g->L + l) * g->NB + b)"),
    "buffer indexed by token instead of rank among kept tokens":
        ("buf_off(off_r, n_r, l, c, rank, h, d, sg->H, sg->D)", "buf_off(off_r, n_r, l, c, t, h, d, sg->H, sg->D)"),
    "buffer: head and dim order swapped":
        ("return off_r + ((l * 2 + c) * n_r + rank) * H * D + h * D + d;",
         "return off_r + ((l * 2 + c) * n_r + rank) * H * D + d * H + h;"),
    "tail zeroing off by one":
        ("if ((nblk - 1) * dg->B + tt < len)", "if ((nblk - 1) * dg->B + tt <= len)"),
    "tail zeroing dropped":
        ("    if (nblk == 0)\n        return;", "    if (nblk >= 0)\n        return;"),
    "skip mask inverted":
        ("return bt->skip[bt->dst_tbl_off[r] + t / bt->G] == 0;", "return bt->skip[bt->dst_tbl_off[r] + t / bt->G] != 0;"),
    "request offset drops the K/V factor":
        ("off += 2 * (int64_t)L * okv_kept_tokens(bt, q) * H * D;", "off += (int64_t)L * okv_kept_tokens(bt, q) * H * D;"),
    "fused: decode slot computed with the prefill block size":
        ("pool_off(dg, bd, l, c, t % dg->B, h, d)", "pool_off(dg, bd, l, c, t % sg->B, h, d)"),
    "pack: prefill table indexed with the skip granule":
        ("const int64_t b = bt->src_tbl[bt->src_tbl_off[r] + t / sg->B];\n                    const int64_t tt = t % sg->B;",
         "const int64_t b = bt->src_tbl[bt->src_tbl_off[r] + t / bt->G];\n                    const int64_t tt = t % sg->B;"),
    "unpack ignores the layer range":
        ("void okv_unpack(const okv_geom *dg, uint8_t *dst, const okv_batch *bt,\n                const uint8_t *buf, int l0, int l1, int r0, int r1)\n{",
         "void okv_unpack(const okv_geom *dg, uint8_t *dst, const okv_batch *bt,\n                const uint8_t *buf, int l0, int l1, int r0, int r1)\n{\n    l0 = 0; l1 = dg->L;"),
    "fused transfer ignores the layer range":
        ("                  uint8_t *dst, const okv_batch *bt, int l0, int l1, int r0, int r1)\n{\n    const int E = sg->E;",
         "                  uint8_t *dst, const okv_batch *bt, int l0, int l1, int r0, int r1)\n{\n    const int E = sg->E;\n    l0 = 0; l1 = sg->L;"),
    "pack ignores the request range":
        ("              uint8_t *buf, int l0, int l1, int r0, int r1)\n{\n    const int E = sg->E;",
         "              uint8_t *buf, int l0, int l1, int r0, int r1)\n{\n    const int E = sg->E;\n    r0 = 0; r1 = bt->n_req;"),
    "unpack: tail zeroing ignores the request range":
        ("        zero_tail(dg, dst, bt, r, l0, l1);\n    }\n}\n\n/* Blocks -> blocks",
         "    }\n    for (int r = 0; r < bt->n_req; ++r)\n        zero_tail(dg, dst, bt, r, l0, l1);\n}\n\n/* Blocks -> blocks"),
}


def _make_copy(tmp_path, name, edit=None):
    d = tmp_path / name
    d.mkdir()
    for f in ("pdkv_oracle.c", "pdkv_oracle.py"):
        shutil.copy(os.path.join(ORACLE_DIR, f), d / f)
    if edit:
        src = (d / "pdkv_oracle.c").read_text()
        assert src.count(edit[0]) >= 1, f"mutation target not found: {edit[0][:50]}"
        (d / "pdkv_oracle.c").write_text(src.replace(edit[0], edit[1]))
    return str(d)


def _load(copy_dir):
    spec = importlib.util.spec_from_file_location("oracle_copy", os.path.join(copy_dir, "pdkv_oracle.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    mod.build(force=True)
    return mod


def _battery_in_child(copy_dir) -> bool:
    """A mutant may index out of bounds and crash: run it in its own process;
    a crash counts as "noticed"."""
    r = subprocess.run([sys.executable, os.path.abspath(__file__), copy_dir], capture_output=True, timeout=600)
    return r.returncode == 0


def battery(o) -> bool:
    """True iff the checker `o` agrees with every independent statement below."""
    # hand-worked literals
    src_g = W.Geometry(W.BLOCK_MAJOR, 2, 2, 4, 2, 2, 5)
    dst_g = W.Geometry(W.LAYER_MAJOR, 2, 2, 4, 2, 4, 3)
    batch = W.Batch(np.array([5], np.int32), np.array([0, 3], np.int64), np.array([3, 0, 4], np.int32),
                    np.array([0, 2], np.int64), np.array([2, 1], np.int32))
    if o.buffer_elems(batch, 4, src_g) != 160:
        return False
    src = np.arange(320, dtype=np.uint16) + 1000
    buf = np.full(160, SENT, np.uint16)
    o.pack(src_g, src, batch, 4, buf)
    dst = np.full(384, SENT, np.uint16)
    o.unpack(dst_g, dst, batch, buf)
    dst2 = np.full(384, SENT, np.uint16)
    o.transfer(src_g, src, dst_g, dst2, batch)
    for l, c, t, h, d, s_el, b_el, d_el in _golden_rows():
        if buf[b_el] != 1000 + s_el or dst[d_el] != 1000 + s_el or dst2[d_el] != 1000 + s_el:
            return False
    # numpy restatement on random tiny workloads, with and without skip masks
    for seed in range(24):
        rng = np.random.default_rng(31000 + seed)
        w = tiny_workload(rng, skip=bool(seed % 2))
        G = w.dst.block_tokens
        s = W.fill_pool_numpy(w.src, w.seed)
        want_buf = numpy_pack(w, s)
        if o.buffer_elems(w.batch, G, w.src) != want_buf.size:
            return False
        b = np.full(want_buf.size, SENT, np.uint16)
        o.pack(w.src, s, w.batch, G, b)
        if not np.array_equal(b, want_buf):
            return False
        d0 = W.sentinel_pool_numpy(w.dst)
        want_dst = numpy_scatter(w, s, d0)
        for fn in (lambda out: o.unpack(w.dst, out, w.batch, b), lambda out: o.transfer(w.src, s, w.dst, out, w.batch)):
            got = d0.copy()
            fn(got)
            if not np.array_equal(got, want_dst):
                return False
        # a single layer touches only that layer of the decode pool
        if w.dst.num_layers > 1:
            got = d0.copy()
            o.unpack(w.dst, got, w.batch, b, layers=(0, 1))
            g6, w6 = got.reshape(w.dst.shape()), want_dst.reshape(w.dst.shape())
            lay = (slice(None), slice(0, 1)) if w.dst.layout == W.BLOCK_MAJOR else (slice(0, 1),)
            rest = (slice(None), slice(1, None)) if w.dst.layout == W.BLOCK_MAJOR else (slice(1, None),)
            if not np.array_equal(g6[lay], w6[lay]) or not (g6[rest] == SENT).all():
                return False
        # layer and request sub-ranges of all three calls
        L, R = w.src.num_layers, w.batch.n_req
        l0 = int(rng.integers(0, L)); l1 = int(rng.integers(l0, L + 1))
        r0 = int(rng.integers(0, R)); r1 = int(rng.integers(r0, R + 1))
        if not subranges_agree_with_numpy(o, w, s, l0, l1, r0, r1):
            return False
        if L > 1 and R > 1 and not subranges_agree_with_numpy(o, w, s, L - 1, L, R - 1, R):
            return False
    return True


def test_unmodified_copy_passes(tmp_path):
    assert _battery_in_child(_make_copy(tmp_path, "clean"))


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(tmp_path, name):
    assert not _battery_in_child(_make_copy(tmp_path, "m", MUTATIONS[name])), f"the pins do not notice: {name}"


if __name__ == "__main__":
    sys.exit(0 if battery(_load(sys.argv[1])) else 1)
