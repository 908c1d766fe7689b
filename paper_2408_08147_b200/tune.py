"""Sweep the library's launch tunables on one workload and print what is fastest.

The defaults were chosen from sweeps like this one on Llama-shaped batches; a
deployment with another geometry (head count, block sizes, element size) can
re-run it and pin the winners with ``pdkv_tune``::

    python -m paper_2408_08147_b200.tune --config 3 --kv-heads 2
    python -m paper_2408_08147_b200.tune --config 4 --ops fused --grid wide

(``pdkv_plan_autotune`` does a short version of this inside the library, per
plan, for the launch shape alone.)

Timing is bench-like: the selected operations are issued back to back on one
stream and each one's CUDA-event time is averaged over ``--reps`` rounds.
"""
from __future__ import annotations

import argparse
import itertools
import sys

GRIDS = {
    "quick": dict(threads=[0, 256, 512], unroll=[0, 1, 4], ctas_per_sm=[2, 4], tile_bytes=[32768, 65536],
                  lc_fastest=[0]),
    "wide": dict(threads=[256, 512, 1024], unroll=[1, 2, 4], ctas_per_sm=[1, 2, 4],
                 tile_bytes=[16384, 32768, 65536, 131072], lc_fastest=[0, 1]),
    "order": dict(threads=[0], unroll=[0], ctas_per_sm=[2], tile_bytes=[32768, 131072],
                  lc_fastest=[0, 1], chunked=[0, 1]),
    "skew": dict(threads=[0], unroll=[0], ctas_per_sm=[2], tile_bytes=[32768], lc_skew=[-1, 0, 4, 8, 16, 32],
                 lc_skew_shift=[0, 1, 2, 3]),
    "bulk": dict(variant=[1, 2], tile_bytes=[8192, 16384, 32768], stages=[2, 3, 4], ctas_per_sm=[2, 3, 4, 6, 8],
                 lc_fastest=[0]),
}
RESET = dict(variant=0, threads=0, unroll=0, group_threads=0, ctas_per_sm=2, tile_bytes=32768, lc_fastest=0, lc_skew=-1, lc_skew_shift=0,
             chunked=0, stages=3, max_ctas=0)


def main(argv=None) -> int:
    import torch

    from . import binding as B
    from . import workloads as W
    from .session import TransferSession

    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--layouts", default="", help="two letters, e.g. AB")
    ap.add_argument("--src-block", type=int, default=0)
    ap.add_argument("--n-req", type=int, default=0)
    ap.add_argument("--kv-heads", type=int, default=0)
    ap.add_argument("--elem-bytes", type=int, default=0)
    ap.add_argument("--head-dim", type=int, default=0)
    ap.add_argument("--num-layers", type=int, default=0)
    ap.add_argument("--ops", default="pack,unpack,fused")
    ap.add_argument("--grid", default="quick", choices=sorted(GRIDS))
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--top", type=int, default=8)
    a = ap.parse_args(argv)
    if not torch.cuda.is_available():
        print("needs a CUDA device", file=sys.stderr)
        return 2

    kw = {}
    for key, val in (("src_block", a.src_block), ("n_req", a.n_req), ("num_kv_heads", a.kv_heads),
                     ("elem_bytes", a.elem_bytes), ("head_dim", a.head_dim), ("num_layers", a.num_layers)):
        if val:
            kw[key] = val
    if a.layouts:
        kw["src_layout"], kw["dst_layout"] = "AB".index(a.layouts[0]), "AB".index(a.layouts[1])
    w = W.make_config(a.config, **kw)
    src_t = torch.empty(w.src.num_bytes(), dtype=torch.uint8, device="cuda")
    W.fill_pool_torch(src_t, w.seed)
    dst_t = torch.zeros(w.dst.num_bytes(), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    ops = a.ops.split(",")
    op_id = {"pack": B.PDKV_OP_PACK, "unpack": B.PDKV_OP_UNPACK, "fused": B.PDKV_OP_TRANSFER}

    grid = GRIDS[a.grid]
    keys = list(grid)
    rows, buf_t = [], None
    try:
        for combo in itertools.product(*[grid[k] for k in keys]):
            cfg = dict(zip(keys, combo))
            if cfg.get("variant", 0) and (128 + cfg["stages"] * cfg["tile_bytes"]) * cfg["ctas_per_sm"] > 225 * 1024:
                continue
            for k, v in {**RESET, **cfg}.items():
                B.pdkv_tune(k, v)
            with TransferSession(w.src, src_t, w.dst, dst_t, w.batch, stream.cuda_stream) as s:
                if buf_t is None:
                    buf_t = torch.zeros(max(16, s.buffer_bytes), dtype=torch.uint8, device="cuda")
                fns = {"pack": lambda: s.pack(buf_t), "unpack": lambda: s.unpack(buf_t), "fused": s.transfer}
                nbytes = {o: sum(s.traffic(op_id[o])) for o in ops}
                with torch.cuda.stream(stream):
                    for o in ops:
                        fns[o]()
                    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(len(ops) + 1)]
                           for _ in range(a.reps)]
                    for r in range(a.reps):
                        for i, o in enumerate(ops):
                            evs[r][i].record(stream)
                            fns[o]()
                        evs[r][len(ops)].record(stream)
                torch.cuda.synchronize()
                gbps = [nbytes[o] / (sum(evs[r][i].elapsed_time(evs[r][i + 1]) for r in range(a.reps)) / a.reps) / 1e6
                        for i, o in enumerate(ops)]
            rows.append((cfg, gbps))
    finally:
        for k, v in RESET.items():
            B.pdkv_tune(k, v)

    print(f"workload: {w.name}  L={w.src.num_layers} H={w.src.num_kv_heads} D={w.src.head_dim} "
          f"E={w.src.elem_bytes}  prefill B={w.src.block_tokens} layout {'AB'[w.src.layout]}  "
          f"decode B={w.dst.block_tokens} layout {'AB'[w.dst.layout]}  ({len(rows)} settings, 0 = automatic)")
    for i, o in enumerate(ops):
        print(f"\nfastest for {o} (GB/s of payload read + written):")
        for cfg, g in sorted(rows, key=lambda r: -r[1][i])[:a.top]:
            print(f"  {g[i]:8.1f}   " + "  ".join(f"{k}={v}" for k, v in cfg.items()))
    return 0


if __name__ == "__main__":
    sys.exit(main())
