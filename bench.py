#!/usr/bin/env python
"""Benchmark of the paged-KVCache transfer path.

One *step* is one pass of the whole hot path over one batch: pack (blocks ->
contiguous buffer), unpack (buffer -> decode blocks) and the fused
blocks-to-blocks transfer, each one library call.  The reported value is the
algorithmic traffic of a step (payload read + payload written + zero padding
written, summed over the three calls) divided by the device time of the step.

    python bench.py --gpus 1 --steps 50 --warmup 5            # this library
    python bench.py --impl reference --steps 3 --warmup 1      # CPU checker arm

Prints exactly one JSON line on stdout (rank 0).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "KV pack+unpack+fused transfer throughput (algorithmic bytes read+written)"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0
KERNEL_SOURCE = os.path.join(ROOT, "paper_2408_08147_b200", "csrc", "pdkv_copy_kernel.cuh")   # device code only

# DRAM traffic per launch from ncu (dram__bytes_read.sum + dram__bytes_write.sum),
# keyed by (workload, op); valid only while the kernel source hashes to KERNEL_SHA.
# Config 2 was captured on a 1/8-size case (4 of 32 requests; profiles/copy_tiles_kernel_config2_small_ncu_full.md)
# and is scaled by 8; config 4 on 2 of 16 requests x 16 of 80 layers (profiles/copy_tiles_kernel_config4_small_ncu_full.md),
# scaled by 40: traffic is proportional to the tokens and layers moved (read = algorithmic to 4 digits, write 4-9% lower
# because the last dirty lines are still in L2 when the short captured kernel ends).
NCU_TRAFFIC: dict = {(2, "pack"): 8 * (1.073972e9 + 1.027700e9), (2, "unpack"): 8 * (1.073934e9 + 1.030297e9),
                     (2, "fused"): 8 * (1.073925e9 + 1.030007e9),
                     (4, "pack"): 40 * (536.960000e6 + 488.121856e6), (4, "unpack"): 40 * (536.996352e6 + 488.964864e6),
                     (4, "fused"): 40 * (536.962816e6 + 487.982848e6)}
NCU_KERNEL_SHA = "5333b1c77fb50ab9"


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def kernel_sha() -> str:
    with open(KERNEL_SOURCE, "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()[:16]


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ---------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------

class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while a region runs
    (read-only queries; nothing is set)."""

    def __init__(self, index: int, period_s: float = 0.02):
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml

            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception as e:  # pragma: no cover
            log(f"[bench] NVML unavailable: {e}")
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thr:
            self._thr.join()

    def summary(self):
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ---------------------------------------------------------------------------
# distributed plumbing (one process per GPU; no data-path collective)
# ---------------------------------------------------------------------------

def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), \
        int(os.environ.get("WORLD_SIZE", 1))


def dist_init(backend: str):
    import torch.distributed as dist

    rank, _, world = dist_env()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world


def barrier():
    import torch.distributed as dist

    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def all_ranks_agree(flag: bool, device=None) -> bool:
    """True only if every rank passed True (a collective decision, so that all ranks
    take the same branch around later barriers)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()):
        return bool(flag)
    t = torch.tensor([1 if flag else 0], dtype=torch.int32, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MIN)
    return bool(t.item())


def reduce_step_time(ms_local: float, units_local: float, device=None):
    """Max of the per-rank times and sum of the per-rank units, on every rank."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()):
        return ms_local, units_local
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


# ---------------------------------------------------------------------------
# workload on the device
# ---------------------------------------------------------------------------

def workload_name(w):
    s, d = w.src, w.dst
    lay = {0: "block-major", 1: "layer-major"}
    return (f"{w.name}: L={s.num_layers} H={s.num_kv_heads} D={s.head_dim} E={s.elem_bytes} "
            f"{w.batch.n_req} req, {int(w.batch.seq_len.sum())} tokens total; prefill {lay[s.layout]} "
            f"B={s.block_tokens} NB={s.num_blocks}; decode {lay[d.layout]} B={d.block_tokens} "
            f"NB={d.num_blocks}")


def alloc_pools(w, torch, seed_offset=0):
    from paper_2408_08147_b200 import workloads as W

    src_t = torch.empty(w.src.num_bytes(), dtype=torch.uint8, device="cuda")
    W.fill_pool_torch(src_t, w.seed + seed_offset)
    dst_t = torch.empty(w.dst.num_bytes(), dtype=torch.uint8, device="cuda")
    dst_t.view(torch.int16).fill_(W.SENTINEL_U16 - 65536 if W.SENTINEL_U16 > 32767 else W.SENTINEL_U16)
    return src_t, dst_t


def token_major_torch(geom, pool_t, tbl, length, torch):
    """[L][2][len][H][D] view-copy of one request, through reshape/index/permute
    (an independent cross-check of the kernels; not the CPU checker)."""
    v = pool_t.view(torch.uint8).view(*geom.shape(), geom.elem_bytes)   # last axis: the bytes of one element
    B = geom.block_tokens
    nb = -(-length // B)
    idx = torch.as_tensor(tbl[:nb].astype("int64"), device=pool_t.device)
    if geom.layout == 0:
        x = v[idx].permute(1, 2, 0, 3, 4, 5, 6)
    else:
        x = v[:, :, idx].permute(0, 1, 2, 4, 3, 5, 6)
    L, H, D = geom.num_layers, geom.num_kv_heads, geom.head_dim
    return x.reshape(L, 2, nb * B, H, D * geom.elem_bytes)[:, :, :length]


def sanity_check(w, src_t, dst_t, torch) -> bool:
    """A few requests' tokens must be identical in both pools after a transfer."""
    b = w.batch
    if b.dst_skip is not None:
        return True
    for r in sorted({0, b.n_req // 2, b.n_req - 1}):
        n = int(b.seq_len[r])
        s = token_major_torch(w.src, src_t, b.src_tbl[b.src_tbl_off[r]:b.src_tbl_off[r + 1]], n, torch)
        d = token_major_torch(w.dst, dst_t, b.dst_tbl[b.dst_tbl_off[r]:b.dst_tbl_off[r + 1]], n, torch)
        if not torch.equal(s, d):
            return False
    return True


# ---------------------------------------------------------------------------
# CPU checker legs
# ---------------------------------------------------------------------------

def oracle_step(O, sub, src_np, dst_np, buf_np, threads):
    G = sub.dst.block_tokens
    O.pack(sub.src, src_np, sub.batch, G, buf_np, threads=threads)
    O.unpack(sub.dst, dst_np, sub.batch, buf_np, threads=threads)
    O.transfer(sub.src, src_np, sub.dst, dst_np, sub.batch, threads=threads)


def op_bytes_of(w):
    """Algorithmic bytes of each operation, from the batch alone: pack reads and writes
    the kept payload; unpack and fused also write the zero padding of unskipped last blocks."""
    import numpy as np

    tok = w.src.token_bytes()
    b = w.batch
    lens = b.seq_len.astype(np.int64)
    Bd = w.dst.block_tokens
    nblk = -(-lens // Bd)
    if b.dst_skip is None:
        kept = int(lens.sum())
        pad = int((nblk * Bd - lens).sum())
    else:
        kept = pad = 0
        for r in range(b.n_req):
            sk = b.dst_skip[b.dst_tbl_off[r]:b.dst_tbl_off[r] + nblk[r]]
            for j in range(int(nblk[r])):
                if not sk[j]:
                    kept += int(min(Bd, lens[r] - j * Bd))
            if nblk[r] and not sk[nblk[r] - 1]:
                pad += int(nblk[r] * Bd - lens[r])
    P = kept * tok
    return {"pack": 2 * P, "unpack": 2 * P + pad * tok, "fused": 2 * P + pad * tok}


def step_bytes_of(w):
    """Algorithmic bytes of one step (pack + unpack + fused)."""
    return sum(op_bytes_of(w).values())


def cpu_baseline(w, src_t, reps=3):
    """Time the CPU checker, as it stands, on the first requests of the batch:
    pack, unpack and fused apart, on one thread and on all cores the sample can
    use (one thread per request), best of `reps`, wall clock."""
    import numpy as np
    import torch

    from oracle import pdkv_oracle as O
    from paper_2408_08147_b200 import workloads as W

    if w.src.elem_bytes != 2:
        return {"value": None, "unit": UNIT, "kind": "oracle", "skipped": "CPU leg is wired for 2-byte elements"}
    cores = os.cpu_count() or 1
    tok_bytes = w.src.token_bytes()

    def sample(n, rate_gbs, budget_s):
        # shrink the sample until 3 ops x reps passes fit the budget at the expected rate
        while n > 1 and 3 * reps * 2 * int(w.batch.seq_len[:n].sum()) * tok_bytes / (rate_gbs * 1e9) > budget_s:
            n -= 1
        sub, s_ids, _ = W.compact_subproblem(w, range(n))
        src_np = W.gather_blocks(src_t.view(torch.int16), w.src, s_ids).cpu().numpy().view(np.uint16)
        dst_np = W.sentinel_pool_numpy(sub.dst)
        buf_np = np.zeros(O.buffer_elems(sub.batch, sub.dst.block_tokens, sub.src), np.uint16)
        return n, sub, src_np, dst_np, buf_np

    def time_ops(sub, src_np, dst_np, buf_np, threads):
        G = sub.dst.block_tokens
        fns = {"pack": lambda: O.pack(sub.src, src_np, sub.batch, G, buf_np, threads=threads),
               "unpack": lambda: O.unpack(sub.dst, dst_np, sub.batch, buf_np, threads=threads),
               "fused": lambda: O.transfer(sub.src, src_np, sub.dst, dst_np, sub.batch, threads=threads)}
        nbytes = op_bytes_of(sub)
        rows = {}
        for name, fn in fns.items():
            best = None
            for _ in range(reps):
                t0 = time.perf_counter()
                fn()
                dt = time.perf_counter() - t0
                best = dt if best is None else min(best, dt)
            rows[name] = {"GBps": nbytes[name] / best / 1e9, "s_best": best}
        total = sum(nbytes.values()) / sum(r["s_best"] for r in rows.values()) / 1e9
        return rows, total

    t_all = time.perf_counter()
    n, sub, src_np, dst_np, buf_np = sample(min(w.batch.n_req, cores, 8), 6.0, 12.0)
    threads = min(cores, n)
    rows_all, total_all = time_ops(sub, src_np, dst_np, buf_np, threads)
    n1, one, one_src, one_dst, one_buf = sample(1, 0.9, 12.0)
    rows_one, total_one = time_ops(one, one_src, one_dst, one_buf, 1)
    return {"value": total_all, "unit": UNIT, "cores": threads, "kind": "oracle",
            "ops": {k: v["GBps"] for k, v in rows_all.items()},
            "single_thread_value": total_one, "single_thread_ops": {k: v["GBps"] for k, v in rows_one.items()},
            "sample": f"first {n} of {w.batch.n_req} requests ({int(sub.batch.seq_len.sum())} tokens, all layers) on "
                      f"{threads} threads, first {n1} request(s) on one thread; pack, unpack and fused timed apart, "
                      f"best of {reps}; {time.perf_counter() - t_all:.1f} s of wall clock in all",
            "host_cpus": cores}


def reference_arm(args):
    """The CPU checker timed as the reference implementation (rank 0 only)."""
    import numpy as np

    rank, _, world = dist_env()
    if rank != 0:
        return
    from oracle import pdkv_oracle as O
    from paper_2408_08147_b200 import workloads as W

    cores = os.cpu_count() or 1
    full = W.make_config(args.config)
    # bounded sample: whole run (warmup + steps) within ~2 minutes at ~0.4 GB/s per thread
    per_step_s = max(0.5, 110.0 / (args.steps + args.warmup))
    threads = min(cores, 8, full.batch.n_req)
    tok = full.src.token_bytes()
    tokens_budget = per_step_s * threads * 0.4e9 / (6 * tok)
    n_req = max(1, min(threads, full.batch.n_req))
    layers = full.src.num_layers
    while layers > 1 and float(full.batch.seq_len[:n_req].sum()) * layers / full.src.num_layers > tokens_budget:
        layers = max(1, layers // 2)
    w = W.make_config(args.config, n_req=n_req, num_layers=layers)
    chunk = W.normal_bf16_bits(1 << 22, w.seed)
    src_np = np.resize(chunk, w.src.num_elems())
    dst_np = W.sentinel_pool_numpy(w.dst)
    buf_np = np.zeros(O.buffer_elems(w.batch, w.dst.block_tokens, w.src), np.uint16)
    for _ in range(args.warmup):
        oracle_step(O, w, src_np, dst_np, buf_np, threads)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(O, w, src_np, dst_np, buf_np, threads)
    dt = time.perf_counter() - t0
    nbytes = step_bytes_of(w)
    value = nbytes * args.steps / dt / 1e9
    sample = (f"{n_req} of {full.batch.n_req} requests, {layers} of {full.src.num_layers} layers "
              f"per step ({nbytes / 1e9:.2f} GB algorithmic), {threads} threads")
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
           "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
           "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "u16", "data": "synthetic",
           "config": {"workload": workload_name(full), "sample": sample},
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                            "sample": sample},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


# ---------------------------------------------------------------------------
# main arm
# ---------------------------------------------------------------------------

def timed_ops(sess, buf_t, stream, steps, warmup, torch, B, device_index=None, sync_ranks=False):
    """Warm up, then time `steps` steps (pack, unpack, fused back to back) with CUDA events on
    the launching stream.  Returns per-operation times, the step time and the clock samples."""
    ops = [("pack", B.PDKV_OP_PACK, lambda: sess.pack(buf_t)),
           ("unpack", B.PDKV_OP_UNPACK, lambda: sess.unpack(buf_t)),
           ("fused", B.PDKV_OP_TRANSFER, lambda: sess.transfer())]

    def run_step(evs=None):
        for i, (_, _, fn) in enumerate(ops):
            if evs is not None:
                evs[i].record(stream)
            fn()
        if evs is not None:
            evs[3].record(stream)

    with torch.cuda.stream(stream):
        for _ in range(warmup):
            run_step()
    torch.cuda.synchronize()
    sess.status()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps)]
    if sync_ranks:
        barrier()
    torch.cuda.synchronize()
    with ClockSampler(device_index) as clk:
        with torch.cuda.stream(stream):
            for k in range(steps):
                run_step(evs[k])
        torch.cuda.synchronize()
    if sync_ranks:
        barrier()
    times = {name: [evs[k][i].elapsed_time(evs[k][i + 1]) for k in range(steps)] for i, (name, _, _) in enumerate(ops)}
    traffic = {name: sum(sess.traffic(op)) for name, op, _ in ops}
    return {"ms_per_step": evs[0][0].elapsed_time(evs[-1][3]) / steps, "times": times, "traffic": traffic,
            "launches_per_step": sum(sess.launches(op) for _, op, _ in ops), "clocks": clk.summary()}


def op_rows(t, peak, peak_kind, plan_ms=None):
    rows = {}
    for name, ms in t["times"].items():
        mean = statistics.fmean(ms)
        ach = t["traffic"][name] / (mean * 1e-3) / 1e9
        rows[name] = {"ms": mean, "ms_median": statistics.median(ms), "ms_best": min(ms), "GBps": ach,
                      "frac_of_" + peak_kind: ach / peak, "frac_of_nominal_8000": ach / 8000.0,
                      "bytes": t["traffic"][name]}
        if plan_ms is not None:
            rows[name]["ms_incl_plan"] = mean + plan_ms
    return rows


def blockwise_leg(sess, stream, reps, fused_ms, fused_bytes, torch, B):
    """Block-by-block baseline (Sec. 2.3, one copy or launch per prefill block from a host loop)."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        sess.transfer_blockwise()
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(reps):
            sess.transfer_blockwise()
        e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    return {"ms": ms, "GBps": fused_bytes / (ms * 1e-3) / 1e9, "gpu_ops_per_call": sess.launches(B.PDKV_OP_BLOCKWISE),
            "fused_speedup": ms / fused_ms}


def side_config(spec, steps, warmup, peak, peak_kind, torch, B, W, TransferSession, local):
    """One of the other benchmark workloads, timed like the headline one (same step, same
    events), with its block-by-block baseline.  `spec` is "4" or "5:256" (config:prefill block)."""
    idx, _, blk = spec.partition(":")
    kw = {"src_block": int(blk)} if blk else {}
    w = W.make_config(int(idx), **kw)
    src_t, dst_t = alloc_pools(w, torch)
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    with TransferSession(w.src, src_t, w.dst, dst_t, w.batch, stream.cuda_stream) as sess:
        buf_t = torch.empty(max(sess.buffer_bytes, 16), dtype=torch.uint8, device=src_t.device)
        t = timed_ops(sess, buf_t, stream, steps, warmup, torch, B, local)
        rows = op_rows(t, peak, peak_kind)
        ok = sanity_check(w, src_t, dst_t, torch)
        bw = blockwise_leg(sess, stream, max(1, min(3, steps)), rows["fused"]["ms"], t["traffic"]["fused"], torch, B)
        out = {"workload": workload_name(w), "steps": steps, "ms_per_step": t["ms_per_step"],
               "GBps": sum(t["traffic"].values()) / (t["ms_per_step"] * 1e-3) / 1e9,
               "payload_bytes": sess.buffer_bytes, "ops": rows, "blockwise_baseline": bw,
               "gpu_launches": t["launches_per_step"] * steps, "sanity_check": "ok" if ok else "MISMATCH",
               "clocks": t["clocks"]}
    del src_t, dst_t, buf_t
    torch.cuda.empty_cache()
    return out


def main_arm(args):
    import numpy as np  # noqa: F401
    import torch

    from paper_2408_08147_b200 import binding as B
    from paper_2408_08147_b200 import workloads as W
    from paper_2408_08147_b200.session import TransferSession

    B.lib()  # fail loudly if the CUDA library is missing
    rank, local, world = dist_env()
    assert torch.cuda.is_available(), "bench.py needs a CUDA device"
    torch.cuda.set_device(local)
    rank, world = dist_init("nccl")
    dev = torch.device("cuda", local)

    for k, v in (args.tune or []):
        B.pdkv_tune(k, int(v))

    kw = {}
    if args.src_block:
        kw["src_block"] = args.src_block
    if args.n_req:
        kw["n_req"] = args.n_req
    if args.elem_bytes:
        kw["elem_bytes"] = args.elem_bytes
    if args.kv_heads:
        kw["num_kv_heads"] = args.kv_heads
    if args.num_layers:
        kw["num_layers"] = args.num_layers
    if args.head_dim:
        kw["head_dim"] = args.head_dim
    if args.layouts:
        kw["src_layout"], kw["dst_layout"] = ("AB".index(args.layouts[0]), "AB".index(args.layouts[1]))
    # the plain command (no workload flags) also times the other benchmark workloads after the headline one
    plain = args.config == 2 and not kw and not args.tune and not args.autotune
    w = W.make_config(args.config, **kw)
    src_t, dst_t = alloc_pools(w, torch, seed_offset=rank)
    torch.cuda.synchronize()          # the fills ran on torch's stream, the library gets its own
    stream = torch.cuda.Stream()
    sess = TransferSession(w.src, src_t, w.dst, dst_t, w.batch, stream.cuda_stream)
    # plan creation (table validation, tile lists, one upload) is outside the timed step: time it apart
    plan_ms = []
    for _ in range(5):
        t0 = time.perf_counter()
        TransferSession(w.src, src_t, w.dst, dst_t, w.batch, stream.cuda_stream).close()
        plan_ms.append((time.perf_counter() - t0) * 1e3)
    buf_t = torch.empty(max(sess.buffer_bytes, 16), dtype=torch.uint8, device=dev)
    tuned = None
    if args.autotune:
        tuned = {str(k): v for k, v in sess.autotune(buf_t).items()}
        torch.cuda.synchronize()

    t = timed_ops(sess, buf_t, stream, args.steps, args.warmup, torch, B, local, sync_ranks=True)
    ok = sanity_check(w, src_t, dst_t, torch)
    step_bytes = sum(t["traffic"].values())
    ms_step, units = reduce_step_time(t["ms_per_step"], float(step_bytes), dev)
    value = units / (ms_step * 1e-3) / 1e9

    peak, peak_kind = measured_peak()
    per_op = op_rows(t, peak, peak_kind, statistics.median(plan_ms))

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": f"u{8 * w.src.elem_bytes}", "data": "synthetic",
           "config": {"workload": workload_name(w), "config_index": args.config,
                      "step": "pdkv_pack + pdkv_unpack + pdkv_transfer, all layers",
                      "payload_bytes": sess.buffer_bytes, "step_bytes": step_bytes,
                      "plan_create_destroy_ms": statistics.median(plan_ms),
                      "autotuned_shapes": tuned,   # (threads, unroll, CTAs/SM, strip skew) per op; zeros = built-in, skew -1 = stride rule
                      "l2": "inputs exceed L2 (pools and buffer are GiB-sized; no flush needed)"
                      if sess.buffer_bytes > (1 << 29) else "L2-resident workload: not an HBM number",
                      "tunables": {k: B.pdkv_tune_get(k) for k in
                                   ("tile_bytes", "ctas_per_sm", "threads", "unroll", "group_threads", "vec32", "lc_fastest", "lc_skew",
                                    "variant")}},
           "ops": per_op, "gpu_launches": t["launches_per_step"] * args.steps,
           "sanity_check": "ok" if ok else "MISMATCH", "clocks": t["clocks"]}

    if rank == 0 and not args.no_extras and not args.no_blockwise:
        out["blockwise_baseline"] = blockwise_leg(sess, stream, max(1, min(5, args.steps)), per_op["fused"]["ms"],
                                                  t["traffic"]["fused"], torch, B)

    # end to end: pinned host pools, H2D of the prefill pool, plan, the three calls, D2H of the decode pool
    if not args.no_extras and not args.no_e2e:
        try:
            out["e2e"] = e2e_leg(args, w, src_t, dst_t, buf_t, stream, step_bytes, torch, B, TransferSession, dev)
        except Exception as e:  # pragma: no cover
            out["e2e"] = {"error": repr(e)}
    sess.close()

    if rank == 0 and world == 1 and not args.no_extras and not args.no_cpu:
        try:
            out["cpu_baseline"] = cpu_baseline(w, src_t)
        except Exception as e:  # pragma: no cover
            out["cpu_baseline"] = {"error": repr(e)}

    # The other workloads (one GPU only: with several ranks every GPU would be held meanwhile).
    # Config 4 is the second workload the 75%-of-HBM target names; 3 and 5 re-create the
    # small-block argument of Sec. 2.3 against the block-by-block baseline.
    rows_by_config = {str(args.config): {"ops": per_op}}
    if rank == 0 and world == 1 and plain and not args.no_extras and args.also:
        del src_t, dst_t, buf_t
        torch.cuda.empty_cache()
        out["configs"] = {}
        for spec in args.also.split(","):
            try:
                res = side_config(spec, max(1, min(args.steps, args.also_steps)), args.warmup, peak, peak_kind,
                                  torch, B, W, TransferSession, local)
            except Exception as e:  # pragma: no cover
                res = {"error": repr(e)}
            out["configs"][spec] = res
            if "ops" in res:
                rows_by_config[spec] = res
                out["gpu_launches"] += res["gpu_launches"]

    # roofline: the launch furthest below the HBM peak among the workloads the target names (2 and 4)
    named = {k: v for k, v in rows_by_config.items() if k in (str(args.config), "4")}
    dom_cfg, dom = min(((c, n) for c, v in named.items() for n in v["ops"]),
                       key=lambda cn: named[cn[0]]["ops"][cn[1]]["GBps"])
    row = named[dom_cfg]["ops"][dom]
    sha = kernel_sha()
    as_specified = not kw and not args.tune and not args.autotune     # the counters were taken on the workload as specified
    traffic_ncu = NCU_TRAFFIC.get((int(dom_cfg), dom)) if sha == NCU_KERNEL_SHA and as_specified else None
    out["roofline"] = {"bound": "hbm", "achieved": row["GBps"], "peak": peak, "unit": "GB/s",
                       "frac": row["GBps"] / peak, "frac_of_nominal_8000": row["GBps"] / 8000.0,
                       "traffic": traffic_ncu, "op": dom, "config": dom_cfg,
                       "kernel": "pdkv::copy_tiles_kernel",
                       "peak_source": f"{peak_kind} (MEASURED_PEAKS.json hbm_gbs)"
                       if peak_kind == "measured" else "fallback 6650 GB/s",
                       "algorithmic_bytes_per_launch": row["bytes"], "ms_per_launch": row["ms"]}
    if rank == 0:
        print(json.dumps(out), flush=True)
    if world > 1:
        import torch.distributed as dist

        dist.destroy_process_group()


def e2e_leg(args, w, src_t, dst_t, buf_t, stream, step_bytes, torch, B, TransferSession, dev):
    """Same step, but the prefill pool starts in pinned host memory and the
    decode pool is read back to pinned host memory, every step, inside the timed
    region; the plan (tables) is also rebuilt from host arrays each step."""
    free_host = None
    try:
        import psutil

        free_host = psutil.virtual_memory().available
    except Exception:
        pass
    _, _, world = dist_env()
    need = (src_t.numel() + dst_t.numel()) * world      # every rank on this node pins its own images
    fits = not (free_host is not None and need > 0.5 * free_host)
    fits = all_ranks_agree(fits, dev)     # one rank skipping alone would leave the others in a barrier
    if not fits:
        return {"value": None, "unit": UNIT,
                "skipped": f"needs {need >> 30} GiB of pinned host memory across {world} ranks, "
                           f"{(free_host or 0) >> 30} GiB available"}
    try:
        h_src = torch.empty(src_t.numel(), dtype=torch.uint8, pin_memory=True)
        h_dst = torch.empty(dst_t.numel(), dtype=torch.uint8, pin_memory=True)
        pinned = True
    except RuntimeError:
        h_src = h_dst = None
        pinned = False
    if not all_ranks_agree(pinned, dev):
        return {"value": None, "unit": UNIT, "skipped": "pinned host allocation failed on a rank"}
    h_src.copy_(src_t)
    steps = max(1, min(args.e2e_steps, args.steps))
    up_down = [0, 0]

    # The batch is cut into request groups that go round three streams, so that one
    # group's download overlaps the next group's upload (PCIe is full duplex) and
    # the kernels in between.  Every group runs the whole step for its requests.
    from paper_2408_08147_b200 import workloads as W

    n_groups = max(1, min(args.e2e_groups, w.batch.n_req))
    cuts = [round(i * w.batch.n_req / n_groups) for i in range(n_groups + 1)]
    groups = [W.slice_batch(w.batch, cuts[i], cuts[i + 1]) for i in range(n_groups)]
    streams = [torch.cuda.Stream() for _ in range(min(3, n_groups))]
    setup = torch.cuda.Stream()
    # one preallocated workspace per group for its plan: no cudaMalloc / cudaFree inside a step
    spaces = [torch.empty(4 << 20, dtype=torch.uint8, device=dev) for _ in range(n_groups)]

    def one():
        sessions, at, up, down = [], 0, 0, 0
        for g, part in enumerate(groups):
            st = streams[g % len(streams)].cuda_stream
            s = TransferSession(w.src, src_t, w.dst, dst_t, part, setup.cuda_stream,   # plan: tables from host
                                workspace_t=spaces[g])
            piece = buf_t[at:at + s.buffer_bytes] if s.buffer_bytes else buf_t[:16]
            at += s.buffer_bytes
            s.upload_blocks(h_src, st)      # pdkv_upload_blocks: H2D of the group's prefill blocks
            s.pack(piece, stream=st)
            s.unpack(piece, stream=st)
            s.transfer(stream=st)
            s.download_blocks(h_dst, st)    # pdkv_download_blocks: D2H of the group's decode blocks
            a, b = s.block_bytes()
            up, down = up + a, down + b
            sessions.append(s)
        for st in streams:
            st.synchronize()
        up_down[:] = [up, down]
        for s in sessions:
            s.close()

    one()
    barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        one()
    torch.cuda.synchronize()
    barrier()
    ms = (time.perf_counter() - t0) * 1e3 / steps
    ms, units = reduce_step_time(ms, float(step_bytes), dev)
    del h_src, h_dst
    return {"value": units / (ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": ms, "steps": steps,
            "h2d_bytes_per_step": int(up_down[0]), "d2h_bytes_per_step": int(up_down[1]),
            "includes": "pdkv_plan_create_in (tables from host arrays, preallocated workspaces), pdkv_upload_blocks from a pinned host image of "
                        "the prefill pool, pack, unpack, fused, pdkv_download_blocks into a pinned host image of "
                        "the decode pool; wall clock",
            "pipeline": f"{n_groups} request groups over {len(streams)} streams"}


def _replay_on(graph, stream, torch):
    with torch.cuda.stream(stream):
        graph.replay()


def overlap_arm(args):
    """Per-layer trigger (Sec. 3.5): layer l is transferred on a side stream as soon
    as a stand-in for layer l's compute (one bf16 GEMM on the main stream) has
    finished, while layer l+1 computes.  Reports compute alone, transfer alone and
    both overlapped -- how much of the transfer is hidden and by how much the compute
    sequence itself is held up -- for the kernels sharing all SMs with the GEMM, for
    plain device copies (no kernel), and for the transfer kernel on an SM partition
    of its own (green contexts) with the GEMM on the remaining SMs."""
    import torch

    from paper_2408_08147_b200 import binding as B
    from paper_2408_08147_b200 import workloads as W
    from paper_2408_08147_b200.session import TransferSession

    B.lib()
    torch.cuda.set_device(0)
    kw = {"n_req": args.n_req} if args.n_req else {}
    if args.layouts:
        kw["src_layout"], kw["dst_layout"] = ("AB".index(args.layouts[0]), "AB".index(args.layouts[1]))
    w = W.make_config(args.config, **kw)
    src_t, dst_t = alloc_pools(w, torch)
    L = w.src.num_layers
    n = args.gemm_n
    a = torch.randn(n, n, device="cuda", dtype=torch.bfloat16)
    b = torch.randn(n, n, device="cuda", dtype=torch.bfloat16)
    c = torch.empty(n, n, device="cuda", dtype=torch.bfloat16)
    # the transfer stream gets the higher priority: its CTAs are placed as soon as
    # a compute CTA retires instead of after the whole compute grid
    plain_main, plain_side = torch.cuda.Stream(), torch.cuda.Stream(priority=-1 if args.side_priority else 0)
    torch.cuda.synchronize()

    def timed(fn, reps, main, side):
        """(whole sequence, main stream alone) in ms per repetition; the second is when the
        compute sequence itself finished, whatever the side stream still had to do."""
        e0, e_main, e1 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        fn()
        torch.cuda.synchronize()
        e0.record(main)
        side.wait_event(e0)
        for _ in range(reps):
            fn()
        e_main.record(main)
        side_done = torch.cuda.Event()
        side_done.record(side)
        main.wait_event(side_done)
        e1.record(main)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps, e0.elapsed_time(e_main) / reps

    def compute_on(main):
        def fn():
            with torch.cuda.stream(main):
                for _ in range(L):
                    torch.matmul(a, b, out=c)
        return fn

    same_blocks = w.src.layout == 0 and w.dst.layout == 0 and w.src.block_tokens == w.dst.block_tokens
    modes = [("register copy, defaults", {"variant": 0}, None),
             ("register copy on at most 32 SMs (grid cap only, SMs shared with the GEMM)",
              {"variant": 0, "ctas_per_sm": 1, "threads": 1024, "unroll": 1, "max_ctas": 32}, None),
             ("register copy, two warps per CTA (64 threads x 4 accesses), 8 CTAs/SM",
              {"variant": 0, "ctas_per_sm": 8, "threads": 64, "unroll": 4, "group_threads": 64}, None),
             ("bulk copy (TMA), 8 KiB tiles x 2 stages x 8 CTAs/SM",
              {"variant": 1, "tile_bytes": 8192, "stages": 2, "ctas_per_sm": 8}, None),
             ("bulk copy with tiled TMA loads, 16 KiB tiles x 4 stages x 3 CTAs/SM",
              {"variant": 2, "tile_bytes": 16384, "stages": 4, "ctas_per_sm": 3}, None)]
    if same_blocks:
        modes.append(("plain device copies, one per block and layer (no kernel)", {"variant": 0}, "copies"))
    for sms in (args.partition_sms or []):
        modes.append((f"register copy on an SM partition of its own ({sms} SMs asked for)",
                      {"variant": 0, "ctas_per_sm": 2}, sms))
    defaults = {k: B.pdkv_tune_get(k) for k in ("variant", "ctas_per_sm", "threads", "unroll", "tile_bytes", "stages",
                                                "max_ctas", "group_threads")}
    with ClockSampler(0) as clk0:
        t_compute, _ = timed(compute_on(plain_main), args.steps, plain_main, plain_side)
    results = {}
    for name, tune, special in modes:
        main, side, part = plain_main, plain_side, None
        tune = dict(tune)
        rec = {}
        try:
            if isinstance(special, int):
                part = B.pdkv_sm_partition_create(0, special)
                got_t, got_c = B.pdkv_sm_partition_info(part)
                side = torch.cuda.ExternalStream(B.pdkv_sm_partition_stream(part, 0))
                main = torch.cuda.ExternalStream(B.pdkv_sm_partition_stream(part, 1))
                rec["sm_partition"] = {"transfer_sms": got_t, "compute_sms": got_c}
        except B.PdkvError as e:
            results[name] = {"unavailable": str(e)}
            continue
        for k, v in {**defaults, **tune}.items():
            B.pdkv_tune(k, v)
        sess = TransferSession(w.src, src_t, w.dst, dst_t, w.batch, side.cuda_stream)
        move = (lambda l: B.pdkv_transfer_copies(sess.plan, l, l + 1, side.cuda_stream)) if special == "copies" else \
            (lambda l: sess.transfer((l, l + 1), side.cuda_stream))

        def transfer_only():
            for l in range(L):
                move(l)

        def overlapped():
            for l in range(L):
                with torch.cuda.stream(main):
                    torch.matmul(a, b, out=c)
                    ev = torch.cuda.Event()
                    ev.record(main)
                side.wait_event(ev)
                move(l)

        t_c, _ = timed(compute_on(main), args.steps, main, side) if part else (t_compute, None)
        t_x, _ = timed(transfer_only, args.steps, main, side)
        with ClockSampler(0) as clk:
            t_o, t_o_main = timed(overlapped, args.steps, main, side)
        rec["clocks_while_overlapped"] = clk.summary()
        rec.update({"compute_alone_ms": t_c, "transfer_alone_ms": t_x, "overlapped_ms": t_o,
                    "compute_sequence_while_overlapped_ms": t_o_main,
                    "serial_ms": t_c + t_x,
                    "hidden_fraction_of_transfer": max(0.0, min(1.0, (t_c + t_x - t_o) / t_x)),
                    # how much longer the whole job takes than the GEMM sequence alone on the full GPU
                    "job_slowdown_vs_compute_on_all_sms": t_o / t_compute - 1.0,
                    "compute_slowdown_vs_all_sms": t_o_main / t_compute - 1.0})
        if special is None:
            # the same per-layer sequence recorded once into a CUDA graph and replayed
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                cur = torch.cuda.current_stream().cuda_stream
                for l in range(L):
                    sess.transfer((l, l + 1), cur)
            rec["transfer_alone_graph_ms"], _ = timed(lambda: _replay_on(graph, side, torch), args.steps, main, side)
        results[name] = rec
        sess.close()
        if part:
            torch.cuda.synchronize()
            del main, side
            B.pdkv_sm_partition_destroy(part)
    for k, v in defaults.items():
        B.pdkv_tune(k, v)
    out = {"mode": "overlap", "config": {"workload": workload_name(w), "layers": L,
                                         "compute_stand_in": f"{L} x torch.matmul bf16 {n}^3 on the main stream",
                                         "transfer_stream_priority": "high" if args.side_priority else "default"},
           "compute_alone_ms": t_compute, "clocks_compute_alone": clk0.summary(), "variants": results}
    print(json.dumps(out), flush=True)


def retrieval_arm(args):
    """Asynchronous retrieval (Sec. 3.5): the batch arrives as request groups that
    are retrieved through a queue of `capacity` receive slots.  Reports makespan
    and mean completion time for capacities 1 (one after another) to 4
    (several transmissions sharing the bandwidth)."""
    import torch

    from paper_2408_08147_b200 import binding as B
    from paper_2408_08147_b200 import workloads as W

    B.lib()
    torch.cuda.set_device(0)
    w = W.make_config(args.config)
    src_t, dst_t = alloc_pools(w, torch)
    torch.cuda.synchronize()
    ps = B.pdkv_pool_create(B.desc_of(w.src), src_t.data_ptr(), src_t.numel(), 0)
    pd = B.pdkv_pool_create(B.desc_of(w.dst), dst_t.data_ptr(), dst_t.numel(), 0)
    n_groups = max(1, min(args.retrieval_groups, w.batch.n_req))
    cuts = [round(i * w.batch.n_req / n_groups) for i in range(n_groups + 1)]
    groups = [W.slice_batch(w.batch, cuts[i], cuts[i + 1]) for i in range(n_groups)]
    out = {"mode": "retrieval", "config": {"workload": workload_name(w), "groups": n_groups}, "capacities": {}}
    for cap in (1, 2, 4):
        q = B.pdkv_queue_create(ps, pd, 0, cap)
        best = None
        for _ in range(max(3, args.steps // 10)):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            pending, done_at = [], []
            for part in groups:
                while True:
                    t = B.pdkv_queue_submit(q, part.seq_len, part.src_tbl_off, part.src_tbl, part.dst_tbl_off,
                                            part.dst_tbl, part.dst_skip)
                    if t is not None:
                        pending.append(t)
                        break
                    B.pdkv_queue_wait(q, pending[0])
                    done_at.append(time.perf_counter() - t0)
                    B.pdkv_queue_release(q, pending.pop(0))
            for t in pending:
                B.pdkv_queue_wait(q, t)
                done_at.append(time.perf_counter() - t0)
                B.pdkv_queue_release(q, t)
            rec = {"makespan_ms": done_at[-1] * 1e3, "mean_completion_ms": statistics.fmean(done_at) * 1e3}
            if best is None or rec["makespan_ms"] < best["makespan_ms"]:
                best = rec
        best["rejected_submits"] = B.pdkv_queue_stats(q)[3]
        out["capacities"][str(cap)] = best
        B.pdkv_queue_destroy(q)
    B.pdkv_pool_destroy(ps)
    B.pdkv_pool_destroy(pd)
    print(json.dumps(out), flush=True)


def p2d_arm(args):
    """Prefill-to-decode transfer between two ranks on two GPUs (Sec. 3.5; launch with
    torchrun --nproc-per-node 2): rank 0 holds the prefill pool and packs, the buffer
    crosses NVLink in one NCCL send / recv, rank 1 unpacks.  Times the block-free
    transfer against the same bytes sent one prefill block's worth at a time."""
    import torch

    from paper_2408_08147_b200 import binding as B
    from paper_2408_08147_b200 import p2d
    from paper_2408_08147_b200 import workloads as W

    rank, local, world = dist_env()
    if world != 2:
        if rank == 0:
            print(json.dumps({"mode": "p2d", "unavailable": "needs exactly two ranks, one GPU each"}), flush=True)
        return
    B.lib()
    host = args.p2d_host_buffers      # buffer in pinned host memory, gloo carries it; the ranks may share a GPU
    local = local % torch.cuda.device_count() if host else local
    torch.cuda.set_device(local)
    dist_init("gloo" if host else "nccl")
    dev = torch.device("cuda", local)
    meta_dev = "cpu" if host else dev
    kw = {"n_req": args.n_req} if args.n_req else {}
    if args.num_layers:
        kw["num_layers"] = args.num_layers
    w = W.make_config(args.config, **kw)
    b = w.batch
    if rank == 0:
        pool_t = torch.empty(w.src.num_bytes(), dtype=torch.uint8, device=dev)
        W.fill_pool_torch(pool_t, w.seed)
    else:
        pool_t = torch.zeros(w.dst.num_bytes(), dtype=torch.uint8, device=dev)
    torch.cuda.synchronize()
    cache = {}

    def buffer(n):                      # one buffer per rank, reused across repetitions
        if cache.get("n", 0) < n:
            cache["t"] = torch.empty(n, dtype=torch.uint8, pin_memory=True) if host else \
                torch.empty(n, dtype=torch.uint8, device=dev)
            cache["n"] = n
        return cache["t"][:n]

    block_bytes = w.src.num_bytes() // w.src.num_blocks
    results = {}
    stage = max(1, args.p2d_layers_per_stage)
    for name, chunk, lps in (("whole buffer", 0, 0), ("one prefill block per message", block_bytes, 0),
                             (f"layer pipeline, {stage} layers per stage (pack | send | unpack overlap)", 0, stage)):
        times, nbytes = [], 0
        for it in range(args.warmup + args.steps):
            barrier()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            if rank == 0:
                nbytes, sess, _ = p2d.send_kv(b.seq_len, p2d.gpu_sender(w.src, pool_t, b.src_tbl_off, b.src_tbl, b.seq_len),
                                              buffer, peer=1, device=meta_dev, chunk_bytes=chunk, layers_per_stage=lps)
            else:
                nbytes, sess, _ = p2d.recv_kv(b.dst_tbl_off, b.dst_skip, w.dst.block_tokens,
                                              p2d.gpu_receiver(w.dst, pool_t, b.dst_tbl_off, b.dst_tbl, b.dst_skip),
                                              buffer, peer=0, device=meta_dev, chunk_bytes=chunk, layers_per_stage=lps)
            torch.cuda.synchronize()
            dt = (time.perf_counter() - t0) * 1e3
            sess.close()
            ms, _ = reduce_step_time(dt, 0.0, meta_dev)
            if it >= args.warmup:
                times.append(ms)
        results[name] = {"ms": statistics.fmean(times), "ms_best": min(times), "buffer_bytes": nbytes,
                         "link_GBps": nbytes / (statistics.fmean(times) * 1e-3) / 1e9,
                         "messages": max(1, -(-nbytes // chunk)) if chunk else
                         (len(p2d.layer_stages(w.src.num_layers, lps)) * b.n_req if lps else 1)}
    if rank == 0:
        a, c = results["whole buffer"]["ms"], results["one prefill block per message"]["ms"]
        pipe = [v["ms"] for k, v in results.items() if k.startswith("layer pipeline")][0]
        print(json.dumps({"mode": "p2d", "config": {"workload": workload_name(w)}, "variants": results,
                          "time_saved_by_block_free": 1.0 - a / c, "time_saved_by_layer_pipeline_vs_whole_buffer": 1.0 - pipe / a,
                          "transport": "gloo, pinned host buffers" if host else "NCCL send/recv between two GPUs",
                          "includes": "meta exchange, plan, pack, send/recv, unpack; wall clock, max over ranks"}),
              flush=True)
    import torch.distributed as dist

    dist.destroy_process_group()


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="pdkv", choices=["pdkv", "reference"])
    ap.add_argument("--config", type=int, default=2, help="workload 1..5 (2 = the headline config)")
    ap.add_argument("--src-block", type=int, default=0)
    ap.add_argument("--elem-bytes", type=int, default=0, help="KV element size override (1 = fp8/int8 KV)")
    ap.add_argument("--kv-heads", type=int, default=0, help="KV head count override (1 = MQA)")
    ap.add_argument("--head-dim", type=int, default=0, help="head dimension override (e.g. 96)")
    ap.add_argument("--n-req", type=int, default=0, help="shrink the batch (profiling captures)")
    ap.add_argument("--num-layers", type=int, default=0, help="shrink the model (profiling captures)")
    ap.add_argument("--layouts", default="", help="two letters, e.g. AB: prefill block-major, decode layer-major")
    ap.add_argument("--tune", nargs=2, action="append", metavar=("KEY", "VALUE"))
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--e2e-groups", type=int, default=16, help="request groups pipelined over three streams in the e2e leg")
    ap.add_argument("--no-extras", action="store_true", help="skip baseline, e2e and CPU legs")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--overlap", action="store_true", help="per-layer transfer overlapped with a compute stand-in")
    ap.add_argument("--retrieval", action="store_true", help="request groups through the asynchronous retrieval queue")
    ap.add_argument("--retrieval-groups", type=int, default=8)
    ap.add_argument("--p2d", action="store_true", help="two ranks, two GPUs: pack -> one NCCL send/recv -> unpack")
    ap.add_argument("--p2d-host-buffers", action="store_true",
                    help="with --p2d: contiguous buffer in pinned host memory, gloo transport; the two ranks may share one GPU")
    ap.add_argument("--p2d-layers-per-stage", type=int, default=4, help="with --p2d: layers per stage of the pipelined variant")
    ap.add_argument("--gemm-n", type=int, default=4096)
    ap.add_argument("--partition-sms", type=int, action="append",
                    help="with --overlap: also run the transfer on an SM partition of this many SMs (repeatable)")
    ap.add_argument("--side-priority", type=int, default=1, help="1: transfer stream has high priority")
    ap.add_argument("--no-blockwise", action="store_true")
    ap.add_argument("--autotune", action="store_true", help="pdkv_plan_autotune before the timed steps (not the default run)")
    ap.add_argument("--also", default="4,3,5:16,5:256",
                    help="workloads timed after the headline one by the plain command (config or config:prefill block)")
    ap.add_argument("--also-steps", type=int, default=10, help="timed steps per workload of --also")
    return ap.parse_args()


if __name__ == "__main__":
    a = parse()
    a.warmup = max(a.warmup, 3) if a.impl == "pdkv" else a.warmup
    if a.overlap:
        overlap_arm(a)
    elif a.retrieval:
        retrieval_arm(a)
    elif a.p2d:
        p2d_arm(a)
    elif a.impl == "reference":
        reference_arm(a)
    else:
        main_arm(a)
