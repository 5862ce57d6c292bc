#!/usr/bin/env python
"""Benchmark of the PatchKV suffix-restore hot path on B200.

One step = one pass of the whole hot path over one batch of synthetic input: patchkv_select_repair (dirty
window, top-k of stored block masses, union, lists) followed by patchkv_restore (dequantise by tag, RoPE
phase correction of K, page placement) of every reused block, on the Llama-3-8B-shaped workload (32 layers,
8 KV heads, head_dim 128, 16384-token suffix, 16-token blocks, tags 30/50/20 bf16/int8/int4, repair set
15 %, device-resident payload, 1280-page pool).  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--sweep]

value      restored KV GB/s (bf16-equivalent: bytes of bf16 K+V written to the pool / time), inputs in HBM.  The
           block of K steps is repeated until at least one second of GPU time has been timed; value and ms_per_step
           are those of the median block, min / max and the SM clocks seen alongside are reported too.
e2e        the same metric through the host-resident entry point: block masses copied from pinned host
           memory, selection lists read back, patchkv_restore_from_host streaming the pinned payload.
roofline   the restore kernel against the measured HBM copy bandwidth.
cpu_baseline / --impl reference   the CPU checker in oracle/ timed on the machine's host cores (a reported
           baseline only; it is a deliberately plain program).
configs    (last key) one compact row per BASELINE configuration: ms, bf16-equivalent GB/s, fraction of the roofline
           that bounds it (HBM or the host link), selection time.
--sweep    instead of the benchmark line: restore / writer fractions by tag and by geometry, restore time by suffix
           length, and the host path's merge-gap sweep, on half-size (16-layer) workloads; one JSON line.
With N > 1 (torchrun) every rank restores its own copy of the workload on its own GPU: the path has no
exchange step, so this is weak scaling without any data-path collective.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import re
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

import patchkv_inputs as pin

METRIC = "restored_kv_gbps_bf16_equiv"
UNIT = "GB/s"
WORKLOAD = "llama3-8b-shaped: L=32 H=8 D=128 base=5e5 n=16384 B=P=16 G=32 tags 30/50/20 repair 15% device-resident"
FALLBACK_HBM_GBS = 6650.0
MIN_TIMED_GPU_SECONDS = 1.0
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "restore_pipe_kernel_llama8b_slice.traffic.txt")


# ------------------------------------------------------------------------------------------ helpers
def workload_config(delta: int, world: int, layers: int = 32, tags: str = "") -> dict:
    """The `config` object of the JSON line, the same for both arms."""
    note = (f" [PROFILING SLICE: {layers} layers]" if layers != 32 else "") + (f" [PROFILING: tag shares {tags}]" if tags else "")
    return {"workload": WORKLOAD + note,
            "delta": delta, "l2": "working set 3.0 GB per step >> 126 MB L2, no flush",
            "parallelism": f"independent replicas x{world}" if world > 1 else "1 gpu"}


def algorithmic_bytes(ck: pin.SuffixCheckpoint, reuse_idx: np.ndarray, reuse_cnt: np.ndarray):
    """(payload bytes read, bf16 bytes written, reused block-layers) of one restore of `ck`."""
    g = ck.geom
    tags = ck.tags.cpu().numpy()
    rec = np.array([pin.record_bytes(t, g) for t in range(4)], dtype=np.int64)
    read = 0
    items = 0
    for l in range(g.n_layers):
        F = reuse_idx[l, :reuse_cnt[l]]
        read += int(rec[tags[l, F]].sum())
        items += len(F)
    # every reused block writes B tokens of K and V in bf16 (the suffix here is a whole number of blocks)
    written = items * 2 * g.block_tokens * g.n_kv_heads * g.head_dim * 2
    return read, written, items


def captured_traffic(block_layers: int, written_bytes: int):
    """DRAM traffic of one restore launch from the committed ncu capture of a slice of the same workload
    (profiles/restore_pipe_kernel_llama8b_slice.traffic.txt).  Reads are proportional to the reused block-layers;
    writes are the launch's bf16 bytes less what the capture shows still dirty in L2 at kernel end.
    Returns (bytes, where it comes from); (None, reason) when the file is absent."""
    try:
        kv = dict(re.findall(r"^(\w+)\s*=\s*(\S+)\s*$", open(TRAFFIC_FILE).read(), flags=re.M))
        reads = float(kv["dram_bytes_read_per_launch"]) / float(kv["block_layers"]) * block_layers
        l2_dirty = float(kv["algorithmic_bytes_written"]) - float(kv["dram_bytes_write_per_launch"])
        return int(reads + written_bytes - l2_dirty), (f"ncu capture {kv['capture']} of a {kv['block_layers']}-block-layer slice, "
                                                       f"scaled (profiles/{os.path.basename(TRAFFIC_FILE)})")
    except Exception as exc:
        return None, f"no capture on file: {exc!r}"[:120]


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.gpu_index), "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def rows(self, t0: float, t1: float):
        """(time, sm MHz, max MHz, active reasons) of the samples taken in [t0, t1] (all samples if none fall inside)."""
        out = []
        for t, line in list(self.lines):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                out.append((t, float(f[1]), float(f[2]),
                            [n for n, val in zip(self.NAMES, f[5:9]) if val.lower().startswith("active")]))
            except ValueError:
                continue
        inside = [r for r in out if t0 - 0.05 <= r[0] <= t1 + 0.25]
        return inside or out

    def stop(self, t0: float, t1: float, blocks=None):
        """Summary of the samples in [t0, t1].  `blocks`: [(host time at the block's end, ms per step)] - each block is
        booked under the SM clock of the sample nearest to it in time."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        rows = self.rows(t0, t1)
        sm = [r[1] for r in rows]
        out = {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max((r[2] for r in rows), default=None),
               "sm_mhz_min": min(sm) if sm else None, "reasons": sorted({n for r in rows for n in r[3]}), "samples": len(sm)}
        if blocks and rows:
            bins = {}
            for t_end, ms in blocks:
                near = min(rows, key=lambda r: abs(r[0] - t_end))
                bins.setdefault(int(near[1]), []).append(ms)
            out["by_sm_mhz"] = {str(mhz): {"blocks": len(v), "ms_per_step_median": round(statistics.median(v), 5)}
                                for mhz, v in sorted(bins.items())}
        return out


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def oracle_sample(ck: pin.SuffixCheckpoint, layers, repeats: int = 1, threads=None):
    """Time the CPU checker (select + restore) on `layers` of the workload.  Returns (seconds per pass,
    bf16-equivalent bytes per pass, threads); `threads` None = all host cores."""
    import oracle
    g = ck.geom
    L = len(layers)
    mass = ck.mass.cpu().numpy().astype(np.uint64)[layers]
    pay = ck.payload.cpu().numpy()
    payloads = [pay[ck.layer_off[l]:ck.layer_off[l] + ck.layer_bytes[l]] for l in layers]
    sub = pin.Geometry(L, g.n_kv_heads, g.head_dim, g.rotary_dim, g.rope_style, g.rope_base, g.block_tokens,
                       g.page_tokens, g.group)
    shape = (L, ck.n_pages, g.page_tokens, g.n_kv_heads, g.head_dim)
    k = np.full(shape, pin.SENTINEL, dtype=np.uint16)
    v = np.full(shape, pin.SENTINEL, dtype=np.uint16)
    tags = ck.tags.cpu().numpy()[layers]
    off = ck.blk_off.cpu().numpy()[layers]
    table = ck.block_table.cpu().numpy()
    threads = oracle.max_threads() if threads is None else threads
    best, written = None, 0
    for _ in range(repeats):
        t0 = time.perf_counter()
        sel = oracle.select(mass, ck.n_suffix_tokens, g.block_tokens, ck.dirty_tokens, ck.top_k, ck.layer_mode)
        rc, _ = oracle.restore(L=L, H=g.n_kv_heads, D=g.head_dim, Dr=g.rotary_dim, rope_style=g.rope_style,
                               rope_base=g.rope_base, B=g.block_tokens, P=g.page_tokens, G=g.group, k_pool=k,
                               v_pool=v, strides=pin.pool_strides(sub, ck.n_pages), n_pages=ck.n_pages,
                               n=ck.n_suffix_tokens, delta=ck.delta, dst_shift=ck.dst_shift, block_table=table,
                               tags=tags, blk_off=off, layer_payload=payloads, reuse_idx=sel["reuse_idx"],
                               reuse_cnt=sel["reuse_cnt"], n_threads=threads)
        dt = time.perf_counter() - t0
        assert rc == 0
        best = dt if best is None else min(best, dt)
        written = int(sel["reuse_cnt"].sum()) * 2 * g.block_tokens * g.n_kv_heads * g.head_dim * 2
    return best, written, threads


def leg_failed(exc: Exception) -> dict:
    """What an optional leg reports when it raised (out of pinned memory on a small box, say): the headline line is
    still printed, with the reason in place of the leg's figures."""
    print(f"bench: optional leg failed: {exc!r}", file=sys.stderr)
    return {"error": repr(exc)[:300]}


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def max_over_ranks(x: float, world: int, device) -> float:
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(bytes_per_rank: float, ms: float, world: int) -> float:
    """Whole-job GB/s when every rank moved bytes_per_rank in ms (the max over ranks)."""
    return world * bytes_per_rank / (ms * 1e-3) / 1e9


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def median_ms(fn, stream, reps: int, warm: int = 3) -> float:
    """Median CUDA-event time of fn() over `reps` calls after `warm` untimed ones, each call waited for."""
    ts = []
    for i in range(warm + reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        fn()
        b.record(stream)
        b.synchronize()
        if i >= warm:
            ts.append(a.elapsed_time(b))
    return statistics.median(ts)


def r3(x):
    return None if x is None else float(f"{x:.4g}")


# ------------------------------------------------------------------------------------------ reference arm
def run_reference(args):
    """The CPU checker as the reference arm: each step is one pass of select + restore over all 32 layers of the
    same workload, on all host cores.  Rank 0 only."""
    rank, _, world = dist_env()
    if rank != 0:
        return
    import oracle
    oracle.build()
    ck = pin.config_llama8b(device="cpu")
    layers = list(range(ck.geom.n_layers))
    times = []
    written = 0
    for i in range(args.warmup + args.steps):
        dt, written, threads = oracle_sample(ck, layers)
        if i >= args.warmup:
            times.append(dt)
    total = sum(times)
    value = written * len(times) / total / 1e9
    sample = f"all {len(layers)} layers per step (select + restore of 870 reused blocks per layer), {threads} threads"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": workload_config(ck.delta, max(world, 1)),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------ our arm
def pinned_copy_ceiling(device, nbytes=1 << 30, reps=10):
    src = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
    dst = torch.empty(nbytes, dtype=torch.uint8, device=device)
    best = None
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        dst.copy_(src, non_blocking=True)
        e1.record()
        e1.synchronize()
        ms = e0.elapsed_time(e1)
        best = ms if best is None else min(best, ms)
    del src, dst
    return nbytes / (best * 1e-3) / 1e9


def copy_engine_table(device, total=1 << 28):
    """GB/s of pinned host-to-device copies by copy size, issued on one stream and alternating between two: what one
    copy costs the engine beyond its bytes, and whether a second stream hides it."""
    src = torch.empty(total, dtype=torch.uint8).pin_memory()
    dst = torch.empty(total, dtype=torch.uint8, device=device)
    streams = [torch.cuda.Stream(device=device) for _ in range(2)]
    out = {}
    for size in (64 << 10, 256 << 10, 1 << 20, 4 << 20, 64 << 20):
        n = min(total // size, 256)
        row = {}
        for ns in (1, 2):
            best = None
            for _ in range(3):
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                with torch.cuda.stream(streams[0]):
                    torch.cuda._sleep(30_000_000)           # ~15 ms: the copies queue up behind it, so the host's issue
                e0.record(streams[0])                       # rate is not what is measured
                streams[1].wait_event(e0)
                for i in range(n):
                    with torch.cuda.stream(streams[i % ns]):
                        dst[i * size:(i + 1) * size].copy_(src[i * size:(i + 1) * size], non_blocking=True)
                streams[0].wait_stream(streams[1])
                e1.record(streams[0])
                e1.synchronize()
                ms = e0.elapsed_time(e1)
                best = ms if best is None else min(best, ms)
            row[f"streams_{ns}"] = r3(n * size / (best * 1e-3) / 1e9)
        out[str(size)] = row
    del src, dst
    return out


def host_leg_on(ctx, cks, label, ceiling, dev, stream, reps=5):
    """restore_from_host of the sessions `cks` (pinned payloads) into a fresh pool: median time and link fractions."""
    from patchkv_inputs.staging import StagedCheckpoint, device_pool
    sts = [StagedCheckpoint(c, dev, payload_on_host=True) for c in cks]
    for s_ in sts:
        ctx.select_repair(s_.select_args(), stream)
    torch.cuda.synchronize()
    hk, hv, hpool = device_pool(cks[0], dev)
    hgeom = sts[0].geom()
    hss = [s_.host_session() for s_ in sts]
    useful = written = items_h = 0
    for c, s_ in zip(cks, sts):
        r_, w_, i_ = algorithmic_bytes(c, s_.reuse_idx.cpu().numpy(), s_.reuse_cnt.cpu().numpy())
        useful, written, items_h = useful + r_, written + w_, items_h + i_
    ts_, stats_ = [], None
    for i in range(2 + reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record(stream)
        rc_, stats_ = ctx.restore_from_host(hgeom, hpool, hss, stream)
        b.record(stream)
        b.synchronize()
        if i >= 2:
            ts_.append(a.elapsed_time(b))
    assert ctx.query_status() == 0 and stats_.bytes_useful == useful
    t_ms = statistics.median(ts_)
    out_ = {"workload": label, "ms": t_ms, "restored_kv_gbps_bf16_equiv": written / (t_ms * 1e-3) / 1e9,
            "payload_gbps": useful / (t_ms * 1e-3) / 1e9, "link_ceiling_gbps": ceiling,
            "frac_of_link": useful / (t_ms * 1e-3) / 1e9 / ceiling, "bytes_useful": int(useful),
            "bytes_copied": int(stats_.bytes_copied), "bytes_wasted": int(stats_.bytes_copied - useful),
            "bytes_direct": int(stats_.bytes_direct), "copies": int(stats_.n_copies), "block_layers": int(items_h),
            "block_layers_per_s": items_h / (t_ms * 1e-3)}
    del sts, hk, hv, hss
    torch.cuda.empty_cache()
    return out_


def run_ours(args):
    rank, local_rank, world = dist_env()
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    torch.cuda.set_device(local_rank)
    dev = torch.device(f"cuda:{local_rank}")

    from paper_2609_26219_b200 import binding as pk
    from paper_2609_26219_b200 import build as pkbuild
    from patchkv_inputs.staging import StagedCheckpoint, device_pool
    if rank == 0:
        pkbuild.build()
    barrier(world)
    ctx = pk.Context(device=local_rank)

    # ---- inputs, resident in HBM before the timed region
    over = {}
    if args.tags:                                           # profiling only: another mix of precision tags
        over["tag_probs"] = tuple(float(x) for x in args.tags.split(","))
        assert len(over["tag_probs"]) == 4
    ck = pin.config_llama8b(device=dev, n_layers=args.layers, **over)
    st = StagedCheckpoint(ck, dev)
    k, v, pool = device_pool(ck, dev)
    geom = st.geom()
    sel_args = st.select_args()
    sess = st.session()
    stream = torch.cuda.current_stream()

    def step(ev=None):
        ctx.select_repair(sel_args, stream)
        if ev:
            ev[0].record(stream)
        ctx.restore(geom, pool, [sess], stream)
        if ev:
            ev[1].record(stream)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    reuse_idx, reuse_cnt = st.reuse_idx.cpu().numpy(), st.reuse_cnt.cpu().numpy()
    read_b, written_b, items = algorithmic_bytes(ck, reuse_idx, reuse_cnt)

    # ---- timed region: blocks of K steps, CUDA events on the launching stream, clocks sampled alongside.  The block
    #      is repeated until at least MIN_TIMED_GPU_SECONDS of GPU time is covered (one short block would be ten
    #      milliseconds and a handful of clock samples); every rank times the same number of blocks.
    K = args.steps
    a0, b0 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a0.record(stream)
    for _ in range(3):
        step()
    b0.record(stream)
    b0.synchronize()
    est_ms = max_over_ranks(a0.elapsed_time(b0) / 3, world, dev)
    n_blocks = 1 if args.single_block else max(1, min(2000, int(np.ceil(MIN_TIMED_GPU_SECONDS * 1e3 / (K * est_ms)))))
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    blocks, restore_ms, probed = [], [], []
    barrier(world)
    torch.cuda.synchronize()
    t0 = time.time()
    for bi in range(2 * n_blocks):
        # Even blocks are the measurement: K steps between two events and nothing else on the stream.  Odd blocks carry
        # an event pair around every restore launch (that is where the roofline's kernel time comes from); those events
        # sit between select and restore and cost a few microseconds per step, so the odd blocks are not part of `value`.
        probe = bi % 2 == 1
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)] if probe else None
        e_begin, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e_begin.record(stream)
        for i in range(K):
            step(evs[i] if probe else None)
        e_end.record(stream)
        e_end.synchronize()
        if probe:
            probed.append(e_begin.elapsed_time(e_end) / K)
            restore_ms.extend(a.elapsed_time(b) for a, b in evs)
        else:
            blocks.append((time.time(), e_begin.elapsed_time(e_end) / K))
    torch.cuda.synchronize()
    barrier(world)
    t1 = time.time()
    clocks = sampler.stop(t0, t1, blocks)
    per_block = [ms for _, ms in blocks]
    ms_per_step = max_over_ranks(statistics.median(per_block), world, dev)
    restore_avg_ms = sum(restore_ms) / len(restore_ms)
    select_us = 1e3 * (statistics.median(per_block) - statistics.median(restore_ms)) if world == 1 else None
    value = aggregate_value(written_b, ms_per_step, world)
    timing = {"blocks": n_blocks, "steps_per_block": K, "gpu_seconds_timed": sum(per_block) * K * 1e-3,
              "ms_per_step_median": statistics.median(per_block), "ms_per_step_min": min(per_block),
              "ms_per_step_max": max(per_block), "restore_kernel_ms_median": statistics.median(restore_ms),
              "restore_kernel_ms_min": min(restore_ms), "restore_kernel_ms_max": max(restore_ms),
              "ms_per_step_with_inner_events_median": statistics.median(probed),
              "note": "value / ms_per_step: median over blocks of K steps with no event inside; the restore kernel's time "
                      "comes from interleaved blocks of the same K steps with an event pair around each restore launch"}
    assert ctx.query_status() == 0

    # ---- the same step captured once in a CUDA graph and replayed (select_repair + restore)
    graph_ms = None
    if world == 1 and not args.no_graph:
        try:
            side = torch.cuda.Stream()
            side.wait_stream(stream)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                ctx.select_repair(sel_args, side)
                ctx.restore(geom, pool, [sess], side)
            for _ in range(3):
                g.replay()
            n_rep = max(K, 100)
            ga, gb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            ga.record()
            for _ in range(n_rep):
                g.replay()
            gb.record()
            gb.synchronize()
            graph_ms = ga.elapsed_time(gb) / n_rep
            assert ctx.query_status() == 0
        except Exception as exc:           # reported, never fatal: the headline numbers do not depend on it
            graph_ms = f"unavailable: {type(exc).__name__}"

    peak, peak_kind = measured_hbm_peak()
    achieved = (read_b + written_b) / (restore_avg_ms * 1e-3) / 1e9
    traffic, traffic_src = captured_traffic(items, written_b)
    roofline = {"bound": "hbm", "kernel": "restore_pipe_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": f"of {peak_kind} copy bandwidth (burst)",
                "frac_of_nominal_8tbs": achieved / 8000.0, "traffic": traffic, "traffic_source": traffic_src,
                "algorithmic_bytes_per_launch": read_b + written_b, "kernel_ms": restore_avg_ms}

    # ---- offload side: write a checkpoint of all 1024 blocks x 32 layers from the pool (not on the resume path)
    writer = None
    if not args.no_writer:
        try:
            L_, NB_ = ck.geom.n_layers, ck.n_blocks
            w_off = torch.zeros((L_, NB_), dtype=torch.int64, device=dev)
            w_lb = torch.zeros(L_, dtype=torch.int64, device=dev)
            w_pay = torch.empty_like(st.payload)
            w_ptrs = torch.tensor([w_pay.data_ptr() + o for o in ck.layer_off], dtype=torch.int64, device=dev)
            w_sess = st.session(layer_payload=w_ptrs, blk_off=w_off, layer_bytes=w_lb)

            def write_once():
                ctx.plan_checkpoint(geom, ck.n_suffix_tokens, st.tags, w_off, w_lb, stream)
                ctx.quantize_gather(geom, pool, w_sess, stream)

            t_w = median_ms(write_once, stream, 30)         # a median over 30: single calls wander by a few per cent
            t_g = median_ms(lambda: ctx.quantize_gather(geom, pool, w_sess, stream), stream, 30)     # the encoder alone
            assert ctx.query_status() == 0 and torch.equal(w_off, st.blk_off)
            pool_read = 2 * L_ * NB_ * ck.geom.block_tokens * ck.geom.n_kv_heads * ck.geom.head_dim * 2
            pay_written = sum(ck.layer_bytes)
            # the same checkpoint streamed to pinned host memory (encode layer l+1 while layer l is copied out)
            cap_ = max(ck.layer_bytes)
            hbufs = [torch.empty(cap_, dtype=torch.uint8).pin_memory() for _ in range(L_)]
            hptrs = torch.tensor([h_.data_ptr() for h_ in hbufs], dtype=torch.int64)
            hcaps = torch.full((L_,), cap_, dtype=torch.int64)
            hsizes = torch.zeros(L_, dtype=torch.int64)
            t_h = median_ms(lambda: ctx.checkpoint_to_host(geom, pool, w_sess, hptrs, hcaps, hsizes, stream), stream, 4, warm=2)
            assert ctx.query_status() == 0 and int(hsizes.sum()) == pay_written
            src_ = torch.empty(1 << 30, dtype=torch.uint8, device=dev)
            dst_ = torch.empty(1 << 30, dtype=torch.uint8).pin_memory()
            d2h_best = None
            for i in range(6):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                dst_.copy_(src_, non_blocking=True)
                b.record()
                b.synchronize()
                d2h_best = a.elapsed_time(b) if d2h_best is None else min(d2h_best, a.elapsed_time(b))
            d2h_ceiling = (1 << 30) / (d2h_best * 1e-3) / 1e9
            del hbufs, src_, dst_
            writer = {"to_host": {"ms": t_h, "payload_gbps": pay_written / (t_h * 1e-3) / 1e9,
                                  "d2h_ceiling_gbps": d2h_ceiling, "frac_of_link": pay_written / (t_h * 1e-3) / 1e9 / d2h_ceiling},
                      "workload": "quantize_gather of all 1024 blocks x 32 layers of the same pool and tags",
                      "ms": t_w, "gather_ms": t_g, "gather_frac_of_hbm_peak": (pool_read + pay_written) / (t_g * 1e-3) / 1e9 / peak,
                      "real_gbps": (pool_read + pay_written) / (t_w * 1e-3) / 1e9,
                      "frac_of_hbm_peak": (pool_read + pay_written) / (t_w * 1e-3) / 1e9 / peak,
                      "bf16_gbps_read": pool_read / (t_w * 1e-3) / 1e9, "payload_bytes": int(pay_written)}
            del w_pay
        except Exception as exc:                          # an optional leg must not cost the bench line
            if world > 1:
                raise
            writer = leg_failed(exc)

    # ---- end to end: host buffers, copies inside the timed region
    e2e = None
    host_link = None
    if not args.no_e2e:
        try:
            ceiling = pinned_copy_ceiling(dev)
            hst = StagedCheckpoint(ck, dev, payload_on_host=True)
            mass_host = ck.mass.cpu().pin_memory()
            idx_host = torch.empty_like(hst.reuse_idx, device="cpu").pin_memory()
            cnt_host = torch.empty_like(hst.reuse_cnt, device="cpu").pin_memory()
            hsel = hst.select_args(host_reuse_idx=idx_host, host_reuse_cnt=cnt_host, sync_to_host=True)
            hs = hst.host_session(reuse_idx=idx_host, reuse_cnt=cnt_host)
            dir_bytes = ck.tags.numel() + ck.blk_off.numel() * 8 + idx_host.numel() * 4 + cnt_host.numel() * 4 + \
                ck.block_table.numel() * 4 + 16 * ck.geom.n_layers
            e2e_steps = max(3, min(args.steps, 10))
            times, copied = [], 0
            for i in range(3 + e2e_steps):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                barrier(world)
                a.record(stream)
                hst.mass.copy_(mass_host, non_blocking=True)                 # stored block masses: host -> device
                ctx.select_repair(hsel, stream)                               # lists also land in the pinned mirrors:
                rc, stats = ctx.restore_from_host(geom, pool, [hs], stream)   # the host planner reads them
                status = ctx.query_status()                                   # waits, reads the device status word back
                b.record(stream)                                              # ... inside the timed region
                b.synchronize()
                assert status == 0
                if i >= 3:
                    times.append(max_over_ranks(a.elapsed_time(b), world, dev))
                    copied = stats.bytes_copied
            e_ms = sum(times) / len(times)
            e2e = {"value": world * written_b / (e_ms * 1e-3) / 1e9, "unit": UNIT,
                   "h2d_bytes_per_step": int(copied + mass_host.numel() * 8 + dir_bytes),
                   "d2h_bytes_per_step": int(idx_host.numel() * 4 + cnt_host.numel() * 4 + 4),
                   "ms_per_step": e_ms, "steps": len(times),
                   "path": "pinned masses H2D, select_repair with pinned host mirrors of the lists (D2H, waited for), "
                           "restore_from_host (pinned payload), status word D2H (waited for); all inside the events"}
            host_link = {"ceiling_gbps": ceiling, "ceiling": "1 GiB pinned cudaMemcpyAsync H2D, best of 10, same run",
                         "payload_gbps": read_b / (e_ms * 1e-3) / 1e9, "frac": read_b / (e_ms * 1e-3) / 1e9 / ceiling,
                         "bytes_copied": int(copied), "bytes_useful": int(read_b), "copies": int(stats.n_copies)}
        except Exception as exc:                          # an optional leg must not cost the bench line
            if world > 1:
                raise
            e2e = leg_failed(exc)

    # ---- selection at scale: stored attention [32][32][64][16384] fp16 (2 GiB) -> masses -> lists
    select_scale = None
    if not args.no_scale_select:
        try:
            torch.cuda.empty_cache()
            gen = torch.Generator(device=dev)
            gen.manual_seed(1004)
            SL = args.scale_layers
            attn = pin.zipf_attention(gen, SL, 32, 64, 16384, dev)
            NBs = 1024
            out = dict(repair_mask=torch.empty((SL, NBs), dtype=torch.uint8, device=dev),
                       repair_idx=torch.empty((SL, NBs), dtype=torch.int32, device=dev),
                       repair_cnt=torch.empty(SL, dtype=torch.int32, device=dev),
                       reuse_idx=torch.empty((SL, NBs), dtype=torch.int32, device=dev),
                       reuse_cnt=torch.empty(SL, dtype=torch.int32, device=dev))
            mass_out = torch.empty((SL, NBs), dtype=torch.int64, device=dev)
            sa = pk.select_args(kind=pk.SCORE_ATTN_F16, n_layers=SL, n_suffix_tokens=16384, block_tokens=16,
                                dirty_tokens=640, top_k=32, layer_mode=pk.LAYERS_INDEPENDENT, attn=attn,
                                mass_out=mass_out, **out)
            t_ms = median_ms(lambda: ctx.select_repair(sa, stream), stream, 10)
            assert ctx.query_status() == 0 and int(out["reuse_cnt"][0]) == 952
            nbytes = attn.numel() * 2
            # the paper's token-level form from stored per-token scores: top 1.5 % of the suffix tokens, request-level
            tmass = pin.zipf_block_mass(gen, SL, 16384, dev)
            st_args = pk.select_args(kind=pk.SCORE_TOKEN_MASS, n_layers=SL, n_suffix_tokens=16384, block_tokens=16,
                                     dirty_tokens=640, top_k=245, layer_mode=pk.LAYERS_SHARED, mass=tmass, **out)
            token_form_us = 1e3 * median_ms(lambda: ctx.select_repair_tokens(st_args, stream), stream, 10)
            ta_args = pk.select_args(kind=pk.SCORE_ATTN_F16, n_layers=SL, n_suffix_tokens=16384, block_tokens=16,
                                     dirty_tokens=640, top_k=245, layer_mode=pk.LAYERS_SHARED, attn=attn, **out)
            token_form_attn_us = 1e3 * median_ms(lambda: ctx.select_repair_tokens(ta_args, stream), stream, 6)
            ti_args = pk.select_args(kind=pk.SCORE_ATTN_F16, n_layers=SL, n_suffix_tokens=16384, block_tokens=16,
                                     dirty_tokens=640, top_k=245, layer_mode=pk.LAYERS_INDEPENDENT, attn=attn, **out)
            token_form_attn_indep_us = 1e3 * median_ms(lambda: ctx.select_repair_tokens(ti_args, stream), stream, 6)
            select_scale = {"token_form_us_from_token_scores": token_form_us,
                            "token_form_us_from_attention": token_form_attn_us,
                            "token_form_attn_gbps": nbytes / (token_form_attn_us * 1e-6) / 1e9,
                            "token_form_attn_frac_of_hbm_peak": nbytes / (token_form_attn_us * 1e-6) / 1e9 / peak,
                            "token_form_us_from_attention_per_layer_sets": token_form_attn_indep_us,
                            "workload": f"stored attention fp16 [{SL}][32][64][16384] ({SL * 64} MiB), 40-block dirty window, top-32 per layer",
                            "select_us": 1e3 * t_ms, "attn_gbps": nbytes / (t_ms * 1e-3) / 1e9,
                            "frac_of_hbm_peak": nbytes / (t_ms * 1e-3) / 1e9 / peak, "launches": 3}
            del attn
            if SL == ck.geom.n_layers:
                # ... then the restore of the blocks that selection leaves to reuse (72 repaired / 952 reused per layer),
                # on the same 8B-shaped payload and pool as the headline step
                sa_lists = pk.select_args(kind=pk.SCORE_BLOCK_MASS, n_layers=SL, n_suffix_tokens=16384, block_tokens=16,
                                          dirty_tokens=640, top_k=32, layer_mode=pk.LAYERS_INDEPENDENT, mass=mass_out, **out)
                ctx.select_repair(sa_lists, stream)               # the lists of the block form, from the masses just computed
                torch.cuda.synchronize()
                sess4 = st.session(reuse_idx=out["reuse_idx"], reuse_cnt=out["reuse_cnt"])
                r4, w4, items4 = algorithmic_bytes(ck, out["reuse_idx"].cpu().numpy(), out["reuse_cnt"].cpu().numpy())
                r_ms = median_ms(lambda: ctx.restore(geom, pool, [sess4], stream), stream, 10)
                assert ctx.query_status() == 0
                select_scale["restore_of_its_reuse_set"] = {
                    "ms": r_ms, "block_layers": int(items4), "restored_kv_gbps_bf16_equiv": w4 / (r_ms * 1e-3) / 1e9,
                    "real_gbps": (r4 + w4) / (r_ms * 1e-3) / 1e9, "frac_of_hbm_peak": (r4 + w4) / (r_ms * 1e-3) / 1e9 / peak}
        except Exception as exc:                          # an optional leg must not cost the bench line
            if world > 1:
                raise
            select_scale = leg_failed(exc)

    # ---- the two host-resident workloads: 7B-shaped / 4 KV heads (one session), 70B-shaped stress (8 sessions)
    host_cfg3 = stress = None
    ceiling = None
    if not args.no_host_configs:
        try:
            ceiling = pinned_copy_ceiling(dev)
            ctx_direct = pk.Context(device=local_rank, flags=pk.FLAG_HOST_DIRECT)
            ctx_staged = pk.Context(device=local_rank, flags=pk.FLAG_HOST_STAGED)

            def host_leg(cks, label, reps=5, both=False):
                out_ = host_leg_on(ctx, cks, label, ceiling, dev, stream, reps)
                if both:     # the same with staging copies only, and with none (the kernel pulls every record itself)
                    for name_, c_ in (("staged_only", ctx_staged), ("zero_copy", ctx_direct)):
                        d_ = host_leg_on(c_, cks, label, ceiling, dev, stream, reps)
                        out_[name_] = {k_: d_[k_] for k_ in ("ms", "payload_gbps", "frac_of_link", "bytes_copied", "bytes_wasted", "copies")}
                return out_

            try:
                del st, k, v
            except NameError:
                pass
            torch.cuda.empty_cache()
            c3 = pin.config_7b_host(device=dev, pin_payload=True)
            host_cfg3 = host_leg([c3], "7b-shaped: L=28 H=4 D=128 base=1e6 n=32768 delta=-3000, pinned host payload, "
                                       "4096-page pool (2x), shuffled free list", both=True)
            del c3
            SLy = args.stress_layers
            waves = []
            for w_ in range(args.stress_waves):          # each wave: SLy of the 80 layers, payload regenerated outside the timed region
                wave_sess = pin.stress_wave(w_, device=dev, layers=SLy)
                waves.append(host_leg(wave_sess, "", reps=3, both=(w_ == 0)))
                del wave_sess
            stress = dict(waves[0])
            stress["workload"] = (f"70b-shaped stress: 8 sessions x 64k-token suffix, H=8 D=128, int4 share 10-60 %, one shared pool "
                                  f"of 32768 pages, pinned host payload; {SLy} of 80 layers resident per wave, {len(waves)} wave(s) "
                                  f"timed (fit rule: the 80-layer pool is 172 GB and its payload 103 GB of pinned memory)")
            tot_ms = sum(w["ms"] for w in waves)
            tot_useful = sum(w["bytes_useful"] for w in waves)
            stress.update(ms=tot_ms, bytes_useful=tot_useful, layers_covered=SLy * len(waves), waves=len(waves),
                          wave_ms=[round(w["ms"], 2) for w in waves],
                          bytes_copied=sum(w["bytes_copied"] for w in waves), bytes_wasted=sum(w["bytes_wasted"] for w in waves),
                          copies=sum(w["copies"] for w in waves),
                          payload_gbps=tot_useful / (tot_ms * 1e-3) / 1e9,
                          frac_of_link=tot_useful / (tot_ms * 1e-3) / 1e9 / ceiling,
                          block_layers=sum(w["block_layers"] for w in waves),
                          block_layers_per_s=sum(w["block_layers"] for w in waves) / (tot_ms * 1e-3),
                          restored_kv_gbps_bf16_equiv=sum(w["restored_kv_gbps_bf16_equiv"] * w["ms"] for w in waves) / tot_ms)
        except Exception as exc:                          # an optional leg must not cost the bench line
            if world > 1:
                raise
            host_cfg3 = host_cfg3 or leg_failed(exc)
            stress = stress or leg_failed(exc)

    # ---- the paper's restore microbenchmark shape (Section V-E): an ~8k-token checkpoint of a 64-layer, 8-KV-head,
    #      head_dim-128 model (geometry from the public Qwen3-32B model card, not from the paper), 32-token blocks,
    #      one fp16 scale per 128 channels, restored whole from pinned host memory in each transport format
    paper_shape = None
    if not args.no_host_configs and ceiling is not None:
        try:
            gm = pin.Geometry(64, 8, 128, 128, pin.ROPE_HALF, 1.0e6, 32, 32, 128)
            rows = {}
            for label, probs in (("FP16(bf16)", (1.0, 0, 0, 0)), ("INT8 K8/V8", (0, 1.0, 0, 0)), ("INT4 K4/V4", (0, 0, 0, 1.0)),
                                 ("mixed 2/6/92 % bf16/K8V8/K8V4", (0.02, 0.06, 0.92, 0.0))):
                cm = pin.make_checkpoint(name="paper-microbench", seed=2024, geom=gm, n=8031, delta=-512, tag_probs=probs,
                                         n_outlier=6, outlier_scale=10.0, n_pages=256, dirty_tokens=0, top_k=0,
                                         device=dev, pin_payload=True)
                r_ = host_leg_on(ctx, [cm], label, ceiling, dev, stream, reps=5)
                rows[label] = {"payload_mib": r_["bytes_useful"] / 2 ** 20, "fetch_and_restore_ms": r_["ms"],
                               "payload_gbps": r_["payload_gbps"], "frac_of_link": r_["frac_of_link"], "copies": r_["copies"]}
                del cm
            paper_shape = {"workload": "8031-token checkpoint, L=64 H=8 D=128, B=P=32, G=128, every block restored from pinned host",
                           "formats": rows,
                           "paper_context_ms": {"FP16": 344.4, "INT8": 183.6, "INT4": 107.2, "PatchKV": 158.0,
                                                "hardware": "A800 server, PCIe Gen4, 23.3 GiB/s pinned ceiling"}}
        except Exception as exc:                          # an optional leg must not cost the bench line
            if world > 1:
                raise
            paper_shape = leg_failed(exc)

    # ---- CPU baseline: the checker, as it stands, on a bounded sample of the same workload (rank 0, N = 1)
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu:
        try:
            import oracle
            oracle.build()
            sample_layers = list(range(ck.geom.n_layers))
            dt, wb, threads = oracle_sample(ck, sample_layers, repeats=3)
            one_layers = sample_layers[:min(4, len(sample_layers))]
            dt1, wb1, _ = oracle_sample(ck, one_layers, repeats=1, threads=1)
            cpu_baseline = {"value": wb / dt / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle",
                            "sample": f"all {len(sample_layers)} layers of the workload (select + restore), best of 3 passes "
                                      f"of {dt:.2f} s on {threads} threads",
                            "single_thread": {"value": wb1 / dt1 / 1e9, "unit": UNIT,
                                              "sample": f"{len(one_layers)} layers, one pass of {dt1:.2f} s on 1 thread"}}
        except Exception as exc:                          # an optional leg must not cost the bench line
            if world > 1:
                raise
            cpu_baseline = leg_failed(exc)

    if rank == 0:
        def get(d, *path):
            for p_ in path:
                if not isinstance(d, dict) or p_ not in d:
                    return None
                d = d[p_]
            return d
        # one compact row per BASELINE configuration; kept as the LAST key so that it is what a truncated record shows
        configs = {
            "1_tiny": "parity only (latency-sized)",
            "2_llama8b_device": {"ms": r3(ms_per_step), "gbps_bf16eq": r3(value), "frac_hbm": r3(roofline["frac"]),
                                 "select_us": r3(select_us), "restore_kernel_ms": r3(restore_avg_ms)},
            "3_7b_host": {"ms": r3(get(host_cfg3, "ms")), "gbps_bf16eq": r3(get(host_cfg3, "restored_kv_gbps_bf16_equiv")),
                          "frac_link": r3(get(host_cfg3, "frac_of_link")),
                          "staged_only_frac_link": r3(get(host_cfg3, "staged_only", "frac_of_link")),
                          "zero_copy_frac_link": r3(get(host_cfg3, "zero_copy", "frac_of_link"))},
            "4_select_scale": {"select_us": r3(get(select_scale, "select_us")), "frac_hbm": r3(get(select_scale, "frac_of_hbm_peak")),
                               "token_form_us": r3(get(select_scale, "token_form_us_from_attention")),
                               "token_form_frac_hbm": r3(get(select_scale, "token_form_attn_frac_of_hbm_peak")),
                               "restore_ms": r3(get(select_scale, "restore_of_its_reuse_set", "ms")),
                               "restore_gbps_bf16eq": r3(get(select_scale, "restore_of_its_reuse_set", "restored_kv_gbps_bf16_equiv")),
                               "restore_frac_hbm": r3(get(select_scale, "restore_of_its_reuse_set", "frac_of_hbm_peak"))},
            "5_stress": {"ms": r3(get(stress, "ms")), "gbps_bf16eq": r3(get(stress, "restored_kv_gbps_bf16_equiv")),
                         "frac_link": r3(get(stress, "frac_of_link")), "layers_covered": get(stress, "layers_covered"),
                         "payload_gb": r3((get(stress, "bytes_useful") or 0) / 1e9)},
            "e2e_llama8b_host": {"ms": r3(get(e2e, "ms_per_step")), "gbps_bf16eq": r3(get(e2e, "value")),
                                 "frac_link": r3(get(host_link, "frac"))},
            "writer": {"ms": r3(get(writer, "ms")), "frac_hbm": r3(get(writer, "frac_of_hbm_peak")),
                       "gather_ms": r3(get(writer, "gather_ms")), "gather_frac_hbm": r3(get(writer, "gather_frac_of_hbm_peak")),
                       "to_host_frac_link": r3(get(writer, "to_host", "frac_of_link"))},
        }
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": workload_config(ck.delta, world, args.layers, args.tags),
            "clocks": clocks, "e2e": e2e, "gpu_launches": 2 * K * n_blocks,
            "gpu_launches_note": f"{n_blocks} timed block(s) x {K} steps x (select_kernel + restore_pipe_kernel); as many again in the interleaved probe blocks",
            "roofline": roofline, "cpu_baseline": cpu_baseline, "timing": timing,
            "select_us": select_us, "restore_ms": restore_avg_ms, "cuda_graph_ms_per_step": graph_ms,
            "block_layers_per_s": world * items / (ms_per_step * 1e-3),
            "real_gbps": world * (read_b + written_b) / (ms_per_step * 1e-3) / 1e9,
            "host_link": host_link, "select_at_scale": select_scale, "host_7b": host_cfg3, "stress": stress,
            "writer": writer, "paper_microbench_shape": paper_shape, "configs": configs,
        }
        print(json.dumps(line), flush=True)
    ctx.close()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------ sweeps
def run_sweep(args):
    """Restore and writer fractions by tag and by geometry, restore time by suffix length, and the merge-gap sweep of
    the host path, each on a workload of at most about 2 GB (half of the benchmark's 32 layers).  One JSON line."""
    torch.cuda.set_device(0)
    dev = torch.device("cuda:0")
    from paper_2609_26219_b200 import binding as pk
    from paper_2609_26219_b200 import build as pkbuild
    from patchkv_inputs.staging import StagedCheckpoint, device_pool
    pkbuild.build()
    ctx = pk.Context(device=0)
    stream = torch.cuda.current_stream()
    peak, peak_kind = measured_hbm_peak()
    LH = 16
    G = pin.Geometry

    def restore_row(ck, reps=20, queued=False):
        st = StagedCheckpoint(ck, dev)
        k, v, pool = device_pool(ck, dev)
        geom = st.geom()
        sa = st.select_args()
        ctx.select_repair(sa, stream)
        torch.cuda.synchronize()
        sess = st.session()
        r, w, items = algorithmic_bytes(ck, st.reuse_idx.cpu().numpy(), st.reuse_cnt.cpu().numpy())
        ms = median_ms(lambda: ctx.restore(geom, pool, [sess], stream), stream, reps, warm=5)
        sel_us = 1e3 * median_ms(lambda: ctx.select_repair(sa, stream), stream, reps, warm=3)
        row = {"us": r3(1e3 * ms), "gbps": r3((r + w) / ms / 1e6), "frac_hbm": r3((r + w) / ms / 1e6 / peak),
               "block_layers": items, "select_us": r3(sel_us)}
        if queued:
            # fifty calls queued back to back between two events: the caller's launch path (argument marshalling, the
            # library's checks, the launch itself) then overlaps the previous call's kernel instead of an idle GPU
            ts = []
            for _ in range(5):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for _ in range(50):
                    ctx.restore(geom, pool, [sess], stream)
                e1.record(stream)
                e1.synchronize()
                ts.append(e0.elapsed_time(e1) / 50)
            q = statistics.median(ts)
            t0 = time.perf_counter()
            for _ in range(200):
                ctx.restore(geom, pool, [sess], stream)
            host_us = (time.perf_counter() - t0) / 200 * 1e6
            torch.cuda.synchronize()
            row.update({"us_queued": r3(1e3 * q), "frac_hbm_queued": r3((r + w) / q / 1e6 / peak), "host_us_per_call": r3(host_us)})
        assert ctx.query_status() == 0
        del st, k, v, pool
        torch.cuda.empty_cache()
        return row

    def writer_row(ck, reps=20):
        g = ck.geom
        st = StagedCheckpoint(ck, dev)
        k, v, pool = device_pool(ck, dev)
        k.view(torch.bfloat16).normal_()
        v.view(torch.bfloat16).normal_()
        geom = st.geom()
        L, NB = g.n_layers, ck.n_blocks
        off = torch.zeros((L, NB), dtype=torch.int64, device=dev)
        lb = torch.zeros(L, dtype=torch.int64, device=dev)
        ctx.plan_checkpoint(geom, ck.n_suffix_tokens, st.tags, off, lb)
        torch.cuda.synchronize()
        sizes = [int(x) for x in lb.cpu()]
        starts = [sum(-(-s // 256) * 256 for s in sizes[:i]) for i in range(L)]
        out = torch.empty(starts[-1] + sizes[-1] + 256, dtype=torch.uint8, device=dev)
        ptrs = torch.tensor([out.data_ptr() + o for o in starts], dtype=torch.int64, device=dev)
        ws = pk.make_session(n_suffix_tokens=ck.n_suffix_tokens, delta=0, dst_shift=ck.dst_shift, block_table=st.block_table,
                             tags=st.tags, blk_off=off, layer_payload=ptrs, layer_bytes=lb, reuse_idx=None, reuse_cnt=None)
        ms = median_ms(lambda: ctx.quantize_gather(geom, pool, ws, stream), stream, reps, warm=5)
        assert ctx.query_status() == 0
        rd = 2 * L * NB * g.block_tokens * g.n_kv_heads * g.head_dim * 2
        wr = sum(sizes)
        del st, k, v, pool, out
        torch.cuda.empty_cache()
        return {"us": r3(1e3 * ms), "gbps": r3((rd + wr) / ms / 1e6), "frac_hbm": r3((rd + wr) / ms / 1e6 / peak)}

    def mk(geom, n, seed, probs=pin.MIX, delta=300, shift=0):
        nb = -(-n // geom.block_tokens)
        pages = -(-(nb * geom.block_tokens + shift) // geom.page_tokens) + 64
        return pin.make_checkpoint(name="sweep", seed=seed, geom=geom, n=n, delta=delta, dst_shift=shift, tag_probs=probs,
                                   n_outlier=6, outlier_scale=10.0, n_pages=pages, dirty_tokens=int(0.088 * n),
                                   top_k=max(1, nb // 16), device=dev)

    out = {"peak_gbps": peak, "peak_kind": peak_kind, "layers": LH,
           "note": "half-size workloads (16 layers, <= 2 GB resident); fractions of the measured HBM copy bandwidth"}
    base = G(LH, 8, 128, 128, pin.ROPE_HALF, 5e5, 16, 16, 32)
    by_tag = {}
    for name, probs in (("mix_30_50_20", pin.MIX), ("bf16", (1, 0, 0, 0)), ("k8v8", (0, 1, 0, 0)), ("k8v4", (0, 0, 1, 0)),
                        ("k4v4", (0, 0, 0, 1))):
        row = {}
        for delta in (429, 0):
            row[f"restore_delta{delta}"] = restore_row(mk(base, 16384, 1002, probs, delta))
        row["writer"] = writer_row(mk(base, 16384, 1002, probs))
        by_tag[name] = row
    out["by_tag"] = by_tag
    geoms = {
        "H16_D128_B16": (G(LH, 16, 128, 128, pin.ROPE_HALF, 1e4, 16, 16, 32), 8192),
        "H8_D128_B16": (base, 16384),
        "H8_D128_B32_P32_G128": (G(LH, 8, 128, 128, pin.ROPE_HALF, 1e6, 32, 32, 128), 16384),
        "H8_D128_interleaved": (G(LH, 8, 128, 128, pin.ROPE_INTERLEAVED, 5e5, 16, 16, 32), 16384),
        "H8_D128_P32_shift5": (G(LH, 8, 128, 128, pin.ROPE_HALF, 5e5, 16, 32, 32), 16384),
        "H4_D128_B16": (G(LH, 4, 128, 128, pin.ROPE_HALF, 1e6, 16, 16, 32), 32768),
        "H8_D64_B16": (G(LH, 8, 64, 64, pin.ROPE_HALF, 1e4, 16, 16, 32), 32768),
        "H2_D128_B16": (G(LH, 2, 128, 128, pin.ROPE_HALF, 1e6, 16, 16, 32), 65536),
        "H2_D128_B32": (G(LH, 2, 128, 128, pin.ROPE_HALF, 1e6, 32, 32, 32), 65536),
        "H4_D64_B16": (G(LH, 4, 64, 64, pin.ROPE_HALF, 1e4, 16, 16, 32), 65536),
    }
    by_geom = {}
    for name, (gm, n) in geoms.items():
        shift = 5 if "shift5" in name else 0
        row = restore_row(mk(gm, n, 7, shift=shift))
        # the same with half the layers: the slope between the two sizes leaves the launch's fixed cost out
        half_geom = dataclasses.replace(gm, n_layers=LH // 2)
        small = restore_row(mk(half_geom, n, 7, shift=shift))
        bytes_full, bytes_half = row["gbps"] * row["us"], small["gbps"] * small["us"]
        row["frac_hbm_marginal"] = r3((bytes_full - bytes_half) / (row["us"] - small["us"]) / peak)
        by_geom[name] = {"restore": row, "writer": writer_row(mk(gm, n, 7, shift=shift))}
    out["by_geometry"] = by_geom
    out["by_suffix_tokens"] = {str(n): restore_row(mk(G(32, 8, 128, 128, pin.ROPE_HALF, 5e5, 16, 16, 32), n, 1002), reps=30, queued=True)
                               for n in (256, 1024, 2048, 4096, 8192, 16384)}
    # merge-gap sweep of the staged host path on the 16-layer 8B-shaped payload, and the zero-copy mode
    ceiling = pinned_copy_ceiling(dev)
    ck = mk(base, 16384, 1002)
    ck.payload = ck.payload.cpu().pin_memory()
    gaps = {}
    for gap in (0, 32 << 10, 64 << 10, 128 << 10, 256 << 10, 1 << 20):
        c = pk.Context(device=0, merge_gap_bytes=gap, flags=pk.FLAG_HOST_STAGED)
        r = host_leg_on(c, [ck], "", ceiling, dev, stream, reps=5)
        gaps[str(gap)] = {"ms": r3(r["ms"]), "frac_link": r3(r["frac_of_link"]), "copies": r["copies"],
                          "wasted_frac": r3(r["bytes_wasted"] / r["bytes_useful"])}
        c.close()
    c = pk.Context(device=0, flags=pk.FLAG_HOST_DIRECT)
    r = host_leg_on(c, [ck], "", ceiling, dev, stream, reps=5)
    c.close()
    r0 = host_leg_on(ctx, [ck], "", ceiling, dev, stream, reps=5)
    out["host_path"] = {"link_ceiling_gbps": r3(ceiling), "copy_engine_gbps_by_copy_bytes": copy_engine_table(dev),
                        "staged_only_by_merge_gap_bytes": gaps,
                        "zero_copy": {"ms": r3(r["ms"]), "frac_link": r3(r["frac_of_link"])},
                        "default_hybrid": {"ms": r3(r0["ms"]), "frac_link": r3(r0["frac_of_link"]), "copies": r0["copies"],
                                           "direct_frac": r3(r0["bytes_direct"] / r0["bytes_useful"]),
                                           "wasted_frac": r3(r0["bytes_wasted"] / r0["bytes_useful"])}}
    print(json.dumps({"sweep": out}), flush=True)
    ctx.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sweep", action="store_true",
                    help="print the per-tag / per-geometry / suffix-length / merge-gap sweeps instead of the benchmark line")
    ap.add_argument("--single-block", action="store_true", help="profiling only: time one block of --steps steps")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-scale-select", action="store_true")
    ap.add_argument("--no-host-configs", action="store_true")
    ap.add_argument("--no-writer", action="store_true")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--stress-layers", type=int, default=pin.STRESS_WAVE_LAYERS)
    ap.add_argument("--stress-waves", type=int, default=pin.STRESS_LAYERS // pin.STRESS_WAVE_LAYERS,
                    help="8 waves of 10 layers cover the full 80-layer stress config (the default)")
    ap.add_argument("--scale-layers", type=int, default=32, help="layers of the selection-at-scale leg (profiling: fewer)")
    ap.add_argument("--tags", default="",
                    help="profiling only: shares of the tags bf16,K8V8,K8V4,K4V4 instead of the workload's 0.3,0.5,0.2,0")
    ap.add_argument("--layers", type=int, default=32,
                    help="profiling only: fewer layers of the same workload (the bench line is quoted on 32)")
    args = ap.parse_args()
    if int(os.environ.get("WORLD_SIZE", 1)) > 1:
        # multi-rank runs time the headline step and the end-to-end leg only: the extra legs pin tens of GB of host
        # memory per rank and say nothing about scaling
        args.no_host_configs = args.no_writer = args.no_scale_select = args.no_graph = True
    if args.impl == "reference":
        run_reference(args)
    elif args.sweep:
        run_sweep(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
