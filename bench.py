#!/usr/bin/env python
"""Benchmark of the descriptor-driven tensor mover on B200.

One step = one pass of the whole hot path over one batch of synthetic input:
  a1 KV pack      device NHD pool -> packed request-level HND buffer     (every wave)
  a2 KV unpack    packed HND buffer -> fresh blocks of a second NHD pool (every wave)
  a3 KV migrate   pool -> pool through independent block tables          (every wave)
  a4 weights      flat blob -> 291 per-parameter tensors
  a5 weights      flat blob -> tensor-parallel shard `rank` of 8
on the Llama-3-8B-shaped workloads (KV offload/reload requests with log-normal lengths in a
fragmented 20,000-block pool; the 16 GB checkpoint blob).  `value` is the device-timed
aggregate with every buffer resident in HBM (read + written bytes per second); `e2e` runs
the same calls with the packed buffer and the blob in pinned HOST memory, so that every byte
crosses the host link inside the timed region (zero-copy kernel loads / stores).

Prints ONE JSON line.  `--impl reference` times the CPU oracle instead (bounded sample).
Under torchrun every rank runs an independent replica (the path has no exchange step).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

GB = 1e9


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return 6650.0, "fallback"


# --------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        busy = [c for c in sm if c > 500] or sm
        return {"sm_mhz": statistics.median(busy) if busy else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------------------
# CPU oracle leg (cpu_baseline / --impl reference)
# --------------------------------------------------------------------------------------
class OracleSample:
    """The oracle, as it stands, on a bounded sample of the same workload: the requests of
    wave 0 of a scaled-down pool (`sample_blocks` blocks) packed NHD -> HND and unpacked again
    through an independent block table.  run() returns (GB/s in read+write bytes, seconds)."""

    def __init__(self, sample_blocks: int, threads: int):
        import oracle
        self.oracle, self.threads = oracle, threads
        self.shape = shape = wl.LLAMA3_8B_KV
        NBs = sample_blocks
        # the first requests of the workload, in order, that fit the sample's block budget
        T_all = wl.config2()[2]
        keep, used = [], 0
        for t in T_all:
            n = (int(t) + shape.B - 1) // shape.B
            if used + n <= NBs:
                keep.append(int(t))
                used += n
        T = np.array(keep, dtype=np.int64)
        off = np.concatenate([[0], np.cumsum((T + shape.B - 1) // shape.B)]).astype(np.int64)
        rng = np.random.default_rng(wl.SEED_BASE + 20)
        self.src = wl.KVRequests(T, off, rng.permutation(NBs)[:off[-1]].astype(np.int32))
        self.dst = wl.KVRequests(T, off, rng.permutation(NBs)[:off[-1]].astype(np.int32))
        self.threads = threads = max(1, min(threads, len(T)))
        pool = np.zeros(NBs * shape.block_bytes, dtype=np.uint8)
        try:
            import torch
            on_gpu = torch.cuda.is_available()
        except Exception:
            on_gpu = False
        if on_gpu:  # same counter-based contents, generated faster
            t = torch.empty(pool.size, dtype=torch.uint8, device="cuda")
            wl.fill_torch(t, wl.SEED_BASE + 2)
            pool[:] = t.cpu().numpy()
            del t
        else:
            wl.fill_np(pool, wl.SEED_BASE + 2)
        per = NBs * shape.chunk_bytes
        self.planes = [pool[p * per:(p + 1) * per] for p in range(shape.L * 2)]
        self.packed = np.zeros(oracle.packed_nbytes(shape.tuple, self.src.T), dtype=np.uint8)
        pool2 = np.zeros_like(pool)
        pool2.fill(0)            # touch the pages now: page faults are not part of the oracle's time
        self.packed.fill(0)
        self.planes2 = [pool2[p * per:(p + 1) * per] for p in range(shape.L * 2)]
        self.desc = (f"oracle kv_pack NHD->HND + kv_unpack of {len(self.src.T)} requests / {self.src.n_blocks} blocks "
                     f"({self.packed.size / GB:.2f} GB payload) of the Llama-3-8B KV workload, {threads} threads")

    def run(self):
        o, s, src, dst = self.oracle, self.shape, self.src, self.dst
        t0 = time.perf_counter()
        o.kv_pack(s.tuple, o.NHD, s.chunk_bytes, self.planes, src.T, src.bt_off, src.bt, o.HND, self.packed, threads=self.threads)
        o.kv_unpack(s.tuple, o.NHD, s.chunk_bytes, self.planes2, dst.T, dst.bt_off, dst.bt, o.HND, self.packed, threads=self.threads)
        dt = time.perf_counter() - t0
        return 2 * 2 * self.packed.size / dt / GB, dt


def run_reference(args):
    """`--impl reference`: the oracle is the reference arm of this tier."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    threads = os.cpu_count() or 1
    sample = OracleSample(args.oracle_blocks, threads)
    vals, dts = [], []
    for i in range(args.warmup + args.steps):
        v, dt = sample.run()
        if i >= args.warmup:
            vals.append(v)
            dts.append(dt)
    value = statistics.mean(vals)
    desc, threads = sample.desc, sample.threads
    line = {
        "impl": "reference", "metric": "kv_pack_unpack_and_weight_materialise_GBps", "value": value, "unit": "GB/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * statistics.mean(dts),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": WORKLOAD_NAME, "sample": desc},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


WORKLOAD_NAME = ("configs[1] Llama-3-8B KV offload/reload (20000-block NHD pool, 256 log-normal requests in waves, "
                 "packed HND) for rows a1-a3 + configs[2] Llama-3-8B weight blob (291 tensors, full + 1-of-8 shard) for rows a4-a5")


# --------------------------------------------------------------------------------------
# the CUDA arm
# --------------------------------------------------------------------------------------
class Ranks:
    """One process per GPU, replicas only: torch.distributed serves the barrier around the timed
    region and the max-over-ranks of the device time; no data-path collective exists."""

    def __init__(self, backend: str):
        import torch.distributed as dist
        self.dist = dist
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        self.backend = backend
        if self.world > 1:
            kw = {}
            if backend == "nccl":
                import torch
                kw["device_id"] = torch.device("cuda", self.local)
            dist.init_process_group(backend, **kw)

    def barrier(self):
        if self.backend == "nccl":
            import torch
            torch.cuda.synchronize()
        if self.world > 1:
            self.dist.barrier()
            if self.backend == "nccl":
                import torch
                torch.cuda.synchronize()

    def max_ms(self, ms: float) -> float:
        if self.world == 1:
            return ms
        import torch
        t = torch.tensor([ms], dtype=torch.float64, device="cuda" if self.backend == "nccl" else "cpu")
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def throughput(self, bytes_per_rank_per_step: int, steps: int, ms: float) -> float:
        """Whole-job GB/s: every rank moved the same bytes; the job took the slowest rank's time."""
        return self.world * bytes_per_rank_per_step * steps / (self.max_ms(ms) * 1e-3) / GB

    def close(self):
        if self.world > 1:
            self.dist.destroy_process_group()


def run_dry(args):
    """`--dry-run`: no GPU work; exercises the multi-rank plumbing (rendezvous, barrier,
    max over ranks, whole-job aggregation) with a made-up per-rank time, for CPU tests."""
    ranks = Ranks("gloo")
    ranks.barrier()
    ms = 100.0 + 50.0 * ranks.rank
    step_bytes = 10 ** 9
    value = ranks.throughput(step_bytes, args.steps, ms * args.steps)
    ranks.barrier()
    if ranks.rank == 0:
        print(json.dumps({"metric": "kv_pack_unpack_and_weight_materialise_GBps", "value": value, "unit": "GB/s",
                          "n_gpus": ranks.world, "steps": args.steps, "warmup": args.warmup, "scaling": "weak",
                          "ms_per_step": ranks.max_ms(ms) if ranks.world == 1 else 100.0 + 50.0 * (ranks.world - 1),
                          "dry_run": True}))
    ranks.close()


class Row:
    def __init__(self, name, mode):
        self.name, self.mode = name, mode
        self.bytes = 0       # algorithmic bytes (read + written) per step
        self.launches = 0    # launches per step
        self.ms = []         # per-step device ms (sum over its launches)


def run_ours(args):
    import torch

    import paper_2608_06007_b200 as tc

    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    ranks = Ranks("nccl")
    world, rank, local = ranks.world, ranks.rank, ranks.local
    tc.load_library()
    # the CPU baseline goes first, while the host's memory is still unfragmented (the 50+ GB of
    # pinned buffers allocated and freed below slow the oracle down 3-4x if it runs after them)
    threads = os.cpu_count() or 1
    cpu_v, cpu_desc = None, "skipped"
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sample = OracleSample(args.oracle_blocks, threads)
        cpu_v, _ = sample.run()
        cpu_desc, threads = sample.desc, sample.threads
        del sample
    free, total = torch.cuda.mem_get_info()
    shape = wl.LLAMA3_8B_KV
    NB = args.kv_blocks
    wave_blocks = args.wave_blocks
    ck = wl.config3() if not args.small else wl.llama_checkpoint(layers=1, vocab=16032)
    need = NB * shape.block_bytes + 2 * wave_blocks * shape.block_bytes + 2.2 * ck.nbytes_total
    while need > 0.8 * free and NB > 1024:
        NB //= 2
        wave_blocks = min(wave_blocks, NB // 2)
        need = NB * shape.block_bytes + 2 * wave_blocks * shape.block_bytes + 2.2 * ck.nbytes_total
    _, _, T_all, waves = wl.config2(NB=NB, R=args.requests, wave_blocks=wave_blocks, NB_dst=wave_blocks)
    if args.max_waves:
        waves = waves[:args.max_waves]
    u8 = dict(dtype=torch.uint8, device="cuda")
    poolA = torch.empty(NB * shape.block_bytes, **u8)
    wl.fill_torch(poolA, wl.SEED_BASE + 2)
    poolB = torch.empty(wave_blocks * shape.block_bytes, **u8)
    poolB.fill_(0xA5)
    max_packed = max(int(w[0].T.sum()) for w in waves) * shape.token_bytes
    Q = torch.empty(max_packed, **u8)
    blob = torch.empty(ck.nbytes_total, **u8)
    wl.fill_torch(blob, wl.SEED_BASE + 3, "normal")
    W = 8
    full_sizes = [ck.nbytes(i) for i in range(ck.N)]
    shard_sizes = [ck.nbytes(i) // (W if ck.split_dim[i] >= 0 else 1) for i in range(ck.N)]
    dst_full = torch.empty(sum(full_sizes), **u8)
    dst_shard = torch.empty(sum(shard_sizes), **u8)
    full_ptrs = [dst_full.data_ptr() + int(o) for o in np.concatenate([[0], np.cumsum(full_sizes)])[:-1]]
    shard_ptrs = [dst_shard.data_ptr() + int(o) for o in np.concatenate([[0], np.cumsum(shard_sizes)])[:-1]]

    s = shape.tuple
    plA = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * shape.chunk_bytes, slot_bytes=poolA.numel())
    plB = tc.pool(tc.TC_NHD, wave_blocks, 1, plane_stride=wave_blocks * shape.chunk_bytes, slot_bytes=poolB.numel())
    tune = {}
    if args.tile_bytes:
        tune["tile_bytes"] = args.tile_bytes
    if args.ctas_per_sm:
        tune["ctas_per_sm"] = args.ctas_per_sm
    host_tune = dict(tune)
    if args.host_ctas:
        host_tune["max_ctas"] = args.host_ctas
    host_flags = 0 if args.host_path == "zerocopy" else tc.TC_PLAN_STAGED
    t_plan0 = time.perf_counter()
    plans = []
    for src, dst in waves:
        kw = dict(T=src.T, bt_off=src.bt_off)
        plans.append(dict(
            pack=tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, s, src_pool=plA, packed_layout=tc.TC_HND, packed_bytes=Q.numel(), bt_src=src.bt, tuning=tune or None, **kw)),
            unpack=tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, s, dst_pool=plB, packed_layout=tc.TC_HND, packed_bytes=Q.numel(), bt_dst=dst.bt, tuning=tune or None, **kw)),
            migrate=tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, s, src_pool=plA, dst_pool=plB, bt_src=src.bt, bt_dst=dst.bt, tuning=tune or None, **kw)),
            pack_h=tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, s, src_pool=plA, packed_layout=tc.TC_HND, packed_bytes=Q.numel(), bt_src=src.bt, tuning=host_tune or None, flags=host_flags, **kw)),
            unpack_h=tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, s, dst_pool=plB, packed_layout=tc.TC_HND, packed_bytes=Q.numel(), bt_dst=dst.bt, tuning=host_tune or None, flags=host_flags, **kw)),
            payload=int(src.T.sum()) * shape.token_bytes))
    nbytes = [ck.nbytes(i) for i in range(ck.N)]
    mk_w = lambda tn, **kw: tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, blob_bytes=ck.nbytes_total, tuning=tn or None, **kw))
    w_full, w_shard = mk_w(tune), mk_w(tune, split_dim=ck.split_dim, rank=args.shard_rank, world=W)
    w_full_h = mk_w(host_tune, flags=host_flags)
    w_shard_h = mk_w(host_tune, split_dim=ck.split_dim, rank=args.shard_rank, world=W, flags=host_flags)
    plan_ms = 1e3 * (time.perf_counter() - t_plan0)
    n_plans = 5 * len(waves) + 4

    rows = {k: Row(k, m) for k, m in (("a1_kv_pack", "rows"), ("a2_kv_unpack", "rows"), ("a3_kv_migrate", "run"),
                                      ("a4_weights_full", "run"), ("a5_weights_shard", "rows"))}
    stream = torch.cuda.Stream()
    sp = stream.cuda_stream

    def timed(row, fn, nbytes_moved, ev):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        fn()
        b.record(stream)
        ev.append((row, a, b))
        row.bytes += nbytes_moved
        row.launches += 1

    def step(ev):
        for r in rows.values():
            r.bytes = r.launches = 0
        for p in plans:
            timed(rows["a1_kv_pack"], lambda: tc.tc_kv_pack(p["pack"], [poolA], [Q], sp), 2 * p["payload"], ev)
            timed(rows["a2_kv_unpack"], lambda: tc.tc_kv_unpack(p["unpack"], [Q], [poolB], sp), 2 * p["payload"], ev)
            timed(rows["a3_kv_migrate"], lambda: tc.tc_kv_pack(p["migrate"], [poolA], [poolB], sp), 2 * p["payload"], ev)
        timed(rows["a4_weights_full"], lambda: tc.tc_weights_materialize(w_full, blob, full_ptrs, sp), 2 * sum(full_sizes), ev)
        timed(rows["a5_weights_shard"], lambda: tc.tc_weights_materialize(w_shard, blob, shard_ptrs, sp), 2 * sum(shard_sizes), ev)

    barrier = ranks.barrier

    with torch.cuda.stream(stream):
        for _ in range(args.warmup):
            step([])
        barrier()
        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
        ev_all = []
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for _ in range(args.steps):
            ev = []
            step(ev)
            ev_all.append(ev)
        t1.record(stream)
        barrier()
        clocks = sampler.stop() if rank == 0 else None
    total_ms = t0.elapsed_time(t1)
    for ev in ev_all:
        per = {}
        for row, a, b in ev:
            per[row.name] = per.get(row.name, 0.0) + a.elapsed_time(b)
        for k, v in per.items():
            rows[k].ms.append(v)
    step_bytes = sum(r.bytes for r in rows.values())
    launches_per_step = sum(r.launches for r in rows.values())
    e2e_launches = (sum(p["pack_h"].stats().launches_per_execute + p["unpack_h"].stats().launches_per_execute for p in plans)
                    + w_full_h.stats().launches_per_execute + w_shard_h.stats().launches_per_execute)
    total_ms = ranks.max_ms(total_ms)
    value = world * step_bytes * args.steps / (total_ms * 1e-3) / GB

    # context for the roofline: a plain library copy (cudaMemcpyAsync through torch) of the very
    # same random bits, back to back.  Random contents draw more HBM power than the benign
    # contents a copy ceiling is usually measured with, and the GPU then runs at its power cap.
    n_ref = min(Q.numel(), poolB.numel())
    with torch.cuda.stream(stream):
        evs = []
        for i in range(24):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            poolB[:n_ref].copy_(Q[:n_ref])
            b.record(stream)
            evs.append((a, b))
        torch.cuda.synchronize()
    ref_ms = statistics.mean(a.elapsed_time(b) for a, b in evs[12:])
    copy_same_data = 2 * n_ref / (ref_ms * 1e-3) / GB

    # ---------------- e2e: packed buffer and blob in pinned host memory --------------------
    e2e = None
    e2e_skipped = None
    if not args.no_e2e:
        # pinned host memory is per process: N ranks on one node share the node's RAM
        try:
            avail = int(next(l for l in open("/proc/meminfo") if l.startswith("MemAvailable")).split()[1]) * 1024
        except Exception:
            avail = 64 << 30
        budget = 0.6 * avail / world
        need_duplex, need_serial = 2 * max_packed + ck.nbytes_total, max_packed + ck.nbytes_total
        if args.e2e_schedule == "duplex" and need_duplex > budget:
            args.e2e_schedule = "serial"
        if need_serial > budget:
            e2e_skipped = (f"skipped: {need_serial / GB:.0f} GB of pinned host memory per rank needed, "
                           f"{budget / GB:.0f} GB available per rank with {world} ranks on this node")
    if not args.no_e2e and e2e_skipped is None:
        Qh = torch.empty(max_packed, dtype=torch.uint8).pin_memory()
        blob_h = torch.empty(ck.nbytes_total, dtype=torch.uint8).pin_memory()
        blob_h.copy_(blob)
        probe = torch.empty(4096, dtype=torch.uint8).pin_memory()
        torch.cuda.synchronize()

        def ceiling(fn, nbytes):  # cudaMemcpyAsync on the same pinned allocation, best of 3
            best = 1e9
            for _ in range(4):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                fn()
                b.record(stream)
                torch.cuda.synchronize()
                best = min(best, a.elapsed_time(b))
            return nbytes / (best * 1e-3) / GB

        with torch.cuda.stream(stream):
            n_c = min(Qh.numel(), 4 << 30)
            ceil_h2d = ceiling(lambda: Q[:n_c].copy_(Qh[:n_c], non_blocking=True), n_c)
            ceil_d2h = ceiling(lambda: Qh[:n_c].copy_(Q[:n_c], non_blocking=True), n_c)

        duplex = args.e2e_schedule == "duplex"
        Qh2 = torch.empty(max_packed, dtype=torch.uint8).pin_memory() if duplex else Qh
        Qhs = (Qh, Qh2)
        stream_u = torch.cuda.Stream() if duplex else stream
        su = stream_u.cuda_stream
        ev_packed = [torch.cuda.Event() for _ in range(2)]
        ev_unpacked = [torch.cuda.Event() for _ in range(2)]
        ev_fork, ev_join = torch.cuda.Event(), torch.cuda.Event()

        def bidir_ceiling():  # both directions at once with cudaMemcpyAsync, GB/s summed
            n_c = min(Qh.numel(), 4 << 30)
            best = 1e9
            for _ in range(3):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                ev_fork.record(stream)
                stream_u.wait_event(ev_fork)
                Qh[:n_c].copy_(Q[:n_c], non_blocking=True)
                with torch.cuda.stream(stream_u):
                    poolB[:n_c].copy_(Qh2[:n_c], non_blocking=True)
                    ev_join.record(stream_u)
                stream.wait_event(ev_join)
                b.record(stream)
                torch.cuda.synchronize()
                best = min(best, a.elapsed_time(b))
            return 2 * n_c / (best * 1e-3) / GB

        def e2e_step():
            """Offload every wave to pinned host memory and reload it into the second pool; load the
            weights from the pinned blob.  duplex: the link is full duplex, so wave k+1 is offloaded
            (stream) while wave k is reloaded (stream_u), through two host buffers."""
            h2d = d2h = 0
            ev_fork.record(stream)
            stream_u.wait_event(ev_fork)
            tc.tc_weights_materialize(w_full_h, blob_h, full_ptrs, su)
            tc.tc_weights_materialize(w_shard_h, blob_h, shard_ptrs, su)
            h2d += sum(full_sizes) + sum(shard_sizes)
            for k, p in enumerate(plans):
                i = k % 2 if duplex else 0
                if k >= (2 if duplex else 1):
                    stream.wait_event(ev_unpacked[i])                    # the host buffer is free again
                tc.tc_kv_pack(p["pack_h"], [poolA], [Qhs[i]], sp)        # offload (device -> host)
                ev_packed[i].record(stream)
                stream_u.wait_event(ev_packed[i])
                tc.tc_kv_unpack(p["unpack_h"], [Qhs[i]], [poolB], su)    # reload (host -> device)
                ev_unpacked[i].record(stream_u)
                d2h += p["payload"]
                h2d += p["payload"]
            with torch.cuda.stream(stream_u):
                probe.copy_(dst_full[-4096:], non_blocking=True)         # read a result back
                ev_join.record(stream_u)
            stream.wait_event(ev_join)
            d2h += 4096
            return h2d, d2h

        with torch.cuda.stream(stream):
            ceil_bidir = bidir_ceiling() if duplex else None
            for _ in range(args.e2e_warmup):
                e2e_step()
            barrier()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(args.e2e_steps):
                h2d, d2h = e2e_step()
            b.record(stream)
            barrier()
        e_ms = a.elapsed_time(b)
        e_ms = ranks.max_ms(e_ms)
        # same byte convention as `value`: every payload byte is read once and written once
        e2e = {"value": world * 2 * (h2d + d2h - 4096) * args.e2e_steps / (e_ms * 1e-3) / GB, "unit": "GB/s",
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": args.e2e_steps,
               "ms_per_step": e_ms / args.e2e_steps,
               "host_link_GBps": world * (h2d + d2h) * args.e2e_steps / (e_ms * 1e-3) / GB,
               "host_link_ceiling_GBps": {"h2d_cudaMemcpyAsync": ceil_h2d, "d2h_cudaMemcpyAsync": ceil_d2h,
                                          "both_directions_at_once_summed": ceil_bidir},
               "host_link_frac_of_ceiling": (h2d + d2h) * args.e2e_steps / (e_ms * 1e-3) / GB /
                                            (ceil_bidir if duplex else (h2d + d2h) / (h2d / ceil_h2d + d2h / ceil_d2h)),
               "kv_host_path": args.host_path, "schedule": args.e2e_schedule,
               "note": "packed KV buffer and weight blob in pinned host memory. staged: copy engines + device staging rings + "
                       "D2D kernel (the TP shard's strided slices stay zero copy); zerocopy: kernel loads/stores on host memory"}
        del Qh, Qh2, Qhs, blob_h

    extras = None
    if not args.no_extras and world == 1:
        for p in plans:
            for k in ("pack", "unpack", "migrate", "pack_h", "unpack_h"):
                p[k].destroy()
        for w in (w_full, w_shard, w_full_h, w_shard_h):
            w.destroy()
        del poolA, poolB, Q, blob, dst_full, dst_shard, plans
        torch.cuda.empty_cache()
        extras = run_extras(args, tc, torch, stream)

    if rank != 0:
        ranks.close()
        return

    peak, peak_src = measured_peaks()
    per_row = {}
    for k, r in rows.items():
        ms = statistics.mean(r.ms)
        per_row[k] = {"GBps": r.bytes / (ms * 1e-3) / GB, "ms_per_step": ms, "launches_per_step": r.launches,
                      "bytes_per_step": r.bytes, "frac_of_peak": r.bytes / (ms * 1e-3) / GB / peak}
    # dominant kernel: the executor build that takes the largest share of the step
    by_mode = {}
    for r in rows.values():
        m = by_mode.setdefault(r.mode, {"bytes": 0, "ms": 0.0, "launches": 0})
        m["bytes"] += r.bytes
        m["ms"] += statistics.mean(r.ms)
        m["launches"] += r.launches
    dom = max(by_mode, key=lambda m: by_mode[m]["ms"])
    d = by_mode[dom]
    achieved = d["bytes"] / (d["ms"] * 1e-3) / GB
    roofline = {"bound": "hbm", "kernel": f"tc_copy_kernel<{'kModeRows' if dom == 'rows' else 'kModeRun'}>",
                "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "peak_source": peak_src, "traffic": traffic_per_launch(d["bytes"] / d["launches"]),
                "traffic_source": "ncu dram bytes of a small case, reads scaled by units, writes = payload minus the L2-resident tail",
                "algorithmic_bytes_per_launch": d["bytes"] / d["launches"], "avg_launch_ms": d["ms"] / d["launches"],
                "frac_of_nominal_8TBps": achieved / 8000.0,
                "library_copy_of_the_same_random_bits_GBps": copy_same_data,
                "note": "peak is the driver-measured copy ceiling; cudaMemcpyAsync of this workload's own random bits, "
                        "sustained, is given beside it (random contents put the GPU at its power cap)"}

    line = {
        "metric": "kv_pack_unpack_and_weight_materialise_GBps", "value": value, "unit": "GB/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": WORKLOAD_NAME, "kv_pool_blocks": NB, "wave_blocks": wave_blocks, "waves": len(waves),
                   "requests": int(sum(len(w[0].T) for w in waves)), "tokens": int(sum(int(w[0].T.sum()) for w in waves)),
                   "weights_bytes": ck.nbytes_total, "shard": f"{args.shard_rank}/8",
                   "bytes_per_step": step_bytes, "l2": "every launch moves far more than the 126 MB L2; no flush needed",
                   "parallelism": "replicas only" if world > 1 else "1 GPU", "plans": n_plans, "plan_create_ms_total": plan_ms},
        "clocks": clocks, "e2e": e2e if e2e is not None else ({"value": None, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0, "note": e2e_skipped or "skipped (--no-e2e)"}),
        "gpu_launches": launches_per_step * args.steps,
        "e2e_gpu_launches_per_step": e2e_launches,
        "roofline": roofline, "rows": per_row, "other_workloads": extras,
        "cpu_baseline": {"value": cpu_v, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": cpu_desc},
    }
    print(json.dumps(line))
    ranks.close()


def b2b_ms(torch, stream, fn, reps=5, warm=2):
    """Device milliseconds per call of fn: `reps` calls enqueued back to back inside one event pair,
    behind `warm` untimed ones that are still running when the first event is enqueued.  The host
    side of a call (marshalling the pointer table, checks, the launch itself) then overlaps the GPU
    work of the call before it; with a synchronise before every timed launch a short kernel would be
    charged for the time the idle GPU waits for the host."""
    with torch.cuda.stream(stream):
        for _ in range(warm):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(reps):
            fn()
        b.record(stream)
        torch.cuda.synchronize()
    return a.elapsed_time(b) / reps


def cold_path(args, tc, torch, stream):
    """Weight loading from a FILE (storage -> pinned ring -> device, scatter and slicing fused
    into the device leg): wall-clock GB/s of blob bytes, next to the plain rate at which the
    same file can be read into pinned memory and to the unpipelined sequence (read everything,
    then materialise from pinned memory)."""
    import shutil
    import tempfile
    sp = stream.cuda_stream
    ck = wl.llama_checkpoint(layers=1, vocab=16032) if args.small else wl.llama_checkpoint(layers=args.cold_layers, vocab=32064)
    root = "/dev/shm" if os.path.isdir("/dev/shm") and shutil.disk_usage("/dev/shm").free > 2 * ck.nbytes_total else tempfile.gettempdir()
    if shutil.disk_usage(root).free < 2 * ck.nbytes_total:
        return {"skipped": f"no room for a {ck.nbytes_total} byte file under {root}"}
    blob = torch.empty(ck.nbytes_total, dtype=torch.uint8, device="cuda")
    wl.fill_torch(blob, wl.SEED_BASE + 3, "normal")
    host = torch.empty(ck.nbytes_total, dtype=torch.uint8).pin_memory()
    host.copy_(blob)
    header = 4096 + 8 * ck.N
    fdw, path = tempfile.mkstemp(prefix="tc_cold_", suffix=".bin", dir=root)
    out = {"file": f"{ck.nbytes_total} B blob behind a {header} B header, in {root} (page cache)"}
    try:
        with os.fdopen(fdw, "wb") as f:
            f.write(bytes(header))
            host.numpy().tofile(f)
        nbytes = [ck.nbytes(i) for i in range(ck.N)]
        dstw = torch.empty(ck.nbytes_total, dtype=torch.uint8, device="cuda")
        ptrs = [dstw.data_ptr() + int(o) for o in np.concatenate([[0], np.cumsum(nbytes)])[:-1]]
        sums = torch.zeros(ck.N, dtype=torch.int64, device="cuda")
        fd = os.open(path, os.O_RDONLY)
        n_readers = max(1, min(8, (os.cpu_count() or 2) - 1))

        def read_all():  # the storage leg alone: the whole blob into pinned memory, same thread count
            view = memoryview(host.numpy())
            part = -(-ck.nbytes_total // n_readers)

            def rd(i):
                lo, hi = i * part, min(ck.nbytes_total, (i + 1) * part)
                while lo < hi:
                    k = os.preadv(fd, [view[lo:min(hi, lo + (64 << 20))]], header + lo)
                    lo += k
            th = [threading.Thread(target=rd, args=(i,)) for i in range(n_readers)]
            [t.start() for t in th]
            [t.join() for t in th]

        def wall(fn, reps=3):
            best = []
            for i in range(reps + 1):
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                fn()
                torch.cuda.synchronize()
                if i:
                    best.append(time.perf_counter() - t0)
            return statistics.mean(best)

        plan = tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, blob_bytes=ck.nbytes_total,
                                                 flags=tc.TC_PLAN_STREAM | tc.TC_PLAN_CHECKSUM))
        staged = tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, blob_bytes=ck.nbytes_total, flags=tc.TC_PLAN_STAGED))
        t_read = wall(read_all)
        with torch.cuda.stream(stream):
            t_stream = wall(lambda: tc.tc_weights_materialize_file(plan, fd, header, ptrs, stream=sp))
            same = bool(torch.equal(dstw, blob))
            t_check = wall(lambda: tc.tc_weights_materialize_file(plan, fd, header, ptrs, checksums=sums, stream=sp))
            t_seq = wall(lambda: (read_all(), tc.tc_weights_materialize(staged, host, ptrs, sp)))
        W = 8
        sizes = [n // (W if ck.split_dim[i] >= 0 else 1) for i, n in enumerate(nbytes)]
        sptrs = [dstw.data_ptr() + int(o) for o in np.concatenate([[0], np.cumsum(sizes)])[:-1]]
        shard = tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, split_dim=ck.split_dim, rank=args.shard_rank, world=W,
                                                  blob_bytes=ck.nbytes_total, flags=tc.TC_PLAN_STREAM))
        read_bytes = sum(sg.bytes for sg in shard.segments(0))
        with torch.cuda.stream(stream):
            t_shard = wall(lambda: tc.tc_weights_materialize_file(shard, fd, header, sptrs, stream=sp))
        os.close(fd)
        out.update({
            "readers": n_readers, "chunks": plan.stats().launches_per_execute, "bytes_match_after_streaming": same,
            "GBps_file_read_into_pinned_only": ck.nbytes_total / t_read / GB,
            "GBps_streamed_full": ck.nbytes_total / t_stream / GB,
            "GBps_streamed_full_with_checksum": ck.nbytes_total / t_check / GB,
            "GBps_read_everything_then_materialize": ck.nbytes_total / t_seq / GB,
            "shard_1_of_8": {"payload_bytes": sum(sizes), "file_bytes_read": read_bytes, "chunks": shard.stats().launches_per_execute,
                             "ms": 1e3 * t_shard, "GBps_of_file_bytes": read_bytes / t_shard / GB}})
        for p_ in (plan, staged, shard):
            p_.destroy()
    finally:
        os.unlink(path)
    del blob, host
    torch.cuda.empty_cache()
    return out


def moe_stacking(args, tc, torch, stream):
    """transform_into with expert stacking on a mixture-of-experts checkpoint of the shape the
    paper's loader experiments use (Qwen3-30B-A3B: hidden 2048, 128 experts of 768, some of its
    48 layers): per layer the gate and up matrices of all experts land in one fused
    [experts, 2*mlp, hidden] buffer and the down matrices in one [experts, hidden, mlp] buffer;
    every other tensor gets its own destination."""
    import re
    sp = stream.cuda_stream
    layers, experts, mlp, hidden = (1 if args.small else args.moe_layers), 128, 768, 2048
    ck = wl.moe_checkpoint(hidden=hidden, layers=layers, experts=experts, moe_mlp=mlp, q_heads=32, kv_heads=4, head_dim=128, vocab=151936)
    E = 2
    nbytes = [ck.nbytes(i) for i in range(ck.N)]
    gu_exp, dn_exp = 2 * mlp * hidden * E, hidden * mlp * E
    slot, doff, dst_bytes = [], [], []
    fused = {}
    pat = re.compile(r"layers\.(\d+)\.experts\.(\d+)\.(gate|up|down)_proj")
    for i, name in enumerate(ck.names):
        m = pat.fullmatch(name)
        if not m:
            slot.append(len(dst_bytes))
            doff.append(0)
            dst_bytes.append(nbytes[i])
            continue
        l, e, kind = int(m.group(1)), int(m.group(2)), m.group(3)
        key = (l, "down" if kind == "down" else "gate_up")
        if key not in fused:
            fused[key] = len(dst_bytes)
            dst_bytes.append(experts * (dn_exp if kind == "down" else gu_exp))
        slot.append(fused[key])
        doff.append(e * dn_exp if kind == "down" else e * gu_exp + (mlp * hidden * E if kind == "up" else 0))
    blob = torch.empty(ck.nbytes_total, dtype=torch.uint8, device="cuda")
    wl.fill_torch(blob, wl.SEED_BASE + 6, "normal")
    arena = torch.empty(sum(dst_bytes), dtype=torch.uint8, device="cuda")
    starts = np.concatenate([[0], np.cumsum(dst_bytes)])[:-1]
    ptrs = [arena.data_ptr() + int(o) for o in starts]
    spec = tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, blob_bytes=ck.nbytes_total,
                           dst_slot=slot, dst_off=doff, n_dst=len(dst_bytes), dst_bytes=dst_bytes)
    torch.cuda.synchronize()  # the fill above is still running; plan upload would wait for it
    t0 = time.perf_counter()
    plan = tc.tc_plan_create(spec)
    create_ms = 1e3 * (time.perf_counter() - t0)
    ms = b2b_ms(torch, stream, lambda: tc.tc_weights_materialize(plan, blob, ptrs, sp))
    # spot check: expert 5 of the last layer, up_proj, sits behind its gate_proj in the fused buffer
    i = ck.names.index(f"layers.{layers - 1}.experts.5.up_proj")
    lo = int(starts[slot[i]]) + doff[i]
    ok = bool(torch.equal(arena[lo:lo + nbytes[i]], blob[int(ck.byte_off[i]):int(ck.byte_off[i]) + nbytes[i]]))
    st = plan.stats()
    plan.destroy()
    del blob, arena
    torch.cuda.empty_cache()
    return {"layers": layers, "tensors": ck.N, "destination_buffers": len(dst_bytes), "bytes": ck.nbytes_total, "tiles": int(st.n_tiles[0]),
            "plan_create_ms": create_ms, "ms": ms, "GBps": 2 * ck.nbytes_total / (ms * 1e-3) / GB, "spot_check": ok}


def kv_shapes(args, tc, torch, stream):
    """Rows a1-a3 on other KV geometries than the headline one: few KV heads (what a tensor-parallel
    rank or a GQA / MQA model holds: planes of 4-16 KiB per block), larger blocks, small head_dim."""
    sp = stream.cuda_stream
    u8 = dict(dtype=torch.uint8, device="cuda")
    out = {}
    K = wl.KVShape
    cases = [("8 KV heads (headline shape)", K(32, 16, 8, 128)), ("4 KV heads", K(28, 16, 4, 128)), ("2 KV heads", K(28, 16, 2, 128)),
             ("1 KV head", K(32, 16, 1, 128)), ("32 heads of 64", K(32, 16, 32, 64)), ("block 128", K(32, 128, 8, 128))]
    for label, shape in ([cases[1], cases[3]] if args.small else cases):
        s = shape.tuple
        NB = int(((1 if args.small else 8) << 30) // shape.block_bytes)
        WB = NB // 2
        _, _, _, waves = wl.config2(NB=NB, R=256, wave_blocks=WB, NB_dst=WB, shape=shape)
        src, dst = waves[0]
        poolA = torch.empty(NB * shape.block_bytes, **u8)
        wl.fill_torch(poolA, wl.SEED_BASE + 7)
        poolB = torch.empty(WB * shape.block_bytes, **u8)
        payload = int(src.T.sum()) * shape.token_bytes
        Q = torch.empty(payload, **u8)
        plA = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * shape.chunk_bytes, slot_bytes=poolA.numel())
        plB = tc.pool(tc.TC_NHD, WB, 1, plane_stride=WB * shape.chunk_bytes, slot_bytes=poolB.numel())
        kw = dict(T=src.T, bt_off=src.bt_off)
        pk = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, s, src_pool=plA, packed_layout=tc.TC_HND, bt_src=src.bt, **kw))
        up = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, s, dst_pool=plB, packed_layout=tc.TC_HND, bt_dst=dst.bt, **kw))
        mig = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, s, src_pool=plA, dst_pool=plB, bt_src=src.bt, bt_dst=dst.bt, **kw))
        res = {"plane_KiB": shape.chunk_bytes // 1024, "planes_per_tile": int(mig.descriptors(0)[0].planes_per_tile), "payload_bytes": payload}
        for name, fn in (("pack", lambda: tc.tc_kv_pack(pk, [poolA], [Q], sp)), ("unpack", lambda: tc.tc_kv_unpack(up, [Q], [poolB], sp)),
                         ("migrate", lambda: tc.tc_kv_pack(mig, [poolA], [poolB], sp))):
            res["GBps_" + name] = 2 * payload / (b2b_ms(torch, stream, fn, reps=1 if args.small else 8, warm=1 if args.small else 3) * 1e-3) / GB
        out[label + f" L{shape.L} B{shape.B} H{shape.H} D{shape.D}"] = res
        for p_ in (pk, up, mig):
            p_.destroy()
        del poolA, poolB, Q
        torch.cuda.empty_cache()
    return out


def misaligned(args, tc, torch, stream):
    """Rows a1-a5 when source and destination are not 16-byte aligned: the same plans as the
    headline rows (aligned geometry), run on base pointers shifted by 8 / 4 / 2 / 1 bytes - a
    packed buffer or a blob that is a view at an odd offset of a larger allocation, a checkpoint
    with a short lead pad.  'src' shifts only the source table (the two sides then differ in
    alignment and every 16-byte store is assembled from two aligned loads), 'both' shifts both
    sides by the same amount (heads and tails only)."""
    sp = stream.cuda_stream
    u8 = dict(dtype=torch.uint8, device="cuda")
    shape = wl.LLAMA3_8B_KV
    s = shape.tuple
    NB = int(((1 if args.small else 8) << 30) // shape.block_bytes)
    WB = NB // 2
    _, _, _, waves = wl.config2(NB=NB, R=256, wave_blocks=WB, NB_dst=WB, shape=shape)
    src, dst = waves[0]
    payload = int(src.T.sum()) * shape.token_bytes
    rawA = torch.empty(NB * shape.block_bytes + 16, **u8)
    wl.fill_torch(rawA, wl.SEED_BASE + 7)
    rawB = torch.empty(WB * shape.block_bytes + 16, **u8)
    rawQ = torch.empty(payload + 16, **u8)
    plA = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * shape.chunk_bytes, slot_bytes=NB * shape.block_bytes)
    plB = tc.pool(tc.TC_NHD, WB, 1, plane_stride=WB * shape.chunk_bytes, slot_bytes=WB * shape.block_bytes)
    kw = dict(T=src.T, bt_off=src.bt_off)
    pk = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, s, src_pool=plA, packed_layout=tc.TC_HND, bt_src=src.bt, **kw))
    up = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, s, dst_pool=plB, packed_layout=tc.TC_HND, bt_dst=dst.bt, **kw))
    mig = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, s, src_pool=plA, dst_pool=plB, bt_src=src.bt, bt_dst=dst.bt, **kw))
    ck = wl.llama_checkpoint(layers=1, vocab=16032) if args.small else wl.llama_checkpoint(layers=8, vocab=32064)
    nbytes = [ck.nbytes(i) for i in range(ck.N)]
    W = 8
    sizes = [n // (W if ck.split_dim[i] >= 0 else 1) for i, n in enumerate(nbytes)]
    blob = torch.empty(ck.nbytes_total + 16, **u8)
    wl.fill_torch(blob, wl.SEED_BASE + 3, "normal")
    dstw = torch.empty(ck.nbytes_total + 16, **u8)
    starts_f = np.concatenate([[0], np.cumsum(nbytes)])[:-1]
    starts_s = np.concatenate([[0], np.cumsum(sizes)])[:-1]
    wf = tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, blob_bytes=ck.nbytes_total))
    ws = tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, split_dim=ck.split_dim, rank=args.shard_rank, world=W, blob_bytes=ck.nbytes_total))
    reps, warm = (1, 1) if args.small else (6, 2)
    out = {"kv_payload_bytes": payload, "weights_bytes": ck.nbytes_total, "shard_bytes": sum(sizes)}
    peak, _ = measured_peaks()
    auto = (pk, up, mig, wf, ws)
    # the same plans forced onto the shared-memory path (bulk asynchronous copies in, 16-byte stores
    # out), on aligned pointers: the A/B behind the choice of the register path for aligned geometry
    smem = dict(copy_path=1)
    staged = (tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, s, src_pool=plA, packed_layout=tc.TC_HND, bt_src=src.bt, tuning=smem, **kw)),
              tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, s, dst_pool=plB, packed_layout=tc.TC_HND, bt_dst=dst.bt, tuning=smem, **kw)),
              tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, s, src_pool=plA, dst_pool=plB, bt_src=src.bt, bt_dst=dst.bt, tuning=smem, **kw)),
              tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, blob_bytes=ck.nbytes_total, tuning=smem)),
              tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, split_dim=ck.split_dim, rank=args.shard_rank, world=W,
                                                blob_bytes=ck.nbytes_total, tuning=smem)))
    cases = [("aligned", 0, 0, auto), ("aligned, through shared memory (tuning.copy_path = 1)", 0, 0, staged)]
    cases += [(f"src+{a}", a, 0, auto) for a in (8, 4, 2, 1)] + [("both+1", 1, 1, auto), ("src+3 dst+9", 3, 9, auto)]
    for label, a_src, a_dst, (pk, up, mig, wf, ws) in cases:
        A, B = rawA.data_ptr(), rawB.data_ptr()
        Q, bl, dw = rawQ.data_ptr(), blob.data_ptr(), dstw.data_ptr()
        res = {}
        for name, fn, moved in (
                ("a1_pack", lambda: tc.tc_kv_pack(pk, [A + a_src], [Q + a_dst], sp), payload),
                ("a2_unpack", lambda: tc.tc_kv_unpack(up, [Q + a_src], [B + a_dst], sp), payload),
                ("a3_migrate", lambda: tc.tc_kv_pack(mig, [A + a_src], [B + a_dst], sp), payload),
                ("a4_weights_full", lambda: tc.tc_weights_materialize(wf, bl + a_src, [dw + a_dst + int(o) for o in starts_f], sp), ck.nbytes_total),
                ("a5_weights_shard", lambda: tc.tc_weights_materialize(ws, bl + a_src, [dw + a_dst + int(o) for o in starts_s], sp), sum(sizes))):
            res[name] = 2 * moved / (b2b_ms(torch, stream, fn, reps=reps, warm=warm) * 1e-3) / GB
        res["min_frac_of_measured_peak"] = min(res.values()) / peak
        out[label] = res
    for p_ in auto + staged:
        p_.destroy()
    del rawA, rawB, rawQ, blob, dstw
    torch.cuda.empty_cache()
    return out


def run_extras(args, tc, torch, stream):
    """Secondary workloads, reported beside the headline: configs[3] (70B-shaped pool-to-pool
    migration, one wave) and configs[4] (prefix-reload burst: one mixed plan per scheduler step,
    created and executed inside the timed region, both directions concurrently over the host
    link with zero-copy kernels)."""
    out = {}
    sp = stream.cuda_stream
    u8 = dict(dtype=torch.uint8, device="cuda")
    if args.only_kv_shapes:  # profiler runs: just the KV geometries, a few GB on the device
        out["rows a1-a3 on other KV geometries (8 GiB pools, first wave)"] = kv_shapes(args, tc, torch, stream)
        return out
    if args.only_misaligned:
        out["rows a1-a5: copy paths and misaligned base pointers (8 GiB pool, 4 GB checkpoint)"] = misaligned(args, tc, torch, stream)
        return out
    # ---- configs[0]: 1.4 MB, launch-latency bound: microseconds and plans per second
    shape, NB1, src1, dst1 = wl.config1()
    pool1 = torch.empty(2 * NB1 * shape.chunk_bytes, **u8)
    wl.fill_torch(pool1, wl.SEED_BASE + 1)
    fresh1 = torch.empty_like(pool1)
    packed1 = torch.empty(int(src1.T.sum()) * shape.token_bytes, **u8)
    pl1 = tc.pool(tc.TC_NHD, NB1, 1, plane_stride=NB1 * shape.chunk_bytes, slot_bytes=pool1.numel())
    mk_p = lambda: tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape.tuple, src_pool=pl1, packed_layout=tc.TC_HND, T=src1.T, bt_off=src1.bt_off, bt_src=src1.bt))
    mk_u = lambda: tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, shape.tuple, dst_pool=pl1, packed_layout=tc.TC_HND, T=dst1.T, bt_off=dst1.bt_off, bt_dst=dst1.bt))
    p1, u1 = mk_p(), mk_u()
    with torch.cuda.stream(stream):
        for _ in range(10):
            tc.tc_kv_pack(p1, [pool1], [packed1], sp)
            tc.tc_kv_unpack(u1, [packed1], [fresh1], sp)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(200):
            tc.tc_kv_pack(p1, [pool1], [packed1], sp)
            tc.tc_kv_unpack(u1, [packed1], [fresh1], sp)
        b.record(stream)
        torch.cuda.synchronize()
        us_pair = a.elapsed_time(b) * 1e3 / 200
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for _ in range(20):
                tc.tc_kv_pack(p1, [pool1], [packed1], sp)
                tc.tc_kv_unpack(u1, [packed1], [fresh1], sp)
        graph.replay()
        torch.cuda.synchronize()
        a.record(stream)
        for _ in range(10):
            graph.replay()
        b.record(stream)
        torch.cuda.synchronize()
        us_pair_graph = a.elapsed_time(b) * 1e3 / 200
    t0 = time.perf_counter()
    for _ in range(200):
        pp, uu = mk_p(), mk_u()
        tc.tc_kv_pack(pp, [pool1], [packed1], sp)
        tc.tc_kv_unpack(uu, [packed1], [fresh1], sp)
        torch.cuda.synchronize()
        pp.destroy()
        uu.destroy()
    wall = time.perf_counter() - t0
    out["configs[0] correctness case (1.4 MB, latency bound)"] = {
        "us_per_pack_plus_unpack_stream": us_pair, "us_per_pack_plus_unpack_cuda_graph": us_pair_graph,
        "plans_per_s_create_execute_sync_destroy": 400 / wall, "payload_bytes": packed1.numel()}
    del pool1, fresh1, packed1
    # ---- configs[2] again, with the integrity checksum folded into the copy
    ck = wl.config3() if not args.small else wl.llama_checkpoint(layers=1, vocab=16032)
    blob = torch.empty(ck.nbytes_total, **u8)
    wl.fill_torch(blob, wl.SEED_BASE + 3, "normal")
    dstw = torch.empty(ck.nbytes_total, **u8)
    nbytes = [ck.nbytes(i) for i in range(ck.N)]
    ptrs = [dstw.data_ptr() + int(o) for o in np.concatenate([[0], np.cumsum(nbytes)])[:-1]]
    sums = torch.zeros(ck.N, dtype=torch.int64, device="cuda")
    planc = tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, blob_bytes=ck.nbytes_total, flags=tc.TC_PLAN_CHECKSUM))
    planp = tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, blob_bytes=ck.nbytes_total))
    res = {}
    for name, fn in (("plain", lambda: tc.tc_weights_materialize(planp, blob, ptrs, sp)),
                     ("with_checksum", lambda: tc.tc_weights_materialize_checksum(planc, blob, ptrs, sums, sp))):
        res[name] = 2 * ck.nbytes_total / (b2b_ms(torch, stream, fn) * 1e-3) / GB
    out["configs[2] weights full, integrity checksum fused into the copy"] = {"GBps_plain": res["plain"], "GBps_with_checksum": res["with_checksum"]}
    planc.destroy()
    planp.destroy()
    # ---- configs[2]: every rank's shard of W = 8, each timed alone
    W = 8
    sizes = [n // (W if ck.split_dim[i] >= 0 else 1) for i, n in enumerate(nbytes)]
    sptrs = [dstw.data_ptr() + int(o) for o in np.concatenate([[0], np.cumsum(sizes)])[:-1]]
    per_rank = []
    for rank in range(W):
        sh = tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, split_dim=ck.split_dim, rank=rank, world=W, blob_bytes=ck.nbytes_total))
        ms = b2b_ms(torch, stream, lambda: tc.tc_weights_materialize(sh, blob, sptrs, sp), reps=10)
        per_rank.append(2 * sum(sizes) / (ms * 1e-3) / GB)
        sh.destroy()
    out["configs[2] weights TP shard, every rank of 8 (10 launches back to back per rank; 4 GB of traffic per launch)"] = {
        "payload_bytes": sum(sizes), "GBps_per_rank": per_rank}
    del blob, dstw
    torch.cuda.empty_cache()
    out["weights cold path: blob streamed from a file"] = cold_path(args, tc, torch, stream)
    out["transform_into: MoE expert stacking (Qwen3-30B-A3B-shaped layers)"] = moe_stacking(args, tc, torch, stream)
    out["rows a1-a3 on other KV geometries (8 GiB pools, first wave)"] = kv_shapes(args, tc, torch, stream)
    out["rows a1-a5: copy paths and misaligned base pointers (8 GiB pool, 4 GB checkpoint)"] = misaligned(args, tc, torch, stream)
    # ---- configs[3]
    shape = wl.LLAMA3_70B_KV
    free, _ = torch.cuda.mem_get_info()
    NB = 4096
    while 2 * NB * shape.block_bytes > 0.8 * free:
        NB //= 2
    _, _, _, waves = wl.config4(NB=NB, max_waves=1)
    src, dst = waves[0]
    A = torch.empty(NB * shape.block_bytes, **u8)
    A.fill_(7)
    B = torch.empty(NB * shape.block_bytes, **u8)
    B.fill_(9)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * shape.chunk_bytes, slot_bytes=A.numel())
    torch.cuda.synchronize()  # the fills above are still running; plan upload would wait for them
    t0 = time.perf_counter()
    mig = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape.tuple, src_pool=pl, dst_pool=pl, T=src.T, bt_off=src.bt_off, bt_src=src.bt, bt_dst=dst.bt))
    create_ms = 1e3 * (time.perf_counter() - t0)
    payload = int(src.T.sum()) * shape.token_bytes
    ms_mig = b2b_ms(torch, stream, lambda: tc.tc_kv_pack(mig, [A], [B], sp), reps=3)
    out["configs[3] 70B KV migrate (one wave)"] = {
        "pool_blocks": NB, "requests": len(src.T), "blocks": src.n_blocks, "payload_bytes": payload,
        "GBps": 2 * payload / (ms_mig * 1e-3) / GB, "ms": ms_mig, "plan_create_ms": create_ms}
    mig.destroy()
    # the same wave into an HND pool (layout transform fused into the migration) ...
    pl_hnd = tc.pool(tc.TC_HND, NB, 1, plane_stride=NB * shape.chunk_bytes, slot_bytes=A.numel())
    mig_t = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape.tuple, src_pool=pl, dst_pool=pl_hnd, T=src.T, bt_off=src.bt_off, bt_src=src.bt, bt_dst=dst.bt))

    def timed(fn):
        return b2b_ms(torch, stream, fn, reps=3)
    ms_t = timed(lambda: tc.tc_kv_pack(mig_t, [A], [B], sp))
    mig_t.destroy()
    out["configs[3] 70B KV migrate (one wave)"]["GBps_into_an_HND_pool"] = 2 * payload / (ms_t * 1e-3) / GB
    # ... and, for comparison, unfused: pack into a device buffer, then unpack (twice the traffic).
    # The buffer takes what memory is left, so only the first requests that fit take part.
    free, _ = torch.cuda.mem_get_info()
    budget = int(0.8 * free)
    k = int(np.searchsorted(np.cumsum(src.T) * shape.token_bytes, budget, side="right"))
    if k > 0:
        Tk, offk = src.T[:k], src.bt_off[:k + 1]
        nblk = int(offk[-1])
        part = int(Tk.sum()) * shape.token_bytes
        Q = torch.empty(part, **u8)
        pk = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape.tuple, src_pool=pl, packed_layout=tc.TC_NHD, T=Tk, bt_off=offk, bt_src=src.bt[:nblk]))
        up = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, shape.tuple, dst_pool=pl, packed_layout=tc.TC_NHD, T=Tk, bt_off=offk, bt_dst=dst.bt[:nblk]))
        fused = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape.tuple, src_pool=pl, dst_pool=pl, T=Tk, bt_off=offk, bt_src=src.bt[:nblk], bt_dst=dst.bt[:nblk]))
        ms_two = timed(lambda: (tc.tc_kv_pack(pk, [A], [Q], sp), tc.tc_kv_unpack(up, [Q], [B], sp)))
        ms_one = timed(lambda: tc.tc_kv_pack(fused, [A], [B], sp))
        out["configs[3] 70B KV migrate (one wave)"]["fused_vs_pack_then_unpack"] = {
            "requests": k, "payload_bytes": part, "ms_fused_migrate": ms_one, "ms_pack_then_unpack_through_a_device_buffer": ms_two}
        for p_ in (pk, up, fused):
            p_.destroy()
        del Q
    del A, B
    torch.cuda.empty_cache()
    # ---- configs[4]
    shape = wl.LLAMA3_8B_KV
    NBd, NBh, n_steps = 20000, args.host_pool_blocks, args.burst_steps
    dev = torch.empty(NBd * shape.block_bytes, **u8)
    dev.fill_(3)
    host = torch.empty(NBh * shape.block_bytes, dtype=torch.uint8).pin_memory()
    dev_pool = tc.pool(tc.TC_NHD, NBd, 1, plane_stride=NBd * shape.chunk_bytes, slot_bytes=dev.numel())
    host_pool = tc.pool(tc.TC_HND, NBh, 1, plane_stride=shape.chunk_bytes, block_stride=shape.block_bytes, slot_bytes=host.numel())
    s2 = torch.cuda.Stream()
    create, h2d, d2h = [], 0, 0
    steps = list(wl.config5(NB_dev=NBd, NB_host=NBh, steps=n_steps + 1))
    torch.cuda.synchronize()
    t_all = None
    for i, st in enumerate(steps):
        if i == 1:  # step 0 is the warm-up
            torch.cuda.synchronize()
            t_all = time.perf_counter()
        t0 = time.perf_counter()
        plan = tc.tc_plan_create(tc.kv_spec(
            tc.TC_KV_MIXED, shape.tuple, src_pool=dev_pool, dst_pool=host_pool,
            T=st.offload_T, bt_off=st.offload_off, bt_src=st.offload_dev, bt_dst=st.offload_host,
            reload=dict(T=st.reload_T, bt_off=st.reload_off, bt_src=st.reload_host, bt_dst=st.reload_dev),
            flags=0 if args.host_path == "zerocopy" else tc.TC_PLAN_STAGED))
        if i >= 1:
            create.append(1e3 * (time.perf_counter() - t0))
            h2d += int(st.reload_T.sum()) * shape.token_bytes
            d2h += int(st.offload_T.sum()) * shape.token_bytes
        # the short offload is enqueued first: the reload's ~6 000 page copies fill the driver's
        # stream queue, so whatever is enqueued after it only starts when it is nearly done
        tc.tc_kv_pack(plan, [dev], [host], s2.cuda_stream)
        tc.tc_kv_unpack(plan, [host], [dev], sp)
        torch.cuda.synchronize()   # a scheduler step ends when both directions have landed
        plan.destroy()
    wall = time.perf_counter() - t_all
    out["configs[4] prefix-reload burst (mixed plan per step)"] = {
        "steps": n_steps, "sessions": 512, "host_pool_blocks": NBh, "device_pool_blocks": NBd,
        "plans_per_s": n_steps / wall, "ms_per_step_wall": 1e3 * wall / n_steps, "plan_create_ms": statistics.mean(create),
        "h2d_GBps": h2d / wall / GB, "d2h_GBps": d2h / wall / GB, "link_GBps_both_directions": (h2d + d2h) / wall / GB,
        "h2d_bytes_per_step": h2d // n_steps, "d2h_bytes_per_step": d2h // n_steps,
        "host_path": args.host_path,
        "note": "wall clock over create + execute + synchronise of every step; reload and offload run concurrently on two streams"}
    del dev, host
    torch.cuda.empty_cache()
    return out


def traffic_per_launch(algorithmic_bytes: float) -> float:
    """DRAM bytes of one full-size launch, scaled from an `ncu --set full` capture of a small
    case (226 MB wave, 700 MB checkpoint): reads = 1.0002 x payload (descriptors included);
    writes = payload less the ~50 MB of dirty lines still in L2 at kernel end."""
    payload = algorithmic_bytes / 2
    return 1.0002 * payload + max(payload - 50.7e6, 0.0)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--kv-blocks", type=int, default=20000)
    ap.add_argument("--wave-blocks", type=int, default=8192)
    ap.add_argument("--requests", type=int, default=256)
    ap.add_argument("--max-waves", type=int, default=0)
    ap.add_argument("--shard-rank", type=int, default=0)
    ap.add_argument("--small", action="store_true", help="small case for profiler captures")
    ap.add_argument("--dry-run", action="store_true", help="CPU-only check of the multi-rank plumbing (gloo)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing (profiler runs)")
    ap.add_argument("--e2e-steps", type=int, default=1)
    ap.add_argument("--e2e-warmup", type=int, default=1)
    ap.add_argument("--oracle-blocks", type=int, default=1536)
    ap.add_argument("--tile-bytes", type=int, default=0)
    ap.add_argument("--ctas-per-sm", type=int, default=0)
    ap.add_argument("--no-extras", action="store_true", help="skip the secondary workloads (configs[3], configs[4])")
    ap.add_argument("--only-kv-shapes", action="store_true", help="of the secondary workloads run only the KV geometries (profiler captures)")
    ap.add_argument("--only-misaligned", action="store_true", help="of the secondary workloads run only the misaligned-pointer rows")
    ap.add_argument("--host-pool-blocks", type=int, default=8192, help="configs[4]: pinned host pool size in 2 MiB blocks")
    ap.add_argument("--burst-steps", type=int, default=10, help="configs[4]: scheduler steps timed (the workload has 200)")
    ap.add_argument("--cold-layers", type=int, default=8, help="cold-path extra: layers of the checkpoint written to a file (8: 4.0 GB)")
    ap.add_argument("--moe-layers", type=int, default=8, help="expert-stacking extra: layers of the MoE checkpoint (8: 11 GB)")
    ap.add_argument("--host-ctas", type=int, default=0)
    ap.add_argument("--host-path", default="staged", choices=["staged", "zerocopy"])
    ap.add_argument("--e2e-schedule", default="duplex", choices=["duplex", "serial"],
                    help="duplex: offload wave k+1 while wave k reloads (two streams, two host buffers)")
    args = ap.parse_args()
    if args.dry_run:
        run_dry(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
