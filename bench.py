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


def mem_available() -> int:
    try:
        return int(next(l for l in open("/proc/meminfo") if l.startswith("MemAvailable")).split()[1]) * 1024
    except Exception:
        return 64 << 30


class PinnedArena:
    """One pinned host allocation for the whole run, carved into the buffers its parts need one
    after the other (pinning 100 GB takes the better part of a minute; doing it once is the point)."""

    def __init__(self, torch, nbytes: int):
        t0 = time.perf_counter()
        self.buf = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
        self.seconds = time.perf_counter() - t0
        self.used = 0

    def reset(self):
        self.used = 0

    def take(self, nbytes: int):
        lo = (self.used + 4095) // 4096 * 4096
        assert lo + nbytes <= self.buf.numel(), "pinned arena too small"
        self.used = lo + nbytes
        return self.buf[lo:lo + nbytes]


def burst_host_blocks(args, avail: int, world: int = 1) -> int:
    """configs[4]: blocks of the pinned host pool - min(262144, half of MemAvailable / 2 MiB)."""
    if args.host_pool_blocks > 0:
        return args.host_pool_blocks
    return min(262144, int(0.5 * avail / world) // wl.LLAMA3_8B_KV.block_bytes)


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
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs.  The sampler is
    started ahead of the region (nvidia-smi takes a moment to come up) and every sample is stamped
    on arrival; stop() keeps the samples that arrived between mark_begin() and mark_end()."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []
        self.t0 = self.t1 = None

    def start(self, wait_s: float = 3.0):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True, bufsize=1)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
            t = time.time()
            while not self.lines and time.time() - t < wait_s:   # until the first sample is in
                time.sleep(0.02)
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def mark_begin(self):
        self.t0 = time.time()

    def mark_end(self):
        self.t1 = time.time()

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        if self.t1 is not None:
            time.sleep(max(0.0, 0.15 - (time.time() - self.t1)))   # the sample in flight when the region ended
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        t0 = self.t0 if self.t0 is not None else 0.0
        t1 = (self.t1 if self.t1 is not None else time.time()) + 0.15
        inside = [ln for ts, ln in self.lines if t0 <= ts <= t1]
        sm, mx, reasons = [], [], set()
        for ln in inside:
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
                "reasons": sorted(reasons), "samples": len(sm), "samples_outside_the_timed_region": len(self.lines) - len(inside)}


# --------------------------------------------------------------------------------------
# CPU oracle leg (cpu_baseline / --impl reference)
# --------------------------------------------------------------------------------------
class OracleSample:
    """The oracle, as it stands, on a bounded sample of the same workload, all five rows of the step:
      a1 + a2  kv_pack NHD -> HND and kv_unpack through an independent block table,
      a3       kv_migrate pool to pool,
               (the first requests of the Llama-3-8B KV workload that fit `sample_blocks` blocks)
      a4 + a5  weights full and the 1-of-8 shard of one decoder layer of the checkpoint (9 tensors,
               436 MB, dim-0 slabs and dim-1 strided slices like the whole),
    split over `threads` host threads by request / tensor, plus a1 + a2 on the first requests
    (`single_blocks` blocks) with ONE thread.  Bytes are counted like the GPU metric: read + written."""

    def __init__(self, sample_blocks: int, threads: int, single_blocks: int = 96):
        import oracle
        self.oracle = oracle
        self.shape = shape = wl.LLAMA3_8B_KV
        NBs = sample_blocks
        T_all = wl.config2()[2]

        def first_requests(budget):
            keep, used = [], 0
            for t in T_all:
                n = (int(t) + shape.B - 1) // shape.B
                if used + n <= budget:
                    keep.append(int(t))
                    used += n
            return np.array(keep, dtype=np.int64)

        def requests(T, seed):
            off = np.concatenate([[0], np.cumsum((T + shape.B - 1) // shape.B)]).astype(np.int64)
            rng = np.random.default_rng(seed)
            return (wl.KVRequests(T, off, rng.permutation(NBs)[:off[-1]].astype(np.int32)),
                    wl.KVRequests(T, off, rng.permutation(NBs)[:off[-1]].astype(np.int32)))

        self.src, self.dst = requests(first_requests(NBs), wl.SEED_BASE + 20)
        self.src1, self.dst1 = requests(first_requests(min(single_blocks, NBs)), wl.SEED_BASE + 21)
        self.threads = max(1, min(threads, len(self.src.T)))
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
        # one decoder layer of the checkpoint, at its offsets inside a blob that holds just that layer
        ck = wl.config3()
        ids = [i for i, n in enumerate(ck.names) if n.startswith("layers.0.")]
        base = int(ck.byte_off[ids[0]])
        self.w_off = [int(ck.byte_off[i]) - base for i in ids]
        self.w_E, self.w_shapes, self.w_split = ck.E[ids], ck.shapes[ids], ck.split_dim[ids]
        self.w_bytes = [ck.nbytes(i) for i in ids]
        self.blob = np.zeros(sum(self.w_bytes), dtype=np.uint8)
        wl.fill_np(self.blob[:1 << 24], wl.SEED_BASE + 3, "normal")   # contents are opaque to the loops
        self.w_full = [np.zeros(n, dtype=np.uint8) for n in self.w_bytes]
        self.w_shard = [np.zeros(n // (8 if sd >= 0 else 1), dtype=np.uint8) for n, sd in zip(self.w_bytes, self.w_split)]
        self.single_bytes = oracle.packed_nbytes(shape.tuple, self.src1.T)
        self.desc = (f"oracle on {self.threads} threads: kv_pack NHD->HND + kv_unpack + kv_migrate of {len(self.src.T)} requests / "
                     f"{self.src.n_blocks} blocks ({self.packed.size / GB:.2f} GB payload) of the Llama-3-8B KV workload, weights full + "
                     f"1-of-8 shard of one decoder layer ({self.blob.size / GB:.2f} GB); 1 thread: kv_pack + kv_unpack of "
                     f"{len(self.src1.T)} requests / {self.src1.n_blocks} blocks ({self.single_bytes / GB:.2f} GB payload)")

    def run(self, single_thread: bool = True):
        """Returns (GB/s over all rows on `threads` threads, seconds of that part, per-part GB/s)."""
        o, s, src, dst, th = self.oracle, self.shape, self.src, self.dst, self.threads
        parts, clock = {}, time.perf_counter
        t0 = clock()
        o.kv_pack(s.tuple, o.NHD, s.chunk_bytes, self.planes, src.T, src.bt_off, src.bt, o.HND, self.packed, threads=th)
        o.kv_unpack(s.tuple, o.NHD, s.chunk_bytes, self.planes2, dst.T, dst.bt_off, dst.bt, o.HND, self.packed, threads=th)
        t1 = clock()
        o.kv_migrate(s.tuple, o.NHD, s.chunk_bytes, self.planes, o.NHD, s.chunk_bytes, self.planes2, src.T, src.bt_off, src.bt, dst.bt, threads=th)
        t2 = clock()
        o.weights(self.w_off, self.w_E, self.w_shapes, np.full(len(self.w_off), -1), 0, 1, self.blob, self.w_full, threads=th)
        t3 = clock()
        o.weights(self.w_off, self.w_E, self.w_shapes, self.w_split, 0, 8, self.blob, self.w_shard, threads=th)
        t4 = clock()
        kv, wf, wsh = self.packed.size, self.blob.size, sum(a.size for a in self.w_shard)
        parts["a1_a2_kv_pack_unpack"] = 2 * 2 * kv / (t1 - t0) / GB
        parts["a3_kv_migrate"] = 2 * kv / (t2 - t1) / GB
        parts["a4_weights_full"] = 2 * wf / (t3 - t2) / GB
        parts["a5_weights_shard"] = 2 * wsh / (t4 - t3) / GB
        total = 2 * (3 * kv + wf + wsh)
        if single_thread:
            src1, dst1 = self.src1, self.dst1
            t5 = clock()
            o.kv_pack(s.tuple, o.NHD, s.chunk_bytes, self.planes, src1.T, src1.bt_off, src1.bt, o.HND, self.packed, threads=1)
            o.kv_unpack(s.tuple, o.NHD, s.chunk_bytes, self.planes2, dst1.T, dst1.bt_off, dst1.bt, o.HND, self.packed, threads=1)
            parts["a1_a2_kv_pack_unpack_1_thread"] = 2 * 2 * self.single_bytes / (clock() - t5) / GB
        return total / (t4 - t0) / GB, t4 - t0, parts


def run_reference(args):
    """`--impl reference`: the oracle is the reference arm of this tier.  The sample of a step is
    sized from a short calibration so that warm-up plus timed steps end within a few minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    threads = os.cpu_count() or 1
    blocks = args.oracle_blocks
    probe = OracleSample(min(64, blocks), threads)
    _, dt, _ = probe.run(single_thread=False)
    per_block = dt / max(1, probe.src.n_blocks)          # the layer of weights rides along: an overestimate
    budget_s = 150.0 / max(1, args.steps + args.warmup)
    blocks = int(max(32, min(blocks, budget_s / per_block)))
    del probe
    sample = OracleSample(blocks, threads)
    vals, dts = [], []
    for i in range(args.warmup + args.steps):
        v, dt, _ = sample.run(single_thread=False)
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
    cpu_v, cpu_desc, cpu_parts = None, "skipped", None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sample = OracleSample(args.oracle_blocks, threads)
        cpu_v, _, cpu_parts = sample.run()
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
    if args.host_copy_path:
        host_tune["copy_path"] = args.host_copy_path
    if args.host_tile_order:
        host_tune["tile_order"] = args.host_tile_order
    torch.cuda.synchronize()  # the fills above: a first cudaMalloc inside plan creation would wait for them
    t_plan0 = time.perf_counter()
    plans = []
    for src, dst in waves:
        kw = dict(T=src.T, bt_off=src.bt_off)
        plans.append(dict(
            pack=tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, s, src_pool=plA, packed_layout=tc.TC_HND, packed_bytes=Q.numel(), bt_src=src.bt, tuning=tune or None, **kw)),
            unpack=tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, s, dst_pool=plB, packed_layout=tc.TC_HND, packed_bytes=Q.numel(), bt_dst=dst.bt, tuning=tune or None, **kw)),
            migrate=tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, s, src_pool=plA, dst_pool=plB, bt_src=src.bt, bt_dst=dst.bt, tuning=tune or None, **kw)),
            src=src, dst=dst, payload=int(src.T.sum()) * shape.token_bytes))
    nbytes = [ck.nbytes(i) for i in range(ck.N)]
    mk_w = lambda tn, **kw: tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, blob_bytes=ck.nbytes_total, tuning=tn or None, **kw))
    w_full, w_shard = mk_w(tune), mk_w(tune, split_dim=ck.split_dim, rank=args.shard_rank, world=W)
    plan_ms = 1e3 * (time.perf_counter() - t_plan0)
    n_plans = 3 * len(waves) + 2

    def host_plans(path):
        """The same calls with the packed buffer and the blob in pinned host memory: plans for the
        staged path (copy engines + staging rings) or the zero-copy path (kernel loads / stores)."""
        flags = tc.TC_PLAN_STAGED if path == "staged" else 0
        hp = dict(kv=[], path=path)
        for p in plans:
            kw = dict(T=p["src"].T, bt_off=p["src"].bt_off, tuning=host_tune or None, flags=flags, packed_layout=tc.TC_HND, packed_bytes=Q.numel())
            hp["kv"].append((tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, s, src_pool=plA, bt_src=p["src"].bt, **kw)),
                             tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, s, dst_pool=plB, bt_dst=p["dst"].bt, **kw)), p["payload"]))
        hp["w_full"] = mk_w(host_tune, flags=flags)
        hp["w_shard"] = mk_w(host_tune, split_dim=ck.split_dim, rank=args.shard_rank, world=W, flags=flags)
        hp["launches"] = (sum(a.stats().launches_per_execute + b.stats().launches_per_execute for a, b, _ in hp["kv"])
                          + hp["w_full"].stats().launches_per_execute + hp["w_shard"].stats().launches_per_execute)
        return hp

    def drop_host_plans(hp):
        for a, b, _ in hp["kv"]:
            a.destroy()
            b.destroy()
        hp["w_full"].destroy()
        hp["w_shard"].destroy()

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

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    with torch.cuda.stream(stream):
        for _ in range(args.warmup):
            step([])
        barrier()
        sampler.mark_begin()
        ev_all = []
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for _ in range(args.steps):
            ev = []
            step(ev)
            ev_all.append(ev)
        t1.record(stream)
        barrier()
        sampler.mark_end()
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
    e2e_all = {}
    e2e_skipped = None
    avail = mem_available()
    want_extras = not args.no_extras and world == 1
    burst_bytes = 0
    if want_extras and (args.extras == "all" or "config4" in args.extras.split(",")) and not args.only_kv_shapes and not args.only_misaligned:
        burst_bytes = burst_host_blocks(args, avail) * shape.block_bytes
    can_duplex = False
    if not args.no_e2e:
        # pinned host memory is per process: N ranks on one node share the node's RAM
        budget = 0.6 * avail / world
        need_duplex, need_serial = 2 * max_packed + ck.nbytes_total, max_packed + ck.nbytes_total
        can_duplex = need_duplex <= budget
        if need_serial > budget:
            e2e_skipped = (f"skipped: {need_serial / GB:.0f} GB of pinned host memory per rank needed, "
                           f"{budget / GB:.0f} GB available per rank with {world} ranks on this node")
    e2e_bytes = 0 if (args.no_e2e or e2e_skipped) else ((2 if can_duplex else 1) * max_packed + ck.nbytes_total + (1 << 20))
    arena = PinnedArena(torch, max(e2e_bytes, burst_bytes)) if max(e2e_bytes, burst_bytes) else None
    args.pinned_arena = arena
    if not args.no_e2e and e2e_skipped is None:
        Qh = arena.take(max_packed)
        Qh2 = arena.take(max_packed) if can_duplex else Qh
        blob_h = arena.take(ck.nbytes_total)
        blob_h.copy_(blob)
        probe = torch.empty(4096, dtype=torch.uint8, pin_memory=True)
        stream_u = torch.cuda.Stream()
        ev_fork, ev_join = torch.cuda.Event(), torch.cuda.Event()
        torch.cuda.synchronize()
        n_c = min(Qh.numel(), 4 << 30)

        def ceiling(fn, nbytes):  # cudaMemcpyAsync on the same pinned allocation, best of 4
            best = 1e9
            for _ in range(4):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                fn()
                b.record(stream)
                torch.cuda.synchronize()
                best = min(best, a.elapsed_time(b))
            return nbytes / (best * 1e-3) / GB

        dup_ev = {}

        def both_ways():  # both directions at once with cudaMemcpyAsync, each timed on its own stream
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            ev_fork.record(stream)
            stream_u.wait_event(ev_fork)
            ev[0].record(stream)
            Qh[:n_c].copy_(Q[:n_c], non_blocking=True)
            ev[1].record(stream)
            with torch.cuda.stream(stream_u):
                ev[2].record(stream_u)
                poolB[:n_c].copy_(Qh2[:n_c], non_blocking=True)
                ev[3].record(stream_u)
                ev_join.record(stream_u)
            stream.wait_event(ev_join)
            dup_ev["ev"] = ev

        with torch.cuda.stream(stream):
            ceil_h2d = ceiling(lambda: Q[:n_c].copy_(Qh[:n_c], non_blocking=True), n_c)
            ceil_d2h = ceiling(lambda: Qh[:n_c].copy_(Q[:n_c], non_blocking=True), n_c)
            ceil_bidir = ceiling(both_ways, 2 * n_c) if can_duplex else None
        ceilings = {"h2d_cudaMemcpyAsync": ceil_h2d, "d2h_cudaMemcpyAsync": ceil_d2h, "both_directions_at_once_summed": ceil_bidir}
        dup_h2d = dup_d2h = None
        if can_duplex:  # the rate of each direction while the other is busy (last repetition)
            dup_d2h = n_c / (dup_ev["ev"][0].elapsed_time(dup_ev["ev"][1]) * 1e-3) / GB
            dup_h2d = n_c / (dup_ev["ev"][2].elapsed_time(dup_ev["ev"][3]) * 1e-3) / GB
            ceilings.update({"h2d_while_d2h_runs": dup_h2d, "d2h_while_h2d_runs": dup_d2h})

        def ideal_ms(h2d_bytes, d2h_bytes):
            """The shortest a step can take at cudaMemcpyAsync rates on contiguous buffers: both directions
            run together at their contended rates until the shorter one is done, the rest runs alone (a
            step moves more bytes to the device than back: the weights only travel one way)."""
            t_h, t_d = h2d_bytes / (dup_h2d * GB), d2h_bytes / (dup_d2h * GB)
            if t_d <= t_h:
                return 1e3 * (t_d + (h2d_bytes - dup_h2d * GB * t_d) / (ceil_h2d * GB))
            return 1e3 * (t_h + (d2h_bytes - dup_d2h * GB * t_h) / (ceil_d2h * GB))

        def run_e2e(hp, duplex, steps, warmup):
            """Offload every wave to pinned host memory and reload it into the second pool; load the
            weights from the pinned blob; read a result back.  duplex: the link is full duplex, so wave
            k+1 is offloaded (stream) while wave k is reloaded (stream_u), through two host buffers."""
            Qhs = (Qh, Qh2)
            su = stream_u.cuda_stream if duplex else sp
            s_u = stream_u if duplex else stream
            ev_packed = [torch.cuda.Event() for _ in range(2)]
            ev_unpacked = [torch.cuda.Event() for _ in range(2)]

            def one_step():
                h2d = d2h = 0
                ev_fork.record(stream)
                s_u.wait_event(ev_fork)
                tc.tc_weights_materialize(hp["w_full"], blob_h, full_ptrs, su)
                tc.tc_weights_materialize(hp["w_shard"], blob_h, shard_ptrs, su)
                h2d += sum(full_sizes) + sum(shard_sizes)
                for k, (pack_h, unpack_h, payload) in enumerate(hp["kv"]):
                    i = k % 2 if duplex else 0
                    if k >= (2 if duplex else 1):
                        stream.wait_event(ev_unpacked[i])                 # the host buffer is free again
                    tc.tc_kv_pack(pack_h, [poolA], [Qhs[i]], sp)         # offload (device -> host)
                    ev_packed[i].record(stream)
                    s_u.wait_event(ev_packed[i])
                    tc.tc_kv_unpack(unpack_h, [Qhs[i]], [poolB], su)     # reload (host -> device)
                    ev_unpacked[i].record(s_u)
                    d2h += payload
                    h2d += payload
                with torch.cuda.stream(s_u):
                    probe.copy_(dst_full[-4096:], non_blocking=True)      # read a result back
                    ev_join.record(s_u)
                stream.wait_event(ev_join)
                d2h += 4096
                return h2d, d2h

            with torch.cuda.stream(stream):
                for _ in range(warmup):
                    one_step()
                barrier()
                marks = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
                marks[0].record(stream)
                for k in range(steps):
                    h2d, d2h = one_step()
                    marks[k + 1].record(stream)
                barrier()
            per_step = [marks[k].elapsed_time(marks[k + 1]) for k in range(steps)]
            e_ms = ranks.max_ms(marks[0].elapsed_time(marks[steps]))
            link = world * (h2d + d2h) * steps / (e_ms * 1e-3) / GB
            serial_ceiling = (h2d + d2h) / (h2d / ceil_h2d + d2h / ceil_d2h)
            # same byte convention as `value`: every payload byte is read once and written once
            return {"value": world * 2 * (h2d + d2h - 4096) * steps / (e_ms * 1e-3) / GB, "unit": "GB/s",
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": steps, "warmup": warmup,
                    "ms_per_step": e_ms / steps, "ms_per_step_median": statistics.median(per_step),
                    "ms_per_step_min_max": [min(per_step), max(per_step)],
                    "host_link_GBps": link, "host_link_ceiling_GBps": ceilings,
                    "host_link_frac_of_ceiling": link / world / (ceil_bidir if duplex else serial_ceiling),
                    "ceiling_used": "both_directions_at_once_summed" if duplex else "serial mix of the one-direction ceilings",
                    "frac_of_ideal_schedule": (ideal_ms(h2d, d2h) / (e_ms / steps)) if duplex else None,
                    "kv_host_path": hp["path"], "schedule": "duplex" if duplex else "serial", "gpu_launches_per_step": hp["launches"]}

        want_duplex = args.e2e_schedule == "duplex" and can_duplex
        runs = [("staged", want_duplex)] if args.host_path == "staged" else []
        runs += [("zerocopy", False), ("zerocopy", True)] if can_duplex else [("zerocopy", False)]
        if args.host_path == "zerocopy":
            runs = [r for r in runs if r[0] == "zerocopy"]
        made = {}
        for path, duplex in runs:
            if path not in made:
                made[path] = host_plans(path)
            key = f"{path}_{'duplex' if duplex else 'serial'}"
            e2e_all[key] = run_e2e(made[path], duplex, args.e2e_steps, args.e2e_warmup)
        if can_duplex and "staged" in made and "zerocopy" in made and args.e2e_schedule == "duplex":
            # the offload by kernel stores straight into pinned memory (they keep their speed while the
            # other direction is busy), the reload and the weights through the copy engines
            st, zc = made["staged"], made["zerocopy"]
            mix = dict(kv=[(z[0], s_[1], s_[2]) for z, s_ in zip(zc["kv"], st["kv"])], path="offload zerocopy, reload staged",
                       w_full=st["w_full"], w_shard=st["w_shard"])
            mix["launches"] = (sum(a.stats().launches_per_execute + b.stats().launches_per_execute for a, b, _ in mix["kv"])
                               + st["w_full"].stats().launches_per_execute + st["w_shard"].stats().launches_per_execute)
            e2e_all["offload_zerocopy_reload_staged_duplex"] = run_e2e(mix, True, args.e2e_steps, args.e2e_warmup)
        for hp in made.values():
            drop_host_plans(hp)
        best = max(e2e_all, key=lambda k: e2e_all[k]["host_link_GBps"])
        e2e = dict(e2e_all[best])
        e2e["note"] = ("the fastest of the host paths measured in this run (all of them under e2e_paths). Packed KV buffer and "
                       "weight blob in pinned host memory. staged: copy engines + device staging rings + D2D kernel (the TP "
                       "shard's strided slices stay zero copy); zerocopy: kernel loads / stores on host memory; host_link_GBps "
                       "counts every byte once, in its direction; `value` counts it read and written like the device metric")
        del Qh, Qh2, blob_h
        arena.reset()

    extras = None
    if want_extras:
        for p in plans:
            for k in ("pack", "unpack", "migrate"):
                p[k].destroy()
        for w in (w_full, w_shard):
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
        "e2e_zerocopy": e2e_all.get("zerocopy_duplex") or e2e_all.get("zerocopy_serial"),
        "e2e_paths": e2e_all or None,
        "roofline": roofline, "rows": per_row, "other_workloads": extras,
        "cpu_baseline": {"value": cpu_v, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": cpu_desc, "parts_GBps": cpu_parts},
    }
    print(json.dumps(line), flush=True)
    if extras and "FAILED" in extras:  # the context may be beyond an orderly teardown
        sys.stderr.flush()
        os._exit(0)
    ranks.close()


def b2b_ms(torch, stream, fn, reps=5, warm=2):
    """Device milliseconds per call of fn: `reps` calls enqueued back to back inside one event pair,
    behind `warm` untimed ones that are still running when the first event is enqueued.  The host
    side of a call (marshalling the pointer table, checks, the launch itself) then overlaps the GPU
    work of the call before it; with a synchronise before every timed launch a short kernel would be
    charged for the time the idle GPU waits for the host.  Whatever other streams still run (the
    fill of a fresh pool on the default stream) is waited for first: plan creation does not."""
    torch.cuda.synchronize()
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
    host = torch.empty(ck.nbytes_total, dtype=torch.uint8, pin_memory=True)
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
    cases += [(f"src+{a}", a, 0, auto) for a in (8, 4, 2, 1)] + [("dst+1", 0, 1, auto), ("both+1", 1, 1, auto), ("src+3 dst+9", 3, 9, auto), ("src+9 dst+3", 9, 3, auto)]
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
    # few KV heads (planes of 8 KiB, four to a tile) through misaligned pointers
    shape = wl.KVShape(28, 16, 2, 128)
    s = shape.tuple
    NB = int(((1 if args.small else 4) << 30) // shape.block_bytes)
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
    few = {"kv_payload_bytes": payload, "planes_per_tile": int(mig.descriptors(0)[0].planes_per_tile)}
    A, B, Q = rawA.data_ptr(), rawB.data_ptr(), rawQ.data_ptr()
    for label, a_src, a_dst in (("aligned", 0, 0), ("src+2", 2, 0), ("both+1", 1, 1)):
        res = {}
        for name, fn in (("a1_pack", lambda: tc.tc_kv_pack(pk, [A + a_src], [Q + a_dst], sp)),
                         ("a2_unpack", lambda: tc.tc_kv_unpack(up, [Q + a_src], [B + a_dst], sp)),
                         ("a3_migrate", lambda: tc.tc_kv_pack(mig, [A + a_src], [B + a_dst], sp))):
            res[name] = 2 * payload / (b2b_ms(torch, stream, fn, reps=reps, warm=warm) * 1e-3) / GB
        res["min_frac_of_measured_peak"] = min(res.values()) / peak
        few[label] = res
    out["2 KV heads (L28 B16 H2 D128, 4 GiB pool)"] = few
    for p_ in (pk, up, mig):
        p_.destroy()
    del rawA, rawB, rawQ
    torch.cuda.empty_cache()
    # rows whose length is not a multiple of 16 (head_dim 100 / 66 / 65 in 2-byte elements): aligned
    # pointers, but every row of a tile has its own alignment
    odd = {}
    for D in (100,) if args.small else (100, 66, 65):
        shape = wl.KVShape(32, 16, 8, D, 2)
        s = shape.tuple
        NB = int(((1 if args.small else 4) << 30) // shape.block_bytes)
        WB = NB // 2
        _, _, _, waves = wl.config2(NB=NB, R=256, wave_blocks=WB, NB_dst=WB, shape=shape)
        src, dst = waves[0]
        payload = int(src.T.sum()) * shape.token_bytes
        A = torch.empty(NB * shape.block_bytes, **u8)
        B = torch.empty(WB * shape.block_bytes, **u8)
        Q = torch.empty(payload, **u8)
        plA = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * shape.chunk_bytes, slot_bytes=A.numel())
        plB = tc.pool(tc.TC_NHD, WB, 1, plane_stride=WB * shape.chunk_bytes, slot_bytes=B.numel())
        kw = dict(T=src.T, bt_off=src.bt_off)
        pk = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, s, src_pool=plA, packed_layout=tc.TC_HND, bt_src=src.bt, **kw))
        up = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, s, dst_pool=plB, packed_layout=tc.TC_HND, bt_dst=dst.bt, **kw))
        mig = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, s, src_pool=plA, dst_pool=plB, bt_src=src.bt, bt_dst=dst.bt, **kw))
        res = {"alignment_of_the_geometry_bytes": int(pk.stats().vec_bytes[0])}
        for name, fn in (("a1_pack", lambda: tc.tc_kv_pack(pk, [A], [Q], sp)), ("a2_unpack", lambda: tc.tc_kv_unpack(up, [Q], [B], sp)),
                         ("a3_migrate", lambda: tc.tc_kv_pack(mig, [A], [B], sp))):
            res[name] = 2 * payload / (b2b_ms(torch, stream, fn, reps=reps, warm=warm) * 1e-3) / GB
        odd[f"rows of {2 * D} bytes"] = res
        for p_ in (pk, up, mig):
            p_.destroy()
        del A, B, Q
        torch.cuda.empty_cache()
    out["row length not a multiple of 16 (L32 B16 H8, 4 GiB pool, aligned pointers)"] = odd
    torch.cuda.empty_cache()
    return out


def extra_config0(args, tc, torch, stream, out):
    sp = stream.cuda_stream
    u8 = dict(dtype=torch.uint8, device="cuda")
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


def extra_weights(args, tc, torch, stream, out):
    sp = stream.cuda_stream
    u8 = dict(dtype=torch.uint8, device="cuda")
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


def extra_config3(args, tc, torch, stream, out):
    """configs[3]: Llama-3-70B-shaped KV migration between two pools on the GPU.  The workload has
    about 35 waves of <= 4096 blocks; five of them are timed - the first, the last and three seeded
    ones in between - each with its own plan (created outside the timed launches)."""
    sp = stream.cuda_stream
    u8 = dict(dtype=torch.uint8, device="cuda")
    shape = wl.LLAMA3_70B_KV
    free, _ = torch.cuda.mem_get_info()
    NB = 4096
    while 2 * NB * shape.block_bytes > 0.8 * free:
        NB //= 2
    _, _, _, waves = wl.config4(NB=NB)
    if args.small:
        waves = waves[:1]
    pick = sorted({0, len(waves) - 1, *[int(x) for x in np.random.default_rng(wl.SEED_BASE + 40).choice(len(waves), size=min(3, len(waves)), replace=False)]})
    A = torch.empty(NB * shape.block_bytes, **u8)
    A.fill_(7)
    B = torch.empty(NB * shape.block_bytes, **u8)
    B.fill_(9)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * shape.chunk_bytes, slot_bytes=A.numel())
    pl_hnd = tc.pool(tc.TC_HND, NB, 1, plane_stride=NB * shape.chunk_bytes, slot_bytes=A.numel())
    torch.cuda.synchronize()  # the fills above are still running; plan upload would wait for them
    per_wave, create, tot_bytes, tot_ms, tot_ms_t = [], [], 0, 0.0, 0.0
    for w in pick:
        src, dst = waves[w]
        kw = dict(T=src.T, bt_off=src.bt_off, bt_src=src.bt, bt_dst=dst.bt)
        t0 = time.perf_counter()
        mig = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape.tuple, src_pool=pl, dst_pool=pl, **kw))
        create.append(1e3 * (time.perf_counter() - t0))
        mig_t = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape.tuple, src_pool=pl, dst_pool=pl_hnd, **kw))
        payload = int(src.T.sum()) * shape.token_bytes
        ms = b2b_ms(torch, stream, lambda: tc.tc_kv_pack(mig, [A], [B], sp), reps=3)
        ms_t = b2b_ms(torch, stream, lambda: tc.tc_kv_pack(mig_t, [A], [B], sp), reps=3)
        per_wave.append({"wave": w, "requests": len(src.T), "blocks": src.n_blocks, "payload_bytes": payload, "ms": ms,
                         "GBps": 2 * payload / (ms * 1e-3) / GB, "GBps_into_an_HND_pool": 2 * payload / (ms_t * 1e-3) / GB})
        tot_bytes += payload
        tot_ms += ms
        tot_ms_t += ms_t
        mig.destroy()
        mig_t.destroy()
    peak, _ = measured_peaks()
    res = {"pool_blocks": NB, "waves_in_workload": len(waves), "waves_timed": pick, "payload_bytes": tot_bytes,
           "GBps": 2 * tot_bytes / (tot_ms * 1e-3) / GB, "frac_of_measured_peak": 2 * tot_bytes / (tot_ms * 1e-3) / GB / peak,
           "GBps_into_an_HND_pool": 2 * tot_bytes / (tot_ms_t * 1e-3) / GB, "ms_total": tot_ms,
           "plan_create_ms": statistics.mean(create), "per_wave": per_wave}
    out["configs[3] 70B KV migrate (first, last and three seeded waves)"] = res
    # for comparison, unfused: pack into a device buffer, then unpack (twice the traffic).  The
    # buffer takes what memory is left, so only the first requests of wave 0 that fit take part.
    src, dst = waves[0]
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
        ms_two = b2b_ms(torch, stream, lambda: (tc.tc_kv_pack(pk, [A], [Q], sp), tc.tc_kv_unpack(up, [Q], [B], sp)), reps=3)
        ms_one = b2b_ms(torch, stream, lambda: tc.tc_kv_pack(fused, [A], [B], sp), reps=3)
        res["fused_vs_pack_then_unpack"] = {"requests": k, "payload_bytes": part, "ms_fused_migrate": ms_one,
                                            "ms_pack_then_unpack_through_a_device_buffer": ms_two}
        for p_ in (pk, up, fused):
            p_.destroy()
        del Q
    del A, B
    torch.cuda.empty_cache()


def extra_config4(args, tc, torch, stream, out):
    """configs[4]: multi-turn prefix-reload burst.  512 sessions; every scheduler step reloads
    about 6 100 cached 2 MiB pages from a paged pinned host pool into scattered device blocks and
    offloads about 1 280 new blocks, one MIXED plan per step (created, executed on two streams,
    synchronised and destroyed inside the timed region), 200 steps.  The ceilings it is held
    against are cudaMemcpyAsync on the burst's own pinned pool, measured here: one direction
    alone and both directions at once."""
    sp = stream.cuda_stream
    u8 = dict(dtype=torch.uint8, device="cuda")
    shape = wl.LLAMA3_8B_KV
    NBd, n_steps = 20000, args.burst_steps
    arena = getattr(args, "pinned_arena", None)
    rule = burst_host_blocks(args, mem_available() + (arena.buf.numel() if arena else 0))
    NBh = min(rule, arena.buf.numel() // shape.block_bytes) if arena else rule
    dev = torch.empty(NBd * shape.block_bytes, **u8)
    dev.fill_(3)
    torch.cuda.synchronize()
    if arena is None:
        arena = PinnedArena(torch, NBh * shape.block_bytes)
    arena.reset()
    host = arena.take(NBh * shape.block_bytes)
    pin_s = arena.seconds
    dev_pool = tc.pool(tc.TC_NHD, NBd, 1, plane_stride=NBd * shape.chunk_bytes, slot_bytes=dev.numel())
    host_pool = tc.pool(tc.TC_HND, NBh, 1, plane_stride=shape.chunk_bytes, block_stride=shape.block_bytes, slot_bytes=host.numel())
    s2 = torch.cuda.Stream()
    # ceilings: contiguous cudaMemcpyAsync on this machine, 4 GiB, best of 3
    n_c = min(host.numel() // 2, 4 << 30)
    fork, join = torch.cuda.Event(), torch.cuda.Event()

    def best_of(fn, nbytes, reps=3):
        best = 1e9
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            with torch.cuda.stream(stream):
                a.record(stream)
                fn()
                b.record(stream)
            torch.cuda.synchronize()
            best = min(best, a.elapsed_time(b))
        return nbytes / (best * 1e-3) / GB

    dup = {}

    def both():  # each direction timed on its own stream while the other runs
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        fork.record(stream)
        s2.wait_event(fork)
        ev[0].record(stream)
        dev[:n_c].copy_(host[:n_c], non_blocking=True)
        ev[1].record(stream)
        with torch.cuda.stream(s2):
            ev[2].record(s2)
            host[n_c:2 * n_c].copy_(dev[n_c:2 * n_c], non_blocking=True)
            ev[3].record(s2)
            join.record(s2)
        stream.wait_event(join)
        dup["ev"] = ev

    ceil_h2d = best_of(lambda: dev[:n_c].copy_(host[:n_c], non_blocking=True), n_c)
    ceil_d2h = best_of(lambda: host[:n_c].copy_(dev[:n_c], non_blocking=True), n_c)
    ceil_both = best_of(both, 2 * n_c)
    # rates of the two directions while both are busy (from the last repetition: the shorter copy ends
    # first, so these are lower bounds of the contended rates)
    dup_h2d = n_c / (dup["ev"][0].elapsed_time(dup["ev"][1]) * 1e-3) / GB
    dup_d2h = n_c / (dup["ev"][2].elapsed_time(dup["ev"][3]) * 1e-3) / GB

    def ideal_ms(h2d_bytes, d2h_bytes):
        """The shortest a step can take at cudaMemcpyAsync rates on contiguous memory: both directions
        run together at their contended rates until the shorter one is done, the rest runs alone."""
        t_h, t_d = h2d_bytes / (dup_h2d * GB), d2h_bytes / (dup_d2h * GB)
        if t_d <= t_h:
            return 1e3 * (t_d + (h2d_bytes - dup_h2d * GB * t_d) / (ceil_h2d * GB))
        return 1e3 * (t_h + (d2h_bytes - dup_d2h * GB * t_h) / (ceil_d2h * GB))

    burst_tune = {}
    if args.host_ctas:
        burst_tune["max_ctas"] = args.host_ctas
    if args.burst_tile_order:
        burst_tune["tile_order"] = args.burst_tile_order
    paths = ["zerocopy", "staged", "mixed"] if args.burst_paths == "all" else [args.burst_paths]
    results = {}
    for path in paths:
        # a comparison path runs a tenth of the steps; the reported one runs them all
        steps_here = n_steps if path == paths[0] else max(2, n_steps // 10)
        create, h2d, d2h = [], 0, 0
        flags = {"staged": tc.TC_PLAN_STAGED, "mixed": tc.TC_PLAN_STAGED | tc.TC_PLAN_OFFLOAD_ZERO_COPY, "zerocopy": 0}[path]
        torch.cuda.synchronize()
        t_all = None
        dev_ms = []
        all_steps = list(wl.config5(NB_dev=NBd, NB_host=NBh, steps=steps_here + 1))  # drawn before the clock starts
        for i, st in enumerate(all_steps):
            if i == 1:  # step 0 is the warm-up
                torch.cuda.synchronize()
                t_all = time.perf_counter()
            t0 = time.perf_counter()
            plan = tc.tc_plan_create(tc.kv_spec(
                tc.TC_KV_MIXED, shape.tuple, src_pool=dev_pool, dst_pool=host_pool,
                T=st.offload_T, bt_off=st.offload_off, bt_src=st.offload_dev, bt_dst=st.offload_host,
                reload=dict(T=st.reload_T, bt_off=st.reload_off, bt_src=st.reload_host, bt_dst=st.reload_dev), flags=flags,
                tuning=burst_tune or None))
            if i >= 1:
                create.append(1e3 * (time.perf_counter() - t0))
                h2d += int(st.reload_T.sum()) * shape.token_bytes
                d2h += int(st.offload_T.sum()) * shape.token_bytes
            # the short offload is enqueued first: the reload's ~6 000 page copies fill the driver's
            # stream queue, so whatever is enqueued after it only starts when it is nearly done
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            ev[2].record(s2)
            tc.tc_kv_pack(plan, [dev], [host], s2.cuda_stream)
            ev[3].record(s2)
            ev[0].record(stream)
            tc.tc_kv_unpack(plan, [host], [dev], sp)
            ev[1].record(stream)
            try:
                torch.cuda.synchronize()   # a scheduler step ends when both directions have landed
            except Exception as e:         # say which step of which path it was
                raise RuntimeError(f"configs[4] burst: host path {path!r}, step {i} of {steps_here}, {len(st.reload_dev)} reload and "
                                   f"{len(st.offload_dev)} offload blocks") from e
            plan.destroy()
            if i >= 1:
                dev_ms.append((ev[0].elapsed_time(ev[1]), ev[2].elapsed_time(ev[3])))
        wall = time.perf_counter() - t_all
        ideal = ideal_ms(h2d / steps_here, d2h / steps_here)
        results[path] = {
            "steps": steps_here, "plans_per_s": steps_here / wall, "ms_per_step_wall": 1e3 * wall / steps_here, "plan_create_ms": statistics.mean(create),
            "h2d_GBps": h2d / wall / GB, "d2h_GBps": d2h / wall / GB, "link_GBps_both_directions": (h2d + d2h) / wall / GB,
            "h2d_bytes_per_step": h2d // steps_here, "d2h_bytes_per_step": d2h // steps_here,
            # the reload is the long leg of every step (5x the offload's bytes): the step cannot end before
            # h2d bytes / H2D ceiling; with the offload sharing the link, before h2d bytes / duplex share
            "device_ms_per_step_reload_stream": statistics.mean(x[0] for x in dev_ms), "device_ms_per_step_offload_stream": statistics.mean(x[1] for x in dev_ms),
            "ideal_ms_per_step_at_contiguous_cudaMemcpyAsync_rates": ideal, "frac_of_ideal_schedule": ideal / (1e3 * wall / steps_here),
            "h2d_frac_of_one_direction_ceiling": h2d / wall / GB / ceil_h2d,
            "h2d_frac_of_its_share_of_the_both_directions_ceiling": h2d / wall / GB / (ceil_both / 2),
            "d2h_frac_of_one_direction_ceiling": d2h / wall / GB / ceil_d2h}
    first = dict(results[paths[0]])
    first.update({
        "sessions": 512, "host_pool_blocks": NBh, "host_pool_rule_min_262144_half_MemAvailable": rule, "host_pool_GB": NBh * shape.block_bytes / GB,
        "pin_seconds": pin_s, "device_pool_blocks": NBd, "host_path": paths[0],
        "ceilings_GBps_cudaMemcpyAsync_on_this_pool": {"h2d": ceil_h2d, "d2h": ceil_d2h, "both_directions_at_once_summed": ceil_both,
                                                       "h2d_while_d2h_runs": dup_h2d, "d2h_while_h2d_runs": dup_d2h},
        "other_host_paths_on_a_tenth_of_the_steps": {k: v for k, v in results.items() if k != paths[0]} or None,
        "note": "wall clock over create + execute + synchronise + destroy of every step; reload and offload run concurrently on two "
                "streams. zerocopy: the kernel loads pages from and stores pages into the pinned host pool itself (one CTA per SM); "
                "staged: host pages travel one cudaMemcpyAsync each through the staging rings; mixed: the reload is staged, the "
                "offload stores straight into the host pool from the kernel"})
    out["configs[4] prefix-reload burst (mixed plan per step)"] = first
    del dev, host
    torch.cuda.empty_cache()


EXTRAS = [
    ("config0", extra_config0),
    ("weights", extra_weights),
    ("cold_path", lambda a, tc, torch, st, out: out.__setitem__("weights cold path: blob streamed from a file", cold_path(a, tc, torch, st))),
    ("moe", lambda a, tc, torch, st, out: out.__setitem__("transform_into: MoE expert stacking (Qwen3-30B-A3B-shaped layers)", moe_stacking(a, tc, torch, st))),
    ("kv_shapes", lambda a, tc, torch, st, out: out.__setitem__("rows a1-a3 on other KV geometries (8 GiB pools, first wave)", kv_shapes(a, tc, torch, st))),
    ("misaligned", lambda a, tc, torch, st, out: out.__setitem__("rows a1-a5: copy paths and misaligned base pointers (8 GiB pool, 4 GB checkpoint)", misaligned(a, tc, torch, st))),
    ("config3", extra_config3),
    ("config4", extra_config4),
]


def run_extras(args, tc, torch, stream):
    """Secondary workloads, reported beside the headline (`--extras a,b` runs only the named ones)."""
    want = None if args.extras == "all" else set(args.extras.split(","))
    if args.only_kv_shapes:  # profiler runs: just the KV geometries, a few GB on the device
        want = {"kv_shapes"}
    if args.only_misaligned:
        want = {"misaligned"}
    out = {}
    todo = [(name, fn) for name, fn in EXTRAS if want is None or name in want]
    for k, (name, fn) in enumerate(todo):
        try:
            fn(args, tc, torch, stream, out)
            torch.cuda.empty_cache()
        except Exception as e:  # noqa: BLE001
            # the headline numbers are already taken: report the failure beside them instead of
            # losing the whole line; a CUDA error is sticky, so the remaining extras are skipped
            import traceback
            traceback.print_exc(file=sys.stderr)
            out["FAILED"] = {"extra": name, "error": repr(e)[:500], "skipped_after_it": [n for n, _ in todo[k + 1:]]}
            break
    return out


def traffic_per_launch(algorithmic_bytes: float) -> float:
    """DRAM bytes of one full-size launch, scaled from an `ncu --set full` capture of a small
    case (226 MB wave, 700 MB checkpoint): reads = 1.0002 x payload (descriptors included);
    writes = payload less the ~50 MB of dirty lines still in L2 at kernel end."""
    payload = algorithmic_bytes / 2
    return 1.0002 * payload + max(payload - 50.7e6, 0.0)


def spawn_ranks(n: int) -> int:
    """`python bench.py --gpus N` without a launcher: start the N ranks ourselves (one process per
    GPU through torch.distributed.run on this node) with the same arguments; rank 0 prints the line."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


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
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--e2e-warmup", type=int, default=1)
    ap.add_argument("--oracle-blocks", type=int, default=1024)
    ap.add_argument("--tile-bytes", type=int, default=0)
    ap.add_argument("--ctas-per-sm", type=int, default=0)
    ap.add_argument("--no-extras", action="store_true", help="skip the secondary workloads (configs[3], configs[4])")
    ap.add_argument("--only-kv-shapes", action="store_true", help="of the secondary workloads run only the KV geometries (profiler captures)")
    ap.add_argument("--only-misaligned", action="store_true", help="of the secondary workloads run only the misaligned-pointer rows")
    ap.add_argument("--extras", default="all", help="secondary workloads to run: all, or a comma list of " + ",".join(n for n, _ in EXTRAS))
    ap.add_argument("--host-pool-blocks", type=int, default=0, help="configs[4]: pinned host pool size in 2 MiB blocks (0: min(262144, half of MemAvailable))")
    ap.add_argument("--burst-steps", type=int, default=200, help="configs[4]: scheduler steps timed (the workload has 200)")
    ap.add_argument("--burst-tile-order", type=int, default=0, help="configs[4]: tuning.tile_order of the step's plans (1: block after block instead of plane after plane)")
    ap.add_argument("--burst-paths", default="all", choices=["staged", "mixed", "zerocopy", "all"],
                    help="configs[4]: host path (all: zerocopy over all the steps, staged and mixed on a tenth of them)")
    ap.add_argument("--cold-layers", type=int, default=8, help="cold-path extra: layers of the checkpoint written to a file (8: 4.0 GB)")
    ap.add_argument("--moe-layers", type=int, default=8, help="expert-stacking extra: layers of the MoE checkpoint (8: 11 GB)")
    ap.add_argument("--host-ctas", type=int, default=0)
    ap.add_argument("--host-copy-path", type=int, default=0, help="tuning.copy_path of the e2e plans (1: through shared memory, bulk copies)")
    ap.add_argument("--host-tile-order", type=int, default=0, help="tuning.tile_order of the e2e plans")
    ap.add_argument("--host-path", default="staged", choices=["staged", "zerocopy"])
    ap.add_argument("--e2e-schedule", default="duplex", choices=["duplex", "serial"],
                    help="duplex: offload wave k+1 while wave k reloads (two streams, two host buffers)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        sys.exit(spawn_ranks(args.gpus))
    if args.dry_run:
        run_dry(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
