#!/usr/bin/env python
"""Throughput of the KDN store / retrieve / compose path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One step is one pass of the whole path over one batch of synthetic Llama-3-8B-shaped KV (32 layers, 8 KV
heads, head_dim 128, bf16, block_size 16, 16384-block pool), for the raw bf16 codec and again for the int8
group-64 codec:
    store     64 chunks x 512 tokens, gathered from fully fragmented block tables      (one batched call)
    retrieve  the same 64 chunks into 2048 other random blocks                         (one batched call)
    compose   10 chunks x 1024 tokens into one 10496-token request at cumulative offsets, theta 5e5, nine of
              the ten parts re-rotated, a 256-token suffix left untouched              (one call)
`value` is algorithmic GB/s over the step with every buffer resident in HBM; `e2e` is the same step with the
chunks in page-locked host memory, so every byte crosses the host link inside the timed region.
With --impl reference the CPU oracle is timed instead, on a bounded sample of the same workload.
The line printed last on stdout is the JSON record.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "store/retrieve/compose algorithmic GB/s (KV tokens/s reloaded alongside)"
UNIT = "GB/s"
WORKLOAD = ("llama3-8b KV (L32 H8 D128 bf16, block_size 16, 16384-block pool): store+retrieve 64x512 tokens, "
            "compose 10x1024 tokens (+256-token suffix), raw bf16 and int8-g64, fully fragmented tables")
N_CHUNKS, CHUNK_TOKENS = 64, 512
N_PARTS, PART_TOKENS, SUFFIX_TOKENS = 10, 1024, 256
RAW, INT8 = 0, 1
FALLBACK_HBM_GBS = 6650.0


def bytes_per_elem(codec: int) -> float:
    """Algorithmic bytes per KV element moved by one op: bf16 on the pool side + the chunk side."""
    return 4.0 if codec == RAW else 2.0 + 1.0 + 4.0 / 64.0


# ------------------------------------------------------------------------------------ CPU oracle leg --

class OracleSample:
    """The CPU oracle, as it stands, on a bounded sample of the bench workload.

    Each of `cores` threads takes its own chunk of `tokens` tokens of the 8B-shaped pool through store, retrieve and
    a re-rotating compose, for both codecs: the same six operations as one GPU step, on fewer tokens."""

    def __init__(self, cores: int, tokens: int):
        import oracle
        from paper_2409_13761_b200 import synth
        self.oracle, self.cores, self.tokens = oracle, cores, tokens
        self.shape = synth.LLAMA3_8B.with_(n_blocks=128)
        k, v = synth.make_pool(self.shape, "cpu")
        self.pool = synth.pool_to_numpy(k, v)
        self.nblk = -(-tokens // self.shape.block_size)
        rng = np.random.default_rng(synth.SEED_TABLES)
        self.tables = [rng.permutation(self.shape.n_blocks)[:self.nblk].astype(np.int32) for _ in range(cores)]
        oracle.lib()
        self.pool_exec = ThreadPoolExecutor(max_workers=cores)

    def _work(self, i: int):
        sh, o, T = self.shape, self.oracle, self.tokens
        dst_pool = np.zeros((sh.n_layers, 2, self.nblk, sh.block_size, sh.n_kv_heads, sh.head_dim), np.uint16)
        dst = np.arange(self.nblk, dtype=np.int32)
        moved = 0.0
        for codec in (RAW, INT8):
            ch = o.store(self.pool, self.tables[i], 0, T, codec)
            o.retrieve(dst_pool, dst, 0, T, codec, ch)
            o.compose(dst_pool, dst, [(ch, T, codec, 1024 * (i + 1), 0)], sh.rope_theta)
            moved += 3 * T * sh.elems_per_token * bytes_per_elem(codec)
        return moved, 2 * 2 * T

    def run_pass(self):
        """One pass over all threads; returns (bytes moved, tokens reloaded, seconds)."""
        t0 = time.perf_counter()
        res = list(self.pool_exec.map(self._work, range(self.cores)))
        dt = time.perf_counter() - t0
        return sum(r[0] for r in res), sum(r[1] for r in res), dt

    def describe(self, passes: int, nbytes: float, dt: float) -> str:
        return ("%d pass(es) x %d threads, each one %d-token 8B-shaped chunk through store, retrieve and a re-rotating "
                "compose, raw bf16 and int8-g64 (%.2f GB moved, %.1f s wall)" % (passes, self.cores, self.tokens, nbytes / 1e9, dt))


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = len(os.sched_getaffinity(0))
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    # a full 512-token chunk per thread takes several seconds; shrink the sample so the whole run stays in minutes
    tokens = 512 if steps + warmup <= 12 else max(16, int(512 * 12 / (steps + warmup)) // 16 * 16)
    smp = OracleSample(cores, tokens)
    for _ in range(warmup):
        smp.run_pass()
    tb = tt = td = 0.0
    for _ in range(steps):
        b, t, dt = smp.run_pass()
        tb, tt, td = tb + b, tt + t, td + dt
    value = tb / td / 1e9
    desc = smp.describe(steps, tb, td)
    rec = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": 1e3 * td / steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16/int8 (fp32 codec, fp64 rotation)",
        "data": "synthetic", "config": {"workload": WORKLOAD, "sample": desc},
        "tokens_per_s_reloaded": tt / td,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(rec))


# ------------------------------------------------------------------------------------------ GPU leg --

class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
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
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])), mx.append(float(parts[1])), pw.append(float(parts[2]))
            except ValueError:
                continue
            for n, p in zip(names, parts[3:7]):
                if p.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


# DRAM bytes (read + write) per launch from the committed ncu capture of a reduced case (8 chunks per
# store/retrieve launch, 2 parts per compose launch; profiles/ncu_full_small_case_llama3_8b.md), scaled by the
# units a bench launch processes.  Valid only for the kernel source the capture was taken from.
NCU_KERNEL_SHA = "59ec05579632cb7b"
NCU_SMALL_CASE_BYTES = {"store_raw": (536.894720e6 + 485.936384e6, 8), "retrieve_raw": (536.895744e6 + 490.880256e6, 8),
                        "compose_raw": (268.468992e6 + 221.113088e6, 2), "store_int8": (536.903680e6 + 252.184576e6, 8),
                        "retrieve_int8": (285.241600e6 + 483.000064e6, 8), "compose_int8": (142.639616e6 + 213.129216e6, 2)}


def measured_traffic(op: str, units: int):
    import hashlib
    try:
        with open(os.path.join(ROOT, "paper_2409_13761_b200", "csrc", "kdn_kernels.cuh"), "rb") as fh:
            if hashlib.sha256(fh.read()).hexdigest()[:16] != NCU_KERNEL_SHA:
                return None                     # kernels changed since the counters were taken
    except OSError:
        return None
    nbytes, small_units = NCU_SMALL_CASE_BYTES[op]
    return nbytes * units / small_units


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def run_gpu(args) -> None:
    import torch
    from paper_2409_13761_b200 import kdn as K, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    shape = synth.LLAMA3_8B
    global N_CHUNKS, N_PARTS
    reduced = bool(args.pool_blocks or args.chunks or args.parts)
    if args.pool_blocks:
        shape = shape.with_(n_blocks=args.pool_blocks)
    N_CHUNKS = args.chunks or N_CHUNKS
    N_PARTS = args.parts or N_PARTS

    # ---- inputs (untimed): pool, tables, chunk buffers; every rank has its own copy of the same workload
    k, v = synth.make_pool(shape, dev, seed=synth.SEED_VALUES + rank)
    ctx = K.kdn_create(local)
    desc = K.pool_desc(shape.n_layers, shape.n_kv_heads, shape.head_dim, shape.block_size, shape.n_blocks,
                       [t.data_ptr() for t in k], [t.data_ptr() for t in v])
    pid = K.kdn_pool_register(ctx, desc)
    stream = torch.cuda.Stream(device=dev)
    s = stream.cuda_stream
    bs = shape.block_size
    blocks_per_chunk = CHUNK_TOKENS // bs
    blocks_per_part = PART_TOKENS // bs
    req_blocks = (N_PARTS * PART_TOKENS + SUFFIX_TOKENS) // bs
    all_src = synth.make_table(N_CHUNKS * blocks_per_chunk, shape.n_blocks, 1, synth.SEED_TABLES)
    all_dst = synth.make_table(N_CHUNKS * blocks_per_chunk, shape.n_blocks, 1, synth.SEED_TABLES + 1, exclude=all_src)
    part_src = synth.make_table(N_PARTS * blocks_per_part, shape.n_blocks, 1, synth.SEED_TABLES + 2,
                                exclude=np.concatenate([all_src, all_dst]))
    req_tab = synth.make_table(req_blocks, shape.n_blocks, 1, synth.SEED_TABLES + 3,
                               exclude=np.concatenate([all_src, all_dst, part_src]))
    d_src = torch.from_numpy(all_src).to(dev)
    d_dst = torch.from_numpy(all_dst).to(dev)
    d_part_src = torch.from_numpy(part_src).to(dev)
    d_req = torch.from_numpy(req_tab).to(dev)
    i32 = 4

    def make_sets(pinned: bool):
        """Chunk buffers and the op lists of one step, per codec."""
        sets = {}
        for codec in (RAW, INT8):
            cb = K.kdn_chunk_bytes(desc, CHUNK_TOKENS, codec)
            pb = K.kdn_chunk_bytes(desc, PART_TOKENS, codec)
            if pinned:
                chunks = torch.empty(N_CHUNKS * cb, dtype=torch.uint8).pin_memory()
                parts = torch.empty(N_PARTS * pb, dtype=torch.uint8).pin_memory()
                mem = K.KDN_MEM_PINNED_HOST
            else:
                chunks = torch.empty(N_CHUNKS * cb, dtype=torch.uint8, device=dev)
                parts = torch.empty(N_PARTS * pb, dtype=torch.uint8, device=dev)
                mem = K.KDN_MEM_DEVICE
            st_ops = [K.XferOp(d_src.data_ptr() + i * blocks_per_chunk * i32, blocks_per_chunk, 0,
                               K.Chunk(chunks.data_ptr() + i * cb, cb, CHUNK_TOKENS, codec, mem)) for i in range(N_CHUNKS)]
            rt_ops = [K.XferOp(d_dst.data_ptr() + i * blocks_per_chunk * i32, blocks_per_chunk, 0,
                               K.Chunk(chunks.data_ptr() + i * cb, cb, CHUNK_TOKENS, codec, mem)) for i in range(N_CHUNKS)]
            part_store = [K.XferOp(d_part_src.data_ptr() + j * blocks_per_part * i32, blocks_per_part, 0,
                                   K.Chunk(parts.data_ptr() + j * pb, pb, PART_TOKENS, codec, mem)) for j in range(N_PARTS)]
            req = K.ComposeReq(d_req.data_ptr(), req_blocks,
                               [K.Chunk(parts.data_ptr() + j * pb, pb, PART_TOKENS, codec, mem, 0) for j in range(N_PARTS)],
                               [j * PART_TOKENS for j in range(N_PARTS)], shape.rope_theta)
            sets[codec] = dict(chunks=chunks, parts=parts, store=st_ops, retrieve=rt_ops, part_store=part_store, req=req)
        return sets

    dev_sets = make_sets(False)
    for codec in (RAW, INT8):                      # fill the compose parts once (untimed)
        K.kdn_store(ctx, pid, dev_sets[codec]["part_store"], s)
    assert K.kdn_status_sync(ctx, s) == K.KDN_OK

    names = ["store_raw", "retrieve_raw", "compose_raw", "store_int8", "retrieve_int8", "compose_int8"]
    chunk_elems = N_CHUNKS * CHUNK_TOKENS * shape.elems_per_token
    part_elems = N_PARTS * PART_TOKENS * shape.elems_per_token
    op_bytes = {"store_raw": chunk_elems * bytes_per_elem(RAW), "retrieve_raw": chunk_elems * bytes_per_elem(RAW),
                "compose_raw": part_elems * bytes_per_elem(RAW), "store_int8": chunk_elems * bytes_per_elem(INT8),
                "retrieve_int8": chunk_elems * bytes_per_elem(INT8), "compose_int8": part_elems * bytes_per_elem(INT8)}
    op_tokens = {n: (N_CHUNKS * CHUNK_TOKENS if "compose" not in n else N_PARTS * PART_TOKENS) for n in names}
    step_bytes = float(sum(op_bytes.values()))
    reload_tokens = sum(op_tokens[n] for n in names if not n.startswith("store"))
    kernel_of = {"store_raw": "kdn_store_kernel<false>", "retrieve_raw": "kdn_retrieve_kernel<false>",
                 "compose_raw": "kdn_compose_kernel<true>", "store_int8": "kdn_store_kernel<true>",
                 "retrieve_int8": "kdn_retrieve_kernel<true>", "compose_int8": "kdn_compose_kernel<true>"}

    def step(sets, events=None):
        i = 0
        for codec in (RAW, INT8):
            for kind in ("store", "retrieve", "compose"):
                if events is not None:
                    events[i].record(stream)
                if kind == "store":
                    K.kdn_store(ctx, pid, sets[codec]["store"], s)
                elif kind == "retrieve":
                    K.kdn_retrieve(ctx, pid, sets[codec]["retrieve"], s)
                else:
                    K.kdn_compose(ctx, pid, [sets[codec]["req"]], s)
                i += 1
        if events is not None:
            events[i].record(stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing
    for _ in range(args.warmup):
        step(dev_sets)
    assert K.kdn_status_sync(ctx, s) == K.KDN_OK
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(len(names) + 1)] for _ in range(args.steps)]
    sampler = ClockSampler(torch.cuda.current_device() if "CUDA_VISIBLE_DEVICES" not in os.environ else local)
    barrier()
    sampler.start()
    launches0 = K.kdn_launch_count(ctx)
    t_begin = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_begin.record(stream)
    for it in range(args.steps):
        step(dev_sets, ev[it])
    t_end.record(stream)
    barrier()
    clocks = sampler.stop()
    launches = K.kdn_launch_count(ctx) - launches0
    status = K.kdn_status_sync(ctx, s)
    assert status == K.KDN_OK, K.kdn_strerror(status)
    elapsed_ms = t_begin.elapsed_time(t_end)
    op_ms = {n: float(np.mean([ev[it][i].elapsed_time(ev[it][i + 1]) for it in range(args.steps)]))
             for i, n in enumerate(names)}

    # ---- end to end: the same step with every chunk in page-locked host memory
    if args.no_e2e:
        if rank == 0:
            print(json.dumps({"note": "profiling run, not a bench record", "ops_ms": op_ms,
                              "ops_gbs": {n: op_bytes[n] / (op_ms[n] * 1e-3) / 1e9 for n in names}}))
        K.kdn_destroy(ctx)
        return
    host_sets = make_sets(True)
    for codec in (RAW, INT8):
        K.kdn_store(ctx, pid, host_sets[codec]["part_store"], s)
    assert K.kdn_status_sync(ctx, s) == K.KDN_OK
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    step(host_sets)
    assert K.kdn_status_sync(ctx, s) == K.KDN_OK
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        step(host_sets)
        st = K.kdn_status_sync(ctx, s)            # the step's result is read back: device status + all copies landed
        assert st == K.KDN_OK
    barrier()
    e2e_ms = (time.perf_counter() - t0) * 1e3
    d2h = sum(K.kdn_chunk_bytes(desc, CHUNK_TOKENS, c) * N_CHUNKS for c in (RAW, INT8)) + 4
    h2d = sum(K.kdn_chunk_bytes(desc, CHUNK_TOKENS, c) * N_CHUNKS + K.kdn_chunk_bytes(desc, PART_TOKENS, c) * N_PARTS
              for c in (RAW, INT8))

    # ---- host-link ceiling, same run: one large pinned cudaMemcpyAsync each way
    probe = host_sets[RAW]["chunks"][: 1 << 30]
    dprobe = dev_sets[RAW]["chunks"][: 1 << 30]
    link = {}
    for name, (dst_t, src_t) in {"h2d": (dprobe, probe), "d2h": (probe, dprobe)}.items():
        best = 0.0
        for _ in range(5):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            with torch.cuda.stream(stream):
                a.record(stream)
                dst_t.copy_(src_t, non_blocking=True)
                b.record(stream)
            torch.cuda.synchronize()
            best = max(best, probe.numel() / (a.elapsed_time(b) * 1e-3) / 1e9)
        link[name + "_gbs"] = best

    # ---- reduce over ranks (max time), print on rank 0
    times = torch.tensor([elapsed_ms, e2e_ms] + [op_ms[n] for n in names], dtype=torch.float64, device=dev)
    if dist is not None:
        dist.all_reduce(times, op=dist.ReduceOp.MAX)
    times = times.cpu().numpy()
    elapsed_ms, e2e_ms = float(times[0]), float(times[1])
    op_ms = {n: float(times[2 + i]) for i, n in enumerate(names)}
    if rank == 0:
        peak, peak_kind = measured_hbm_peak()
        ms_per_step = elapsed_ms / args.steps
        value = world * step_bytes / (ms_per_step * 1e-3) / 1e9
        ops = {n: {"ms": op_ms[n], "gbs": op_bytes[n] / (op_ms[n] * 1e-3) / 1e9,
                   "frac_of_%s_copy_peak" % peak_kind: op_bytes[n] / (op_ms[n] * 1e-3) / 1e9 / peak,
                   "frac_of_8000": op_bytes[n] / (op_ms[n] * 1e-3) / 1e9 / 8000.0,
                   "tokens_per_s": op_tokens[n] / (op_ms[n] * 1e-3), "kernel": kernel_of[n]} for n in names}
        top = max(names, key=lambda n: op_ms[n])
        traffic = measured_traffic(top, N_CHUNKS if "compose" not in top else N_PARTS)
        rec = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16/int8 (fp32 codec and rotation, fp64 angles)", "data": "synthetic",
            "config": {"workload": WORKLOAD if not reduced else "REDUCED (%d chunks, %d parts, %d blocks): not the bench workload" % (N_CHUNKS, N_PARTS, shape.n_blocks), "l2": "inputs larger than L2 (every op streams >= 1.9 GB once)",
                       "bytes_per_step": step_bytes},
            "tokens_per_s_reloaded": world * reload_tokens / (sum(op_ms[n] for n in names if not n.startswith("store")) * 1e-3),
            "ops": ops,
            "roofline": {"bound": "hbm", "kernel": kernel_of[top], "op": top, "achieved": ops[top]["gbs"], "peak": peak,
                         "peak_kind": "of " + peak_kind, "unit": "GB/s", "frac": ops[top]["gbs"] / peak,
                         "frac_of_nominal_8000": ops[top]["gbs"] / 8000.0, "traffic": traffic},
            "e2e": {"value": world * step_bytes / (e2e_ms / e2e_steps * 1e-3) / 1e9, "unit": UNIT,
                    "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e2e_steps,
                    "ms_per_step": e2e_ms / e2e_steps,
                    "host_link_gbs": (h2d + d2h) / (e2e_ms / e2e_steps * 1e-3) / 1e9, "host_link_peak": link},
            "gpu_launches": int(launches), "clocks": clocks,
        }
        if not args.no_cpu_baseline and world == 1:
            cores = len(os.sched_getaffinity(0))
            smp = OracleSample(cores, 256)
            b, t, dt = smp.run_pass()
            rec["cpu_baseline"] = {"value": b / dt / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
                                   "sample": smp.describe(1, b, dt), "tokens_per_s_reloaded": t / dt}
        print(json.dumps(rec))
    K.kdn_destroy(ctx)
    if dist is not None:
        dist.destroy_process_group()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="kdn", choices=["kdn", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=4)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-link leg (profiling runs)")
    ap.add_argument("--pool-blocks", type=int, default=0, help="smaller pool for profiler captures (default 16384)")
    ap.add_argument("--chunks", type=int, default=0, help="chunks per store/retrieve batch (default 64)")
    ap.add_argument("--parts", type=int, default=0, help="parts per composed request (default 10)")
    args = ap.parse_args()
    args.warmup = max(3, args.warmup) if args.impl == "kdn" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
