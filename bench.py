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
RAW, INT8, INT4, INT8KC, INT4KC = 0, 1, 2, 3, 4
FALLBACK_HBM_GBS = 6650.0


def bytes_per_elem(codec: int) -> float:
    """Algorithmic bytes per KV element moved by one op: bf16 on the pool side + the chunk side."""
    return {RAW: 4.0, INT8: 2.0 + 1.0 + 4.0 / 64.0, INT4: 2.0 + 0.5 + 4.0 / 64.0,
            INT8KC: 2.0 + 1.0 + 4.0 / 64.0, INT4KC: 2.0 + 0.5 + 4.0 / 64.0}[codec]


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

    def __init__(self, index):
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
NCU_KERNEL_SHA = "87ac4bdc4bfba822"
NCU_SMALL_CASE_BYTES = {"store_raw": (536.904960e6 + 487.936512e6, 8), "retrieve_raw": (536.927232e6 + 490.151680e6, 8), "compose_raw": (268.491776e6 + 222.266368e6, 2), "store_int8": (536.923136e6 + 248.528896e6, 8), "retrieve_int8": (285.255936e6 + 482.943488e6, 8), "compose_int8": (142.667776e6 + 214.036992e6, 2)}


def measured_traffic(op: str, units: float):
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


def make_workload(args, synth):
    """Sizes of one step.  llama3-8b is the benchmark workload; llama3-70b is the batched-retrieve configuration."""
    if args.workload == "llama3-70b":
        shape = synth.LLAMA3_70B
        assign = synth.assign_chunks(32, 4, 16)                       # 32 requests x 4 chunks out of a library of 16
        w = dict(name="llama3-70b", shape=shape, lib=16, chunk_tokens=2048, retr=assign.reshape(-1), part_lib=16,
                 part_tokens=2048, reqs=[list(map(int, row)) for row in assign], suffix=0, exclusive=False,
                 text=("llama3-70b KV (L80 H8 D128 bf16, block_size 16, 16384-block pool): store a library of 16x2048 "
                       "tokens, retrieve 32 requests x 4 chunks (fills the pool), compose the same 32x4 at cumulative "
                       "offsets; raw bf16 and int8-g64, fully fragmented tables"))
    else:
        shape = synth.LLAMA3_8B
        n_chunks, n_parts = args.chunks or N_CHUNKS, args.parts or N_PARTS
        if args.pool_blocks:
            shape = shape.with_(n_blocks=args.pool_blocks)
        w = dict(name="llama3-8b", shape=shape, lib=n_chunks, chunk_tokens=CHUNK_TOKENS, retr=np.arange(n_chunks),
                 part_lib=n_parts, part_tokens=PART_TOKENS, reqs=[list(range(n_parts))], suffix=SUFFIX_TOKENS,
                 exclusive=True, text=WORKLOAD)
        if args.pool_blocks or args.chunks or args.parts:
            w["text"] = "REDUCED (%d chunks, %d parts, %d blocks): not the bench workload" % (n_chunks, n_parts, shape.n_blocks)
    return w


def run_gpu(args) -> None:
    import torch
    from paper_2409_13761_b200 import kdn as K, shard, synth

    rank, world, local = shard.rank_env()
    dist = None
    if world > 1 or "TORCHELASTIC_RUN_ID" in os.environ:        # launched by torch.distributed.run, even with one rank
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    W = make_workload(args, synth)
    shape = W["shape"]
    T, PT, bs = W["chunk_tokens"], W["part_tokens"], shape.block_size
    n_lib, n_retr, n_plib = W["lib"], len(W["retr"]), W["part_lib"]
    n_parts_total = sum(len(r) for r in W["reqs"])

    # ---- inputs (untimed): pool, tables, chunk buffers; every rank has its own copy of the same workload
    k, v = synth.make_pool(shape, dev, seed=synth.SEED_VALUES + rank)
    ctx = K.kdn_create(local)
    desc = K.pool_desc(shape.n_layers, shape.n_kv_heads, shape.head_dim, shape.block_size, shape.n_blocks,
                       [t.data_ptr() for t in k], [t.data_ptr() for t in v])
    pid = K.kdn_pool_register(ctx, desc)
    stream = torch.cuda.Stream(device=dev)
    s = stream.cuda_stream
    bpc, bpp = T // bs, PT // bs
    req_blocks = [(len(r) * PT + W["suffix"]) // bs for r in W["reqs"]]
    taken = np.zeros(0, dtype=np.int64)

    def table(n, seed):
        nonlocal taken
        t = synth.make_table(n, shape.n_blocks, 1, seed, exclude=taken if W["exclusive"] else None)
        if W["exclusive"]:
            taken = np.concatenate([taken, t])
        return torch.from_numpy(t).to(dev)

    d_src = table(n_lib * bpc, synth.SEED_TABLES)                 # where the library chunks are gathered from
    d_dst = table(n_retr * bpc, synth.SEED_TABLES + 1)            # where retrievals land
    d_part_src = table(n_plib * bpp, synth.SEED_TABLES + 2)
    d_req = table(sum(req_blocks), synth.SEED_TABLES + 3)         # all composed requests, back to back
    i32 = 4

    def make_sets(pinned_lib, pinned_retr=(), codecs=(RAW, INT8)):
        """Chunk buffers and the op lists of one step, per codec.  pinned_lib: the whole library lives in page-locked
        host memory; pinned_retr: only these retrievals read a host copy of their chunk."""
        sets = {}
        for codec in codecs:
            cb, pb = K.kdn_chunk_bytes(desc, T, codec), K.kdn_chunk_bytes(desc, PT, codec)
            if pinned_lib:
                chunks = torch.empty(n_lib * cb, dtype=torch.uint8).pin_memory()
                parts = torch.empty(n_plib * pb, dtype=torch.uint8).pin_memory()
                mem = K.KDN_MEM_PINNED_HOST
            else:
                chunks = torch.empty(n_lib * cb, dtype=torch.uint8, device=dev)
                parts = torch.empty(n_plib * pb, dtype=torch.uint8, device=dev)
                mem = K.KDN_MEM_DEVICE
            host_copy = {}
            for r in pinned_retr:
                c = int(W["retr"][r])
                if c not in host_copy:
                    host_copy[c] = torch.empty(cb, dtype=torch.uint8).pin_memory()
            st_ops = [K.XferOp(d_src.data_ptr() + c * bpc * i32, bpc, 0,
                               K.Chunk(chunks.data_ptr() + c * cb, cb, T, codec, mem)) for c in range(n_lib)]
            rt_ops = []
            for r, c in enumerate(W["retr"]):
                c = int(c)
                ch = (K.Chunk(host_copy[c].data_ptr(), cb, T, codec, K.KDN_MEM_PINNED_HOST) if r in pinned_retr
                      else K.Chunk(chunks.data_ptr() + c * cb, cb, T, codec, mem))
                rt_ops.append(K.XferOp(d_dst.data_ptr() + r * bpc * i32, bpc, 0, ch))
            part_store = [K.XferOp(d_part_src.data_ptr() + j * bpp * i32, bpp, 0,
                                   K.Chunk(parts.data_ptr() + j * pb, pb, PT, codec, mem)) for j in range(n_plib)]
            reqs, first = [], 0
            for ids, nb_req in zip(W["reqs"], req_blocks):
                reqs.append(K.ComposeReq(d_req.data_ptr() + first * i32, nb_req,
                                         [K.Chunk(parts.data_ptr() + j * pb, pb, PT, codec, mem, 0) for j in ids],
                                         [i * PT for i in range(len(ids))], shape.rope_theta))
                first += nb_req
            sets[codec] = dict(chunks=chunks, parts=parts, host_copy=host_copy, store=st_ops, retrieve=rt_ops,
                               part_store=part_store, reqs=reqs)
        return sets

    dev_sets = make_sets(False)
    for codec in (RAW, INT8):                      # fill the compose parts once (untimed)
        K.kdn_store(ctx, pid, dev_sets[codec]["part_store"], s)
    assert K.kdn_status_sync(ctx, s) == K.KDN_OK

    names = ["store_raw", "retrieve_raw", "compose_raw", "store_int8", "retrieve_int8", "compose_int8"]
    E = shape.elems_per_token
    tokens_of = {"store": n_lib * T, "retrieve": n_retr * T, "compose": n_parts_total * PT}
    op_tokens = {n: tokens_of[n.split("_")[0]] for n in names}
    op_bytes = {n: op_tokens[n] * E * bytes_per_elem(INT8 if n.endswith("int8") else RAW) for n in names}
    step_bytes = float(sum(op_bytes.values()))
    reload_tokens = sum(op_tokens[n] for n in names if not n.startswith("store"))
    kernel_of = {"store_raw": "kdn_store_kernel<0, 4>", "retrieve_raw": "kdn_retrieve_kernel<0, 4>",
                 "compose_raw": "kdn_compose_kernel<1, 4>", "store_int8": "kdn_store_kernel<2, 4>",
                 "retrieve_int8": "kdn_retrieve_kernel<2, 4>", "compose_int8": "kdn_compose_kernel<3, 4>"}

    def step(sets, events=None, kinds=("store", "retrieve", "compose")):
        i = 0
        for codec in (RAW, INT8):
            for kind in ("store", "retrieve", "compose"):
                if events is not None:
                    events[i].record(stream)
                if kind not in kinds:
                    pass
                elif kind == "store":
                    K.kdn_store(ctx, pid, sets[codec]["store"], s)
                elif kind == "retrieve":
                    K.kdn_retrieve(ctx, pid, sets[codec]["retrieve"], s)
                else:
                    K.kdn_compose(ctx, pid, sets[codec]["reqs"], s)
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
    try:                                            # address the GPU by UUID: indices shift under CUDA_VISIBLE_DEVICES
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(local).uuid)
    except Exception:
        gpu_id = str(local)
    sampler = ClockSampler(gpu_id)
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

    # ---- storage shell: payload checksum over the raw chunk library (read-only stream; not part of `value`)
    lib_buf = dev_sets[RAW]["chunks"]
    csum_out = torch.zeros(1, dtype=torch.int64, device=dev)
    for _ in range(3):
        K.kdn_checksum(local, lib_buf.data_ptr(), lib_buf.numel(), csum_out.data_ptr(), s)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = max(1, min(args.steps, 20))
    a.record(stream)
    for _ in range(reps):
        K.kdn_checksum(local, lib_buf.data_ptr(), lib_buf.numel(), csum_out.data_ptr(), s)
    b.record(stream)
    torch.cuda.synchronize()
    shell_ops = {"checksum_raw_library": {"ms": a.elapsed_time(b) / reps, "bytes": lib_buf.numel(),
                                          "gbs": lib_buf.numel() / (a.elapsed_time(b) / reps * 1e-3) / 1e9}}

    # ---- the int4 codec (a widening beyond the benchmark step; timed on its own, not part of `value`)
    int4_ops = {}
    i4 = make_sets(False, codecs=(INT4,))[INT4]
    K.kdn_store(ctx, pid, i4["part_store"], s)
    for name, fn, arg in (("store_int4", K.kdn_store, i4["store"]), ("retrieve_int4", K.kdn_retrieve, i4["retrieve"]),
                          ("compose_int4", K.kdn_compose, i4["reqs"])):
        for _ in range(3):
            fn(ctx, pid, arg, s)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = max(1, min(args.steps, 20))
        a.record(stream)
        for _ in range(reps):
            fn(ctx, pid, arg, s)
        b.record(stream)
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / reps
        nbytes = tokens_of[name.split("_")[0]] * E * bytes_per_elem(INT4)
        int4_ops[name] = {"ms": ms, "gbs": nbytes / (ms * 1e-3) / 1e9, "tokens_per_s": tokens_of[name.split("_")[0]] / (ms * 1e-3)}
    assert K.kdn_status_sync(ctx, s) == K.KDN_OK
    del i4
    torch.cuda.empty_cache()

    # ---- per-channel key codecs (keys grouped along tokens; timed on their own, not part of `value`), and what they
    # buy: the error of the stored keys, over all channels and over the channels without the x20 outlier gain
    kc_ops = {}

    def key_error_db(codec_id, ops_set):
        """Retrieve chunk 0 and compare layer 0's keys with their source blocks: signal-to-noise ratio in dB.
        Only where source and destination tables are disjoint (the 8B workload)."""
        if not W["exclusive"]:
            return None
        K.kdn_store(ctx, pid, ops_set["store"][:1], s)
        K.kdn_retrieve(ctx, pid, [K.XferOp(d_dst.data_ptr(), bpc, 0, ops_set["store"][0].chunk)], s)
        assert K.kdn_status_sync(ctx, s) == K.KDN_OK
        x = k[0][d_src[:bpc].long()].float().reshape(-1, shape.row_elems)
        y = k[0][d_dst[:bpc].long()].float().reshape(-1, shape.row_elems)
        ordinary = (synth.outlier_gain(shape)[0, 0].reshape(-1) == 1).to(dev)
        snr = lambda a, b: float(10 * torch.log10((a * a).mean() / ((a - b) ** 2).mean()))
        return {"all_channels": snr(x, y), "ordinary_channels": snr(x[:, ordinary], y[:, ordinary])}

    quality = {"int4_g64": key_error_db(INT4, make_sets(False, codecs=(INT4,))[INT4]),
               "int8_g64": key_error_db(INT8, dev_sets[INT8])}
    for codec, cname in ((INT8KC, "int8kc"), (INT4KC, "int4kc")):
        kc = make_sets(False, codecs=(codec,))[codec]
        K.kdn_store(ctx, pid, kc["part_store"], s)
        for name, fn, arg in (("store_" + cname, K.kdn_store, kc["store"]), ("retrieve_" + cname, K.kdn_retrieve, kc["retrieve"]),
                              ("compose_" + cname, K.kdn_compose, kc["reqs"])):
            for _ in range(3):
                fn(ctx, pid, arg, s)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps = max(1, min(args.steps, 20))
            a.record(stream)
            for _ in range(reps):
                fn(ctx, pid, arg, s)
            b.record(stream)
            torch.cuda.synchronize()
            ms = a.elapsed_time(b) / reps
            nbytes = tokens_of[name.split("_")[0]] * E * bytes_per_elem(codec)
            kc_ops[name] = {"ms": ms, "gbs": nbytes / (ms * 1e-3) / 1e9, "tokens_per_s": tokens_of[name.split("_")[0]] / (ms * 1e-3)}
        assert K.kdn_status_sync(ctx, s) == K.KDN_OK
        quality[cname] = key_error_db(codec, kc)
        del kc
        torch.cuda.empty_cache()
    kc_ops["stored_key_snr_db"] = quality

    # ---- keep-lists: every chunk holds a seeded random half of its span's tokens (timed on its own, not in `value`)
    sparse_ops = {}
    rng = np.random.default_rng(synth.SEED_ASSIGN)
    n_keep = T // 2
    keep_np = np.stack([np.sort(rng.choice(T, n_keep, replace=False)) for _ in range(n_lib)]).astype(np.int32)
    d_keep = torch.from_numpy(keep_np).to(dev)
    for codec, cname in ((RAW, "raw"), (INT8, "int8")):
        cb = K.kdn_chunk_bytes(desc, n_keep, codec)
        buf = torch.empty(n_lib * cb, dtype=torch.uint8, device=dev)
        keeps = [d_keep.data_ptr() + c * n_keep * i32 for c in range(n_lib)]
        st_ops = [K.XferOp(d_src.data_ptr() + c * bpc * i32, bpc, 0, K.Chunk(buf.data_ptr() + c * cb, cb, n_keep, codec)) for c in range(n_lib)]
        rt_ops = [K.XferOp(d_dst.data_ptr() + c * bpc * i32, bpc, 0, K.Chunk(buf.data_ptr() + c * cb, cb, n_keep, codec)) for c in range(n_lib)]
        for name, fn, arg in (("store_sparse_" + cname, K.kdn_store_sparse, st_ops), ("retrieve_sparse_" + cname, K.kdn_retrieve_sparse, rt_ops)):
            for _ in range(3):
                fn(ctx, pid, arg, keeps, s)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps = max(1, min(args.steps, 20))
            a.record(stream)
            for _ in range(reps):
                fn(ctx, pid, arg, keeps, s)
            b.record(stream)
            torch.cuda.synchronize()
            ms = a.elapsed_time(b) / reps
            nbytes = n_lib * n_keep * E * bytes_per_elem(codec)
            sparse_ops[name] = {"ms": ms, "gbs": nbytes / (ms * 1e-3) / 1e9, "tokens_per_s": n_lib * n_keep / (ms * 1e-3),
                                "kept": "%d of %d tokens per chunk, seeded random" % (n_keep, T)}
        assert K.kdn_status_sync(ctx, s) == K.KDN_OK
        del buf
    torch.cuda.empty_cache()

    # ---- one chunk per call: what a single retrieve costs (CUDA events around 50 back-to-back calls; not in `value`)
    single_ops = {}
    for codec, cname in ((RAW, "raw"), (INT8, "int8")):
        one = dev_sets[codec]["retrieve"][:1]
        for _ in range(5):
            K.kdn_retrieve(ctx, pid, one, s)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        a.record(stream)
        for _ in range(50):
            K.kdn_retrieve(ctx, pid, one, s)
        b.record(stream)
        host_us = (time.perf_counter() - t0) / 50 * 1e6
        torch.cuda.synchronize()
        us = a.elapsed_time(b) / 50 * 1e3
        nbytes = T * E * bytes_per_elem(codec)
        single_ops["retrieve_one_chunk_" + cname] = {"us_per_call": us, "host_us_per_call": host_us, "gbs": nbytes / us / 1e3,
                                                      "tokens": T, "bytes_moved": nbytes}

    # ---- file-backed chunks: a few chunks of the library written to and read back from one file (wall clock around
    # the call plus the stream sync, since the calling thread does the file I/O; not part of `value`)
    file_ops = {}
    import tempfile
    tmpdir = "/dev/shm" if os.path.isdir("/dev/shm") and os.access("/dev/shm", os.W_OK) else None
    n_file = min(8, n_lib)
    for codec, cname in ((RAW, "raw"), (INT8, "int8")):
        cb = K.kdn_chunk_bytes(desc, T, codec)
        with tempfile.NamedTemporaryFile(dir=tmpdir, prefix="kdn_bench_") as tf:
            fd = tf.fileno()
            st_ops = [K.XferOp(d_src.data_ptr() + c * bpc * i32, bpc, 0, K.Chunk(0, cb, T, codec)) for c in range(n_file)]
            rt_ops = [K.XferOp(d_dst.data_ptr() + c * bpc * i32, bpc, 0, K.Chunk(0, cb, T, codec)) for c in range(n_file)]
            offs = [c * cb for c in range(n_file)]
            for name, fn, arg in (("store_file_" + cname, K.kdn_store_file, st_ops), ("retrieve_file_" + cname, K.kdn_retrieve_file, rt_ops)):
                best = None
                for _ in range(3):
                    torch.cuda.synchronize()
                    t0 = time.perf_counter()
                    fn(ctx, pid, arg, [fd] * n_file, offs, s)
                    assert K.kdn_status_sync(ctx, s) == K.KDN_OK
                    dt = time.perf_counter() - t0
                    best = dt if best is None else min(best, dt)
                file_ops[name] = {"ms": best * 1e3, "file_gbs": n_file * cb / best / 1e9, "file_bytes": n_file * cb,
                                  "where": "tmpfs" if tmpdir else "default temporary directory (page cache)"}

    if args.no_e2e:
        if rank == 0:
            print(json.dumps({"note": "profiling run, not a bench record", "ops_ms": op_ms,
                              "ops_gbs": {n: op_bytes[n] / (op_ms[n] * 1e-3) / 1e9 for n in names}, "int4": int4_ops, "sparse": sparse_ops, "shell": shell_ops, "file": file_ops, "kc": kc_ops}))
        K.kdn_destroy(ctx)
        return

    # ---- end to end: chunks in page-locked host memory, every byte crosses the host link inside the timed region
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    if W["name"] == "llama3-8b":
        # the whole step with the entire library on the host
        del dev_sets
        torch.cuda.empty_cache()
        host_sets = make_sets(True)
        e2e_kinds = ("store", "retrieve", "compose")
        for codec in (RAW, INT8):
            K.kdn_store(ctx, pid, host_sets[codec]["part_store"], s)
        e2e_bytes = step_bytes
        d2h = sum(K.kdn_chunk_bytes(desc, T, c) * n_lib for c in (RAW, INT8)) + 4
        h2d = sum(K.kdn_chunk_bytes(desc, T, c) * n_retr + K.kdn_chunk_bytes(desc, PT, c) * n_parts_total for c in (RAW, INT8))
        e2e_what = "whole step, every chunk in page-locked host memory"
    else:
        # the batched retrieve with four of its chunks on the host, copied in on the side stream while the
        # device-resident retrievals run
        pinned_retr = (5, 50, 90, 120)
        host_sets = make_sets(False, pinned_retr)
        for codec in (RAW, INT8):
            host_sets[codec]["chunks"].copy_(dev_sets[codec]["chunks"])
            for c, hb in host_sets[codec]["host_copy"].items():
                cb = hb.numel()
                hb.copy_(dev_sets[codec]["chunks"][c * cb:(c + 1) * cb])
        e2e_kinds = ("retrieve",)
        e2e_bytes = op_bytes["retrieve_raw"] + op_bytes["retrieve_int8"]
        d2h = 4
        h2d = sum(K.kdn_chunk_bytes(desc, T, c) * len(pinned_retr) for c in (RAW, INT8))
        e2e_what = "batched retrieve, 4 of %d chunks in page-locked host memory (side stream)" % n_retr
    assert K.kdn_status_sync(ctx, s) == K.KDN_OK
    step(host_sets, kinds=e2e_kinds)
    assert K.kdn_status_sync(ctx, s) == K.KDN_OK
    layerwise = None
    if W["name"] != "llama3-8b":
        # layer-wise delivery of one host-resident chunk: when is the first layer range usable, when the last?
        layerwise = {}
        r0 = pinned_retr[0]
        for codec, cname in ((RAW, "raw"), (INT8, "int8")):
            op = [host_sets[codec]["retrieve"][r0]]
            for mode, lps in (("whole", shape.n_layers), ("by_8_layers", 8)):
                evs = [torch.cuda.Event(enable_timing=True) for _ in range(shape.n_layers)]
                t_start = torch.cuda.Event(enable_timing=True)
                for e in evs + [t_start]:
                    e.record(stream)
                torch.cuda.synchronize()
                K.kdn_retrieve_layerwise(ctx, pid, op, lps, s, 0, [e.cuda_event for e in evs])   # warm
                torch.cuda.synchronize()
                t_start.record(stream)
                K.kdn_retrieve_layerwise(ctx, pid, op, lps, s, 0, [e.cuda_event for e in evs])
                torch.cuda.synchronize()
                layerwise["%s_%s" % (cname, mode)] = {"first_layers_ready_ms": t_start.elapsed_time(evs[min(lps, shape.n_layers) - 1]),
                                                      "all_layers_ready_ms": t_start.elapsed_time(evs[-1]),
                                                      "chunk_bytes": K.kdn_chunk_bytes(desc, T, codec)}
        assert K.kdn_status_sync(ctx, s) == K.KDN_OK
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        step(host_sets, kinds=e2e_kinds)
        st = K.kdn_status_sync(ctx, s)            # the step's result is read back: device status + all copies landed
        assert st == K.KDN_OK
    barrier()
    e2e_ms = (time.perf_counter() - t0) * 1e3

    # ---- host-link ceiling, same run: one large pinned cudaMemcpyAsync each way
    probe = torch.empty(1 << 30, dtype=torch.uint8).pin_memory()
    dprobe = torch.empty(1 << 30, dtype=torch.uint8, device=dev)
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
    times = shard.max_over_ranks([elapsed_ms, e2e_ms] + [op_ms[n] for n in names], device=dev)
    elapsed_ms, e2e_ms = float(times[0]), float(times[1])
    op_ms = {n: float(times[2 + i]) for i, n in enumerate(names)}
    if rank == 0:
        peak, peak_kind = measured_hbm_peak()
        ms_per_step = elapsed_ms / args.steps
        value = shard.job_throughput(step_bytes, world, ms_per_step * 1e-3) / 1e9
        ops = {n: {"ms": op_ms[n], "gbs": op_bytes[n] / (op_ms[n] * 1e-3) / 1e9,
                   "frac_of_%s_copy_peak" % peak_kind: op_bytes[n] / (op_ms[n] * 1e-3) / 1e9 / peak,
                   "frac_of_8000": op_bytes[n] / (op_ms[n] * 1e-3) / 1e9 / 8000.0,
                   "tokens_per_s": op_tokens[n] / (op_ms[n] * 1e-3), "kernel": kernel_of[n]} for n in names}
        top = max(names, key=lambda n: op_ms[n])
        units = {"store": n_lib * T / CHUNK_TOKENS, "retrieve": n_retr * T / CHUNK_TOKENS,
                 "compose": n_parts_total * PT / PART_TOKENS}[top.split("_")[0]]
        traffic = measured_traffic(top, units) if shape.elems_per_token == 65536 else None
        rec = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16/int8 (fp32 codec and rotation, fp64 angles)", "data": "synthetic",
            "config": {"workload": W["text"], "l2": "inputs larger than L2 (every op streams >= 1.9 GB once)",
                       "bytes_per_step": step_bytes},
            "tokens_per_s_reloaded": world * reload_tokens / (sum(op_ms[n] for n in names if not n.startswith("store")) * 1e-3),
            "ops": ops, "ops_int4_not_in_value": int4_ops, "ops_keep_list_not_in_value": sparse_ops, "ops_shell_not_in_value": shell_ops,
            "ops_file_not_in_value": file_ops, "ops_single_chunk_not_in_value": single_ops, "ops_per_channel_key_codecs_not_in_value": kc_ops,
            "roofline": {"bound": "hbm", "kernel": kernel_of[top], "op": top, "achieved": ops[top]["gbs"], "peak": peak,
                         "peak_kind": "of " + peak_kind, "unit": "GB/s", "frac": ops[top]["gbs"] / peak,
                         "frac_of_nominal_8000": ops[top]["gbs"] / 8000.0, "traffic": traffic},
            "e2e": {"value": world * e2e_bytes / (e2e_ms / e2e_steps * 1e-3) / 1e9, "unit": UNIT,
                    "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e2e_steps,
                    "ms_per_step": e2e_ms / e2e_steps, "what": e2e_what,
                    "host_link_gbs": (h2d + d2h) / (e2e_ms / e2e_steps * 1e-3) / 1e9, "host_link_peak": link,
                    "layerwise_one_host_chunk": layerwise},
            "gpu_launches": int(launches), "clocks": clocks,
        }
        if not args.no_cpu_baseline and world == 1:
            cores = len(os.sched_getaffinity(0))
            smp = OracleSample(cores, 256)
            b, t, dt = smp.run_pass()
            rec["cpu_baseline"] = {"value": b / dt / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
                                   "sample": smp.describe(1, b, dt), "tokens_per_s_reloaded": t / dt}
            one = OracleSample(1, 128)                       # the same oracle on one core, on a smaller chunk
            b1, t1, dt1 = one.run_pass()
            rec["cpu_baseline"]["one_core"] = {"value": b1 / dt1 / 1e9, "unit": UNIT, "sample": one.describe(1, b1, dt1)}
        print(json.dumps(rec))
    K.kdn_destroy(ctx)
    if dist is not None:
        dist.destroy_process_group()


def run_sweep(args) -> None:
    """GB/s against chunk length on the 8B shape: chunk length 128-8192 tokens x block_size {16, 32} x codec x block-table
    fragmentation (runs of all / 64 / 8 / 1 consecutive physical blocks), store and retrieve, each point batching enough
    distinct chunks to move at least 2 GiB.  Prints one JSON line per point and a final line with all of them."""
    import torch
    from paper_2409_13761_b200 import kdn as K, synth

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    shape16 = synth.LLAMA3_8B
    k, v = synth.make_pool(shape16, dev)
    ctx = K.kdn_create(0)
    pools = {}
    for bs in (16, 32):
        nb = shape16.n_blocks * 16 // bs
        d = K.pool_desc(shape16.n_layers, shape16.n_kv_heads, shape16.head_dim, bs, nb,
                        [t.data_ptr() for t in k], [t.data_ptr() for t in v])           # same memory, other block size
        pools[bs] = (d, K.kdn_pool_register(ctx, d), nb)
    stream = torch.cuda.Stream(device=dev)
    s = stream.cuda_stream
    E = shape16.elems_per_token
    arena = torch.empty((2 << 30) + (256 << 20), dtype=torch.uint8, device=dev)
    peak, peak_kind = measured_hbm_peak()
    points = []
    for bs in (16, 32):
        desc, pid, nb = pools[bs]
        for T in (128, 256, 512, 1024, 2048, 4096, 8192):
            for codec in (RAW, INT8):
                bpe = bytes_per_elem(codec)
                n = max(1, -(-(2 << 30) // int(T * E * bpe)))
                cb = K.kdn_chunk_bytes(desc, T, codec)
                blocks = -(-T // bs)
                for run in (None, 64, 8, 1):
                    r = blocks if run is None else run
                    src = synth.make_table(n * blocks, nb, r, synth.SEED_TABLES)
                    dst = synth.make_table(n * blocks, nb, r, synth.SEED_TABLES + 1, exclude=src)
                    d_src, d_dst = torch.from_numpy(src).to(dev), torch.from_numpy(dst).to(dev)
                    ops = {"store": [K.XferOp(d_src.data_ptr() + i * blocks * 4, blocks, 0,
                                               K.Chunk(arena.data_ptr() + i * cb, cb, T, codec)) for i in range(n)],
                           "retrieve": [K.XferOp(d_dst.data_ptr() + i * blocks * 4, blocks, 0,
                                                  K.Chunk(arena.data_ptr() + i * cb, cb, T, codec)) for i in range(n)]}
                    row = {"block_size": bs, "chunk_tokens": T, "codec": "int8-g64" if codec else "raw", "chunks": n,
                           "run_blocks": "all" if run is None else run, "gib_moved": n * T * E * bpe / 2 ** 30}
                    for name, fn in (("store", K.kdn_store), ("retrieve", K.kdn_retrieve)):
                        for _ in range(3):
                            fn(ctx, pid, ops[name], s)
                        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        a.record(stream)
                        for _ in range(args.steps):
                            fn(ctx, pid, ops[name], s)
                        b.record(stream)
                        torch.cuda.synchronize()
                        ms = a.elapsed_time(b) / args.steps
                        row[name + "_gbs"] = n * T * E * bpe / (ms * 1e-3) / 1e9
                        row[name + "_us"] = ms * 1e3
                    assert K.kdn_status_sync(ctx, s) == K.KDN_OK
                    points.append(row)
                    print(json.dumps(row), flush=True)
    K.kdn_destroy(ctx)
    print(json.dumps({"sweep": "llama3-8b chunk length x block_size x codec x fragmentation", "peak_gbs": peak,
                      "peak_kind": peak_kind, "reps": args.steps, "points": points}))


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="kdn", choices=["kdn", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=4)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-link leg (profiling runs)")
    ap.add_argument("--sweep", action="store_true", help="chunk-length / block-size / codec / fragmentation sweep (1 GPU)")
    ap.add_argument("--workload", default="llama3-8b", choices=["llama3-8b", "llama3-70b"],
                    help="llama3-8b is the benchmark workload; llama3-70b is the batched-retrieve configuration")
    ap.add_argument("--pool-blocks", type=int, default=0, help="smaller pool for profiler captures (default 16384)")
    ap.add_argument("--chunks", type=int, default=0, help="chunks per store/retrieve batch (default 64)")
    ap.add_argument("--parts", type=int, default=0, help="parts per composed request (default 10)")
    args = ap.parse_args()
    args.warmup = max(3, args.warmup) if args.impl == "kdn" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    elif args.sweep:
        run_sweep(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
