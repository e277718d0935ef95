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
The same run then times, outside `value`: both ends of the chunk-length sweep (128- and 8192-token chunks, block_size
16 and 32, both codecs, fully fragmented tables) and the largest configuration, Llama-3-70B-shaped KV (80 layers,
library of 16 x 2048-token chunks, 32 requests x 4 chunks filling the 80 GiB pool, four of the retrievals reading
their chunk from page-locked host memory on a side stream).  `roofline.per_op` lists every op of both workloads as
[GB/s, fraction of the nominal 8000 GB/s], from the median CUDA-event time of the op over the timed steps.
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
RAW, INT8, INT4, INT8KC, INT4KC, INT8TD, INT4TD = 0, 1, 2, 3, 4, 5, 6
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


# DRAM bytes (read + write) per launch from a profiler capture of a reduced case (8 chunks per store/retrieve
# launch, 2 parts per compose launch), scaled by the units a bench launch processes: every byte is touched once,
# so traffic grows in proportion.  Valid only for the kernel source the capture was taken from (its hash).
NCU_KERNEL_SHA = "d1f836c912029be7"
NCU_SMALL_CASE_BYTES = {"store_raw": (536.921088e6 + 488.388608e6, 8), "retrieve_raw": (536.921088e6 + 490.368768e6, 8), "compose_raw": (268.505856e6 + 223.703552e6, 2), "store_int8": (536.938240e6 + 250.342912e6, 8), "retrieve_int8": (285.271040e6 + 482.806528e6, 8), "compose_int8": (142.674944e6 + 213.722368e6, 2)}


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


def make_workload(name, args, synth):
    """Sizes of one step.  llama3-8b is the workload `value` is measured on; llama3-70b is the batched configuration."""
    if name == "llama3-70b":
        shape = synth.LLAMA3_70B
        assign = synth.assign_chunks(32, 4, 16)                       # 32 requests x 4 chunks out of a library of 16
        return dict(name="llama3-70b", shape=shape, lib=16, chunk_tokens=2048, retr=assign.reshape(-1), part_lib=16,
                    part_tokens=2048, reqs=[list(map(int, row)) for row in assign], suffix=0, exclusive=False,
                    text=("llama3-70b KV (L80 H8 D128 bf16, block_size 16, 16384-block pool): store a library of 16x2048 "
                          "tokens, retrieve 32 requests x 4 chunks (fills the pool), compose the same 32x4 at cumulative "
                          "offsets; raw bf16 and int8-g64, fully fragmented tables"))
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


NAMES = ["store_raw", "retrieve_raw", "compose_raw", "store_int8", "retrieve_int8", "compose_int8"]


class Leg:
    """One workload on one GPU: the pool, a library context, block tables, and the op lists of a step."""

    def __init__(self, W, rank, local):
        import torch
        from paper_2409_13761_b200 import kdn as K, synth
        self.torch, self.K, self.synth, self.W = torch, K, synth, W
        self.dev = dev = torch.device("cuda", local)
        self.local = local
        shape = self.shape = W["shape"]
        self.T, self.PT, self.bs = W["chunk_tokens"], W["part_tokens"], shape.block_size
        self.n_lib, self.n_retr, self.n_plib = W["lib"], len(W["retr"]), W["part_lib"]
        self.n_parts_total = sum(len(r) for r in W["reqs"])
        # inputs (untimed): every rank has its own copy of the same workload
        self.k, self.v = synth.make_pool(shape, dev, seed=synth.SEED_VALUES + rank)
        self.ctx = K.kdn_create(local)
        self.desc = K.pool_desc(shape.n_layers, shape.n_kv_heads, shape.head_dim, shape.block_size, shape.n_blocks,
                                [t.data_ptr() for t in self.k], [t.data_ptr() for t in self.v])
        self.pid = K.kdn_pool_register(self.ctx, self.desc)
        self.stream = torch.cuda.Stream(device=dev)
        self.s = self.stream.cuda_stream
        self.bpc, self.bpp = self.T // self.bs, self.PT // self.bs
        self.req_blocks = [(len(r) * self.PT + W["suffix"]) // self.bs for r in W["reqs"]]
        self._taken = np.zeros(0, dtype=np.int64)
        self.d_src = self._table(self.n_lib * self.bpc, synth.SEED_TABLES)        # where the library chunks are gathered from
        self.d_dst = self._table(self.n_retr * self.bpc, synth.SEED_TABLES + 1)   # where retrievals land
        self.d_part_src = self._table(self.n_plib * self.bpp, synth.SEED_TABLES + 2)
        self.d_req = self._table(sum(self.req_blocks), synth.SEED_TABLES + 3)     # all composed requests, back to back
        E = self.E = shape.elems_per_token
        self.tokens_of = {"store": self.n_lib * self.T, "retrieve": self.n_retr * self.T, "compose": self.n_parts_total * self.PT}
        self.op_tokens = {n: self.tokens_of[n.split("_")[0]] for n in NAMES}
        self.op_bytes = {n: self.op_tokens[n] * E * bytes_per_elem(INT8 if n.endswith("int8") else RAW) for n in NAMES}
        self.step_bytes = float(sum(self.op_bytes.values()))
        self.reload_tokens = sum(self.op_tokens[n] for n in NAMES if not n.startswith("store"))
        self.kernels = {}

    def _table(self, n, seed):
        W, shape = self.W, self.shape
        t = self.synth.make_table(n, shape.n_blocks, 1, seed, exclude=self._taken if W["exclusive"] else None)
        if W["exclusive"]:
            self._taken = np.concatenate([self._taken, t])
        return self.torch.from_numpy(t).to(self.dev)

    def make_sets(self, pinned_lib, pinned_retr=(), codecs=(RAW, INT8)):
        """Chunk buffers and the op lists of one step, per codec.  pinned_lib: the whole library lives in page-locked
        host memory; pinned_retr: only these retrievals read a host copy of their chunk."""
        K, torch, W, dev, desc = self.K, self.torch, self.W, self.dev, self.desc
        T, PT, bpc, bpp, i32 = self.T, self.PT, self.bpc, self.bpp, 4
        sets = {}
        for codec in codecs:
            cb, pb = K.kdn_chunk_bytes(desc, T, codec), K.kdn_chunk_bytes(desc, PT, codec)
            if pinned_lib:
                chunks = torch.empty(self.n_lib * cb, dtype=torch.uint8).pin_memory()
                parts = torch.empty(self.n_plib * pb, dtype=torch.uint8).pin_memory()
                mem = K.KDN_MEM_PINNED_HOST
            else:
                chunks = torch.empty(self.n_lib * cb, dtype=torch.uint8, device=dev)
                parts = torch.empty(self.n_plib * pb, dtype=torch.uint8, device=dev)
                mem = K.KDN_MEM_DEVICE
            host_copy = {}
            for r in pinned_retr:
                c = int(W["retr"][r])
                if c not in host_copy:
                    host_copy[c] = torch.empty(cb, dtype=torch.uint8).pin_memory()
            st_ops = [K.XferOp(self.d_src.data_ptr() + c * bpc * i32, bpc, 0,
                               K.Chunk(chunks.data_ptr() + c * cb, cb, T, codec, mem)) for c in range(self.n_lib)]
            rt_ops = []
            for r, c in enumerate(W["retr"]):
                c = int(c)
                ch = (K.Chunk(host_copy[c].data_ptr(), cb, T, codec, K.KDN_MEM_PINNED_HOST) if r in pinned_retr
                      else K.Chunk(chunks.data_ptr() + c * cb, cb, T, codec, mem))
                rt_ops.append(K.XferOp(self.d_dst.data_ptr() + r * bpc * i32, bpc, 0, ch))
            part_store = [K.XferOp(self.d_part_src.data_ptr() + j * bpp * i32, bpp, 0,
                                   K.Chunk(parts.data_ptr() + j * pb, pb, PT, codec, mem)) for j in range(self.n_plib)]
            reqs, first = [], 0
            for ids, nb_req in zip(W["reqs"], self.req_blocks):
                reqs.append(K.ComposeReq(self.d_req.data_ptr() + first * i32, nb_req,
                                         [K.Chunk(parts.data_ptr() + j * pb, pb, PT, codec, mem, 0) for j in ids],
                                         [i * PT for i in range(len(ids))], self.shape.rope_theta))
                first += nb_req
            sets[codec] = dict(chunks=chunks, parts=parts, host_copy=host_copy, store=st_ops, retrieve=rt_ops,
                               part_store=part_store, reqs=reqs)
        return sets

    def fill_parts(self, sets, codecs=(RAW, INT8)):
        for codec in codecs:                      # the compose parts are stored once (untimed)
            self.K.kdn_store(self.ctx, self.pid, sets[codec]["part_store"], self.s)
        self.check()

    def check(self):
        st = self.K.kdn_status_sync(self.ctx, self.s)
        assert st == self.K.KDN_OK, self.K.kdn_strerror(st)

    def step(self, sets, events=None, kinds=("store", "retrieve", "compose"), note_kernels=False):
        K, ctx, pid, s = self.K, self.ctx, self.pid, self.s
        i = 0
        for codec, cname in ((RAW, "raw"), (INT8, "int8")):
            for kind in ("store", "retrieve", "compose"):
                if events is not None:
                    events[i].record(self.stream)
                if kind not in kinds:
                    pass
                elif kind == "store":
                    K.kdn_store(ctx, pid, sets[codec]["store"], s)
                elif kind == "retrieve":
                    K.kdn_retrieve(ctx, pid, sets[codec]["retrieve"], s)
                else:
                    K.kdn_compose(ctx, pid, sets[codec]["reqs"], s)
                if note_kernels and kind in kinds:
                    self.kernels[kind + "_" + cname] = K.kdn_last_launch(ctx)      # the instantiation the library chose
                i += 1
        if events is not None:
            events[i].record(self.stream)

    def time_steps(self, sets, steps, warmup, barrier, sample_clocks=True):
        """`steps` timed passes after `warmup` untimed ones.  Returns total ms, per-op ms (median over the steps of the
        CUDA-event time of each op), kernels launched, clocks."""
        torch, K = self.torch, self.K
        self.step(sets, note_kernels=True)
        for _ in range(max(0, warmup - 1)):
            self.step(sets)
        self.check()
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(len(NAMES) + 1)] for _ in range(steps)]
        try:                                            # address the GPU by UUID: indices shift under CUDA_VISIBLE_DEVICES
            gpu_id = "GPU-" + str(torch.cuda.get_device_properties(self.local).uuid)
        except Exception:
            gpu_id = str(self.local)
        sampler = ClockSampler(gpu_id) if sample_clocks else None
        barrier()
        if sampler:
            sampler.start()
        launches0 = K.kdn_launch_count(self.ctx)
        t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_begin.record(self.stream)
        for it in range(steps):
            self.step(sets, ev[it])
        t_end.record(self.stream)
        barrier()
        clocks = sampler.stop() if sampler else None
        launches = K.kdn_launch_count(self.ctx) - launches0
        self.check()
        per_op = {n: [ev[it][i].elapsed_time(ev[it][i + 1]) for it in range(steps)] for i, n in enumerate(NAMES)}
        op_ms = {n: float(np.median(per_op[n])) for n in NAMES}
        return t_begin.elapsed_time(t_end), op_ms, int(launches), clocks

    def timed(self, fn, reps, warm=3):
        """Mean CUDA-event milliseconds of `reps` back-to-back calls of fn() after `warm` untimed ones."""
        torch = self.torch
        for _ in range(warm):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(self.stream)
        for _ in range(reps):
            fn()
        b.record(self.stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    def close(self):
        self.torch.cuda.synchronize()
        self.K.kdn_destroy(self.ctx)
        self.ctx = None
        self.k = self.v = None
        self.d_src = self.d_dst = self.d_part_src = self.d_req = None
        self.torch.cuda.empty_cache()


EXTRAS = ("shell", "int4", "kc", "sparse", "single", "file", "td")


def extras_8b(leg, dev_sets, reps, which=EXTRAS):
    """Widenings beyond the benchmark step, each timed on its own on the 8B workload (none is part of `value`)."""
    torch, K, synth = leg.torch, leg.K, leg.synth
    ctx, pid, s, dev, desc, shape, W = leg.ctx, leg.pid, leg.s, leg.dev, leg.desc, leg.shape, leg.W
    T, E, bpc, i32, n_lib = leg.T, leg.E, leg.bpc, 4, leg.n_lib
    out = {}

    if "shell" in which:
        # storage shell: payload checksum over the raw chunk library (a read-only stream)
        lib_buf = dev_sets[RAW]["chunks"]
        csum_out = torch.zeros(1, dtype=torch.int64, device=dev)
        ms = leg.timed(lambda: K.kdn_checksum(leg.local, lib_buf.data_ptr(), lib_buf.numel(), csum_out.data_ptr(), s), reps)
        out["ops_shell_not_in_value"] = {"checksum_raw_library": {"ms": ms, "bytes": lib_buf.numel(), "gbs": lib_buf.numel() / (ms * 1e-3) / 1e9}}

    def three(sets, codec, cname, dst):
        leg.K.kdn_store(ctx, pid, sets["part_store"], s)
        for name, fn, arg in (("store_" + cname, K.kdn_store, sets["store"]), ("retrieve_" + cname, K.kdn_retrieve, sets["retrieve"]),
                              ("compose_" + cname, K.kdn_compose, sets["reqs"])):
            ms = leg.timed(lambda: fn(ctx, pid, arg, s), reps)
            tok = leg.tokens_of[name.split("_")[0]]
            nbytes = tok * E * bytes_per_elem(codec)
            dst[name] = {"ms": ms, "gbs": nbytes / (ms * 1e-3) / 1e9, "tokens_per_s": tok / (ms * 1e-3),
                         "kernel": K.kdn_last_launch(ctx)["kernel"]}
        leg.check()

    if "int4" in which:
        # the int4 codec
        int4_ops = {}
        i4 = leg.make_sets(False, codecs=(INT4,))[INT4]
        three(i4, INT4, "int4", int4_ops)
        del i4
        torch.cuda.empty_cache()
        out["ops_int4_not_in_value"] = int4_ops

    if "kc" in which:
        # per-channel key codecs, and what they buy: the error of the stored keys, over all channels and over the channels
        # without the x20 outlier gain
        def key_error_db(ops_set):
            """Retrieve chunk 0 and compare layer 0's keys with their source blocks: signal-to-noise ratio in dB."""
            if not W["exclusive"]:
                return None
            K.kdn_store(ctx, pid, ops_set["store"][:1], s)
            K.kdn_retrieve(ctx, pid, [K.XferOp(leg.d_dst.data_ptr(), bpc, 0, ops_set["store"][0].chunk)], s)
            leg.check()
            x = leg.k[0][leg.d_src[:bpc].long()].float().reshape(-1, shape.row_elems)
            y = leg.k[0][leg.d_dst[:bpc].long()].float().reshape(-1, shape.row_elems)
            ordinary = (synth.outlier_gain(shape)[0, 0].reshape(-1) == 1).to(dev)
            snr = lambda a, b: float(10 * torch.log10((a * a).mean() / ((a - b) ** 2).mean()))
            return {"all_channels": snr(x, y), "ordinary_channels": snr(x[:, ordinary], y[:, ordinary])}

        kc_ops = {}
        i4q = leg.make_sets(False, codecs=(INT4,))[INT4]
        quality = {"int4_g64": key_error_db(i4q), "int8_g64": key_error_db(dev_sets[INT8])}
        del i4q
        torch.cuda.empty_cache()
        for codec, cname in ((INT8KC, "int8kc"), (INT4KC, "int4kc")):
            kc = leg.make_sets(False, codecs=(codec,))[codec]
            three(kc, codec, cname, kc_ops)
            quality[cname] = key_error_db(kc)
            del kc
            torch.cuda.empty_cache()
        kc_ops["stored_key_snr_db"] = quality
        out["ops_per_channel_key_codecs_not_in_value"] = kc_ops

    if "sparse" in which:
        # keep-lists: every chunk holds a seeded random half of its span's tokens
        sparse_ops = {}
        rng = np.random.default_rng(synth.SEED_ASSIGN)
        n_keep = T // 2
        keep_np = np.stack([np.sort(rng.choice(T, n_keep, replace=False)) for _ in range(n_lib)]).astype(np.int32)
        d_keep = torch.from_numpy(keep_np).to(dev)
        for codec, cname in ((RAW, "raw"), (INT8, "int8"), (INT4, "int4")):
            cb = K.kdn_chunk_bytes(desc, n_keep, codec)
            buf = torch.empty(n_lib * cb, dtype=torch.uint8, device=dev)
            keeps = [d_keep.data_ptr() + c * n_keep * i32 for c in range(n_lib)]
            st_ops = [K.XferOp(leg.d_src.data_ptr() + c * bpc * i32, bpc, 0, K.Chunk(buf.data_ptr() + c * cb, cb, n_keep, codec)) for c in range(n_lib)]
            rt_ops = [K.XferOp(leg.d_dst.data_ptr() + c * bpc * i32, bpc, 0, K.Chunk(buf.data_ptr() + c * cb, cb, n_keep, codec)) for c in range(n_lib)]
            for name, fn, arg in (("store_sparse_" + cname, K.kdn_store_sparse, st_ops), ("retrieve_sparse_" + cname, K.kdn_retrieve_sparse, rt_ops)):
                ms = leg.timed(lambda: fn(ctx, pid, arg, keeps, s), reps)
                nbytes = n_lib * n_keep * E * bytes_per_elem(codec)
                sparse_ops[name] = {"ms": ms, "gbs": nbytes / (ms * 1e-3) / 1e9, "tokens_per_s": n_lib * n_keep / (ms * 1e-3),
                                    "kept": "%d of %d tokens per chunk, seeded random" % (n_keep, T)}
            leg.check()
            del buf
        torch.cuda.empty_cache()
        out["ops_keep_list_not_in_value"] = sparse_ops

    if "single" in which:
        # one chunk per call: what a single retrieve costs (CUDA events around back-to-back calls, each call another chunk
        # of the library into its own blocks, so nothing is served from L2)
        single_ops = {}
        for codec, cname in ((RAW, "raw"), (INT8, "int8")):
            ones = [K.xfer_array([op]) for op in dev_sets[codec]["retrieve"]]
            n_calls = 2 * len(ones)
            for arr in ones[:8]:
                K.lib.kdn_retrieve(ctx, pid, arr, 1, s, 0)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            a.record(leg.stream)
            for i in range(n_calls):
                K.lib.kdn_retrieve(ctx, pid, ones[i % len(ones)], 1, s, 0)
            b.record(leg.stream)
            host_us = (time.perf_counter() - t0) / n_calls * 1e6
            torch.cuda.synchronize()
            leg.check()
            us = a.elapsed_time(b) / n_calls * 1e3
            nbytes = T * E * bytes_per_elem(codec)
            single_ops["retrieve_one_chunk_" + cname] = {"us_per_call": us, "host_us_per_call_through_ctypes": host_us, "gbs": nbytes / us / 1e3,
                                                          "frac_of_8000": nbytes / us / 1e3 / 8000.0, "tokens": T, "bytes_moved": nbytes}
        # the same call from plain C (the example program: one raw chunk, 200 calls): host time per call without Python
        try:
            import re
            import tempfile
            from paper_2409_13761_b200 import build as _build
            with tempfile.TemporaryDirectory() as td_:
                exe = _build.build_example("single_chunk", td_)
                res = subprocess.run([exe], capture_output=True, text=True, timeout=300, env=_build.example_env())
            m = re.search(r"ok host_us=([0-9.]+) device_us=([0-9.]+) gbs=([0-9.]+)", res.stdout)
            single_ops["from_c_example"] = ({"host_us_per_call": float(m.group(1)), "device_us_per_call": float(m.group(2)),
                                             "gbs": float(m.group(3)), "note": "one chunk re-read every call (half of it may sit in L2)"}
                                            if m else {"error": (res.stdout + res.stderr)[-300:]})
        except Exception as exc:                      # no C compiler on the box: the ctypes figure stands alone
            single_ops["from_c_example"] = {"error": str(exc)[:200]}
        out["ops_single_chunk_not_in_value"] = single_ops

    if "file" in which:
        # file-backed chunks: a few chunks of the library written to and read back from files (wall clock around the call
        # plus the stream sync, since the calling thread does the file I/O)
        file_ops = {}
        import tempfile
        tmpdir = "/dev/shm" if os.path.isdir("/dev/shm") and os.access("/dev/shm", os.W_OK) else None
        n_file = min(8, n_lib)
        for codec, cname in ((RAW, "raw"), (INT8, "int8")):
            cb = K.kdn_chunk_bytes(desc, T, codec)
            st_ops = [K.XferOp(leg.d_src.data_ptr() + c * bpc * i32, bpc, 0, K.Chunk(0, cb, T, codec)) for c in range(n_file)]
            rt_ops = [K.XferOp(leg.d_dst.data_ptr() + c * bpc * i32, bpc, 0, K.Chunk(0, cb, T, codec)) for c in range(n_file)]
            for layout in ("one_file", "file_per_chunk"):
                files = [tempfile.NamedTemporaryFile(dir=tmpdir, prefix="kdn_bench_") for _ in range(1 if layout == "one_file" else n_file)]
                try:
                    fds = [files[0].fileno()] * n_file if layout == "one_file" else [f.fileno() for f in files]
                    offs = [c * cb for c in range(n_file)] if layout == "one_file" else [0] * n_file
                    for name, fn, arg in (("store_file_" + cname, K.kdn_store_file, st_ops), ("retrieve_file_" + cname, K.kdn_retrieve_file, rt_ops)):
                        best = None
                        for _ in range(3):
                            torch.cuda.synchronize()
                            t0 = time.perf_counter()
                            fn(ctx, pid, arg, fds, offs, s)
                            leg.check()
                            dt = time.perf_counter() - t0
                            best = dt if best is None else min(best, dt)
                        file_ops[name + "_" + layout] = {"ms": best * 1e3, "file_gbs": n_file * cb / best / 1e9, "file_bytes": n_file * cb,
                                                         "where": "tmpfs" if tmpdir else "default temporary directory (page cache)"}
                finally:
                    for f in files:
                        f.close()
        out["ops_file_not_in_value"] = file_ops

    if "td" in which:
        # token-delta Rice codecs (quantise, then entropy-code along tokens): how small the chunks get and how fast they are
        # stored and decoded, on inputs whose neighbouring tokens correlate with coefficient rho (rho = 0: the ordinary
        # uncorrelated input, the worst case for this codec).  This leg rewrites the library's source blocks, so it runs last.
        td = {}
        n_td = min(n_lib, 32)
        bf16_bytes = n_td * T * E * 2
        for rho in (0.0, 0.9, 0.99):
            for c in range(n_td):
                x = synth.correlated_tokens(shape, T, rho, synth.SEED_VALUES + 100 + c, dev)
                synth.place_tokens(leg.k, leg.v, leg.d_src[c * bpc:(c + 1) * bpc].cpu().numpy(), 0, x)
            del x
            for codec, cname in ((INT8TD, "int8td"), (INT4TD, "int4td")):
                cb = K.kdn_chunk_bytes(desc, T, codec)
                lay = K.kdn_td_layout(desc, T, codec)
                buf = torch.empty(n_td * cb, dtype=torch.uint8, device=dev)
                st_ops = [K.XferOp(leg.d_src.data_ptr() + c * bpc * i32, bpc, 0, K.Chunk(buf.data_ptr() + c * cb, cb, T, codec)) for c in range(n_td)]
                rt_ops = [K.XferOp(leg.d_dst.data_ptr() + c * bpc * i32, bpc, 0, K.Chunk(buf.data_ptr() + c * cb, cb, T, codec)) for c in range(n_td)]
                reqs = [K.ComposeReq(leg.d_dst.data_ptr() + c * bpc * i32, bpc, [K.Chunk(buf.data_ptr() + c * cb, cb, T, codec, K.KDN_MEM_DEVICE, 4096)],
                                     [0], shape.rope_theta) for c in range(n_td)]
                ms_store = leg.timed(lambda: K.kdn_store(ctx, pid, st_ops, s), min(reps, 5), warm=2)
                leg.check()
                used = sum(int(buf[c * cb + 8 * lay["segments"]:c * cb + 8 * lay["segments"] + 8].view(torch.int64).item()) for c in range(n_td))
                ms_retr = leg.timed(lambda: K.kdn_retrieve(ctx, pid, rt_ops, s), min(reps, 5), warm=2)
                ms_comp = leg.timed(lambda: K.kdn_compose(ctx, pid, reqs, s), min(reps, 5), warm=2)
                leg.check()
                # delivery from page-locked host memory: the chunks packed back to back, only their bytes in use (wall
                # clock around the call and the status read, as in the end-to-end leg)
                useds = [int(buf[c * cb + 8 * lay["segments"]:c * cb + 8 * lay["segments"] + 8].view(torch.int64).item()) for c in range(n_td)]
                starts = np.concatenate([[0], np.cumsum([(u + 255) // 256 * 256 for u in useds])])
                arena = torch.empty(int(starts[-1]), dtype=torch.uint8).pin_memory()
                for c in range(n_td):
                    arena[int(starts[c]):int(starts[c]) + useds[c]].copy_(buf[c * cb:c * cb + useds[c]])
                torch.cuda.synchronize()
                h_ops = [K.XferOp(leg.d_dst.data_ptr() + c * bpc * i32, bpc, 0,
                                  K.Chunk(arena.data_ptr() + int(starts[c]), cb, T, codec, K.KDN_MEM_PINNED_HOST)) for c in range(n_td)]
                K.kdn_retrieve(ctx, pid, h_ops, s)
                leg.check()
                t0 = time.perf_counter()
                for _ in range(3):
                    K.kdn_retrieve(ctx, pid, h_ops, s)
                    leg.check()
                host_ms = (time.perf_counter() - t0) / 3 * 1e3
                del arena
                moved = used + bf16_bytes                        # coded bytes on the chunk side, bf16 on the pool side
                td["%s_rho_%s" % (cname, rho)] = {
                    "chunk_bytes_used": used, "bits_per_element": 8.0 * used / (n_td * T * E), "smaller_than_bf16_by": bf16_bytes / used,
                    "store_ms": ms_store, "store_gbs": moved / (ms_store * 1e-3) / 1e9,
                    "retrieve_ms": ms_retr, "retrieve_gbs": moved / (ms_retr * 1e-3) / 1e9, "retrieve_tokens_per_s": n_td * T / (ms_retr * 1e-3),
                    "compose_ms": ms_comp, "compose_gbs": moved / (ms_comp * 1e-3) / 1e9,
                    "retrieve_frac_of_8000": moved / (ms_retr * 1e-3) / 1e9 / 8000.0,
                    # the decoder is bound by the integer ALU pipe, not by HBM: 148 SMs x 4 schedulers x one ALU-pipe
                    # instruction every other cycle x 1.965 GHz x 32 lanes, at about 20 such operations per symbol
                    "retrieve_roofline": {"bound": "alu", "unit": "symbols/s", "achieved": n_td * T * E / (ms_retr * 1e-3),
                                          "peak": 148 * 4 * 0.5 * 1.965e9 * 32 / 20.0,
                                          "frac": n_td * T * E / (ms_retr * 1e-3) / (148 * 4 * 0.5 * 1.965e9 * 32 / 20.0)},
                    "from_host_ms": host_ms, "from_host_link_gbs": used / (host_ms * 1e-3) / 1e9,
                    "from_host_bf16_gbs_delivered": bf16_bytes / (host_ms * 1e-3) / 1e9}
                del buf
                if codec == INT4TD:
                    # the same chunks holding only half of their tokens (a seeded random keep-list per chunk): token dropping
                    # and coding together, against the bf16 bytes of the whole span
                    n_keep = T // 2
                    rng = np.random.default_rng(11)
                    keep = torch.from_numpy(np.stack([np.sort(rng.choice(T, n_keep, replace=False)) for _ in range(n_td)]).astype(np.int32)).to(dev)
                    keeps = [keep.data_ptr() + c * n_keep * i32 for c in range(n_td)]
                    cbk = K.kdn_chunk_bytes(desc, n_keep, codec)
                    layk = K.kdn_td_layout(desc, n_keep, codec)
                    bufk = torch.empty(n_td * cbk, dtype=torch.uint8, device=dev)
                    sk = [K.XferOp(leg.d_src.data_ptr() + c * bpc * i32, bpc, 0, K.Chunk(bufk.data_ptr() + c * cbk, cbk, n_keep, codec)) for c in range(n_td)]
                    rk = [K.XferOp(leg.d_dst.data_ptr() + c * bpc * i32, bpc, 0, K.Chunk(bufk.data_ptr() + c * cbk, cbk, n_keep, codec)) for c in range(n_td)]
                    ms_sk = leg.timed(lambda: K.kdn_store_sparse(ctx, pid, sk, keeps, s), min(reps, 5), warm=2)
                    leg.check()
                    usedk = sum(int(bufk[c * cbk + 8 * layk["segments"]:c * cbk + 8 * layk["segments"] + 8].view(torch.int64).item()) for c in range(n_td))
                    ms_rk = leg.timed(lambda: K.kdn_retrieve_sparse(ctx, pid, rk, keeps, s), min(reps, 5), warm=2)
                    leg.check()
                    td["%s_rho_%s" % (cname, rho)]["half_of_the_tokens_kept"] = {
                        "chunk_bytes_used": usedk, "bits_per_kept_element": 8.0 * usedk / (n_td * n_keep * E),
                        "smaller_than_bf16_of_the_whole_span_by": bf16_bytes / usedk,
                        "store_ms": ms_sk, "retrieve_ms": ms_rk, "retrieve_kept_tokens_per_s": n_td * n_keep / (ms_rk * 1e-3),
                        "retrieve_gbs": (usedk + bf16_bytes / 2) / (ms_rk * 1e-3) / 1e9}
                    del bufk, keep
            torch.cuda.empty_cache()
        td["what"] = ("%d chunks x %d tokens; GB/s counts the bytes the chunks use plus the bf16 bytes on the pool side; "
                      "rho = correlation of neighbouring tokens in the synthetic input" % (n_td, T))
        out["ops_token_delta_rice_not_in_value"] = td
    return out


def sweep_extract(leg, reps):
    """Both ends of the chunk-length sweep on the 8B pool: chunk length {128, 8192} x block_size {16, 32} x codec {raw,
    int8-g64}, fully fragmented tables, store and retrieve, each point batching enough distinct chunks to move >= 2 GiB."""
    torch, K, synth = leg.torch, leg.K, leg.synth
    shape, dev, s = leg.shape, leg.dev, leg.s
    E = leg.E
    arena = torch.empty((2 << 30) + (256 << 20), dtype=torch.uint8, device=dev)
    points = []
    for bs in (16, 32):
        nb = shape.n_blocks * shape.block_size // bs
        desc = K.pool_desc(shape.n_layers, shape.n_kv_heads, shape.head_dim, bs, nb,
                           [t.data_ptr() for t in leg.k], [t.data_ptr() for t in leg.v])      # same memory, other block size
        pid = K.kdn_pool_register(leg.ctx, desc)
        for T in (128, 8192):
            for codec in (RAW, INT8):
                bpe = bytes_per_elem(codec)
                n = max(1, -(-(2 << 30) // int(T * E * bpe)))
                cb = K.kdn_chunk_bytes(desc, T, codec)
                blocks = -(-T // bs)
                src = synth.make_table(n * blocks, nb, 1, synth.SEED_TABLES)
                dst = synth.make_table(n * blocks, nb, 1, synth.SEED_TABLES + 1, exclude=src)
                d_src, d_dst = torch.from_numpy(src).to(dev), torch.from_numpy(dst).to(dev)
                row = {"block_size": bs, "chunk_tokens": T, "codec": "int8" if codec else "raw", "chunks": n}
                for name, fn, tab in (("store", K.kdn_store, d_src), ("retrieve", K.kdn_retrieve, d_dst)):
                    ops = [K.XferOp(tab.data_ptr() + i * blocks * 4, blocks, 0, K.Chunk(arena.data_ptr() + i * cb, cb, T, codec)) for i in range(n)]
                    ms = leg.timed(lambda: fn(leg.ctx, pid, ops, s), reps)
                    row[name + "_gbs"] = n * T * E * bpe / (ms * 1e-3) / 1e9
                leg.check()
                points.append(row)
    del arena
    torch.cuda.empty_cache()
    return points


def shard_extract(leg, reps):
    """The 8B pool seen by one rank of a head-sharded (tensor-parallel) engine: 4, 2 and 1 of the 8 KV heads per GPU,
    i.e. token rows of 512, 256 and 128 elements and pool blocks of 16, 8 and 4 KiB (the same memory registered with
    fewer heads and more blocks).  Store, retrieve and compose of 512-token chunks, raw and int8-g64, fully fragmented
    tables, enough chunks per launch to move 2 GiB on the pool side."""
    torch, K, synth = leg.torch, leg.K, leg.synth
    shape, dev, s = leg.shape, leg.dev, leg.s
    arena = torch.empty((2 << 30) + (256 << 20), dtype=torch.uint8, device=dev)
    T, bs, points = 512, shape.block_size, []
    for heads in (4, 2, 1):
        k = shape.n_kv_heads // heads
        nb = shape.n_blocks * k
        E = shape.elems_per_token // k
        desc = K.pool_desc(shape.n_layers, heads, shape.head_dim, bs, nb,
                           [t.data_ptr() for t in leg.k], [t.data_ptr() for t in leg.v])      # same memory, narrower rows
        pid = K.kdn_pool_register(leg.ctx, desc)
        blocks = T // bs
        for codec in (RAW, INT8):
            bpe = bytes_per_elem(codec)
            n = max(1, (2 << 30) // int(T * E * 2))
            cb = K.kdn_chunk_bytes(desc, T, codec)
            src = synth.make_table(n * blocks, nb, 1, synth.SEED_TABLES)
            dst = synth.make_table(n * blocks, nb, 1, synth.SEED_TABLES + 1, exclude=src)
            d_src, d_dst = torch.from_numpy(src).to(dev), torch.from_numpy(dst).to(dev)
            chunk = lambda i, base=0: K.Chunk(arena.data_ptr() + i * cb, cb, T, codec, K.KDN_MEM_DEVICE, base)
            st = [K.XferOp(d_src.data_ptr() + i * blocks * 4, blocks, 0, chunk(i)) for i in range(n)]
            rt = [K.XferOp(d_dst.data_ptr() + i * blocks * 4, blocks, 0, chunk(i)) for i in range(n)]
            rq = [K.ComposeReq(d_dst.data_ptr(), n * blocks, [chunk(i) for i in range(n)], [i * T for i in range(n)], shape.rope_theta)]
            row = {"kv_heads_per_gpu": heads, "row_elems": heads * shape.head_dim, "block_bytes": bs * heads * shape.head_dim * 2,
                   "codec": "int8" if codec else "raw", "chunks": n}
            for name, fn in (("store", lambda: K.kdn_store(leg.ctx, pid, st, s)), ("retrieve", lambda: K.kdn_retrieve(leg.ctx, pid, rt, s)),
                             ("compose", lambda: K.kdn_compose(leg.ctx, pid, rq, s))):
                for _ in range(8):                        # every ring slot of the context has sized its rotation table
                    fn()
                ms = leg.timed(fn, reps)
                row[name + "_gbs"] = n * T * E * bpe / (ms * 1e-3) / 1e9
            leg.check()
            points.append(row)
    del arena
    torch.cuda.empty_cache()
    return points


def host_link_peak(torch, stream, dev):
    """Host-link ceiling of this run: one 1 GiB pinned cudaMemcpyAsync each way, best of 5."""
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
    return link


def leg_70b(args, rank, local, barrier, steps):
    """The batched 70B configuration: device-resident timing of the six ops, then the batched retrieve with four of its
    chunks in page-locked host memory (side stream) and the layer-wise delivery of one host-resident chunk."""
    import torch
    from paper_2409_13761_b200 import synth
    W = make_workload("llama3-70b", args, synth)
    leg = Leg(W, rank, local)
    K = leg.K
    dev_sets = leg.make_sets(False)
    leg.fill_parts(dev_sets)
    elapsed_ms, op_ms, launches, _ = leg.time_steps(dev_sets, steps, 3, barrier, sample_clocks=False)
    res = {"workload": W["text"], "steps": steps, "ms_per_step": elapsed_ms / steps, "op_ms": op_ms,
           "op_bytes": dict(leg.op_bytes), "op_tokens": dict(leg.op_tokens), "kernels": dict(leg.kernels),
           "launches": launches, "step_bytes": leg.step_bytes}
    if not args.no_e2e:
        pinned_retr = (5, 50, 90, 120)
        host_sets = leg.make_sets(False, pinned_retr)
        for codec in (RAW, INT8):
            host_sets[codec]["chunks"].copy_(dev_sets[codec]["chunks"])
            for c, hb in host_sets[codec]["host_copy"].items():
                cb = hb.numel()
                hb.copy_(dev_sets[codec]["chunks"][c * cb:(c + 1) * cb])
        del dev_sets
        torch.cuda.empty_cache()
        leg.step(host_sets, kinds=("retrieve",))
        leg.check()
        n_e2e = max(1, min(steps, args.e2e_steps))
        barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            leg.step(host_sets, kinds=("retrieve",))
            leg.check()                                   # the step's result is read back: device status + all copies landed
        barrier()
        ms = (time.perf_counter() - t0) * 1e3 / n_e2e
        h2d = sum(K.kdn_chunk_bytes(leg.desc, leg.T, c) * len(pinned_retr) for c in (RAW, INT8))
        res["side_stream"] = {"what": "batched retrieve, 4 of %d chunks in page-locked host memory (side stream), raw + int8" % leg.n_retr,
                              "ms_per_step": ms, "h2d_bytes_per_step": int(h2d), "host_link_gbs": h2d / (ms * 1e-3) / 1e9,
                              "gbs": (leg.op_bytes["retrieve_raw"] + leg.op_bytes["retrieve_int8"]) / (ms * 1e-3) / 1e9}
        # layer-wise delivery of one host-resident chunk: when is the first layer range usable, when the last?
        layerwise = {}
        shape = leg.shape
        for codec, cname in ((RAW, "raw"), (INT8, "int8")):
            op = [host_sets[codec]["retrieve"][pinned_retr[0]]]
            for mode, lps in (("whole", shape.n_layers), ("by_8_layers", 8)):
                evs = [torch.cuda.Event(enable_timing=True) for _ in range(shape.n_layers)]
                t_start = torch.cuda.Event(enable_timing=True)
                for e in evs + [t_start]:
                    e.record(leg.stream)
                torch.cuda.synchronize()
                K.kdn_retrieve_layerwise(leg.ctx, leg.pid, op, lps, leg.s, 0, [e.cuda_event for e in evs])   # warm
                torch.cuda.synchronize()
                t_start.record(leg.stream)
                K.kdn_retrieve_layerwise(leg.ctx, leg.pid, op, lps, leg.s, 0, [e.cuda_event for e in evs])
                torch.cuda.synchronize()
                layerwise["%s_%s" % (cname, mode)] = {"first_layers_ready_ms": t_start.elapsed_time(evs[min(lps, shape.n_layers) - 1]),
                                                      "all_layers_ready_ms": t_start.elapsed_time(evs[-1]),
                                                      "chunk_bytes": K.kdn_chunk_bytes(leg.desc, leg.T, codec)}
        leg.check()
        res["layerwise_one_host_chunk"] = layerwise
        res["host_link_peak"] = host_link_peak(torch, leg.stream, leg.dev)
        del host_sets
    leg.close()
    return res


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

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    if args.workload == "llama3-70b":                           # the 70B configuration on its own
        res = leg_70b(args, rank, local, barrier, args.steps)
        if rank == 0:
            peak, peak_kind = measured_hbm_peak()
            res["op_gbs"] = {n: res["op_bytes"][n] / (res["op_ms"][n] * 1e-3) / 1e9 for n in NAMES}
            res["note"] = "llama3-70b leg on its own, not a bench record"
            print(json.dumps(res))
        if dist is not None:
            dist.destroy_process_group()
        return

    W = make_workload("llama3-8b", args, synth)
    leg = Leg(W, rank, local)
    shape, T, PT, E = leg.shape, leg.T, leg.PT, leg.E
    ctx, pid, s, desc = leg.ctx, leg.pid, leg.s, leg.desc
    n_lib, n_retr, n_parts_total = leg.n_lib, leg.n_retr, leg.n_parts_total
    dev_sets = leg.make_sets(False)
    leg.fill_parts(dev_sets)

    # ---- device-resident timing: the step `value` is measured on
    elapsed_ms, op_ms, launches, clocks = leg.time_steps(dev_sets, args.steps, args.warmup, barrier)
    reps = max(1, min(args.steps, 20))
    extras = extras_8b(leg, dev_sets, reps, tuple(x for x in args.extras.split(",") if x))
    full = not (args.pool_blocks or args.chunks or args.parts)
    sweep_points = sweep_extract(leg, min(reps, 10)) if full and not args.no_sweep else None
    shard_points = shard_extract(leg, min(reps, 10)) if full and not args.no_sweep else None

    if args.no_e2e:
        if rank == 0:
            print(json.dumps({"note": "profiling run, not a bench record", "ops_ms": op_ms, "kernels": leg.kernels,
                              "ops_gbs": {n: leg.op_bytes[n] / (op_ms[n] * 1e-3) / 1e9 for n in NAMES}, **extras,
                              "sweep_extract": sweep_points, "head_sharded_shapes": shard_points}))
        leg.close()
        return

    # ---- end to end: the whole step with the entire library in page-locked host memory, so every byte crosses the
    # host link inside the timed region
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    del dev_sets
    torch.cuda.empty_cache()
    host_sets = leg.make_sets(True)
    leg.fill_parts(host_sets)
    d2h = sum(K.kdn_chunk_bytes(desc, T, c) * n_lib for c in (RAW, INT8)) + 4
    h2d = sum(K.kdn_chunk_bytes(desc, T, c) * n_retr + K.kdn_chunk_bytes(desc, PT, c) * n_parts_total for c in (RAW, INT8))
    leg.step(host_sets)
    leg.check()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        leg.step(host_sets)
        leg.check()                                   # the step's result is read back: device status + all copies landed
    barrier()
    e2e_ms = (time.perf_counter() - t0) * 1e3
    link = host_link_peak(torch, leg.stream, dev)
    step_bytes, op_bytes, op_tokens, reload_tokens, kernels = leg.step_bytes, leg.op_bytes, leg.op_tokens, leg.reload_tokens, dict(leg.kernels)
    del host_sets
    leg.close()

    # ---- the largest configuration: the batched 70B workload (not part of `value`; its per-op figures go into the
    # roofline table below)
    r70 = None
    if full and not args.no_70b:
        r70 = leg_70b(args, rank, local, barrier, max(3, min(args.steps, 10)))

    # ---- reduce over ranks (max time), print on rank 0
    vals = [elapsed_ms, e2e_ms] + [op_ms[n] for n in NAMES] + ([r70["op_ms"][n] for n in NAMES] if r70 else [])
    times = shard.max_over_ranks(vals, device=dev)
    elapsed_ms, e2e_ms = float(times[0]), float(times[1])
    op_ms = {n: float(times[2 + i]) for i, n in enumerate(NAMES)}
    if r70:
        r70["op_ms"] = {n: float(times[2 + len(NAMES) + i]) for i, n in enumerate(NAMES)}
    if rank == 0:
        peak, peak_kind = measured_hbm_peak()
        ms_per_step = elapsed_ms / args.steps
        value = shard.job_throughput(step_bytes, world, ms_per_step * 1e-3) / 1e9
        gbs = {n: op_bytes[n] / (op_ms[n] * 1e-3) / 1e9 for n in NAMES}
        ops = {n: {"ms": op_ms[n], "gbs": gbs[n], "frac_of_%s_copy_peak" % peak_kind: gbs[n] / peak, "frac_of_8000": gbs[n] / 8000.0,
                   "tokens_per_s": op_tokens[n] / (op_ms[n] * 1e-3), "kernel": kernels[n]["kernel"], "launch": kernels[n]} for n in NAMES}
        top = max(NAMES, key=lambda n: op_ms[n])
        units = {"store": n_lib * T / CHUNK_TOKENS, "retrieve": n_retr * T / CHUNK_TOKENS,
                 "compose": n_parts_total * PT / PART_TOKENS}[top.split("_")[0]]
        traffic = measured_traffic(top, units) if shape.elems_per_token == 65536 else None
        # every op of both workloads as [GB/s, fraction of the nominal 8000 GB/s]; median CUDA-event time per op
        per_op = {"fractions": "of the nominal 8000 GB/s; GB/s = algorithmic bytes / median CUDA-event time of the op",
                  "8b": {n: [round(gbs[n], 1), round(gbs[n] / 8000.0, 4)] for n in NAMES}}
        if r70:
            g70 = {n: r70["op_bytes"][n] / (r70["op_ms"][n] * 1e-3) / 1e9 for n in NAMES}
            per_op["70b"] = {n: [round(g70[n], 1), round(g70[n] / 8000.0, 4)] for n in NAMES}
            per_op["70b_ms_per_step"] = round(r70["ms_per_step"], 3)
            if "side_stream" in r70:
                per_op["70b_host_link"] = [round(r70["side_stream"]["host_link_gbs"], 2), round(r70["host_link_peak"]["h2d_gbs"], 2)]
        if sweep_points:
            for name in ("store", "retrieve"):
                worst = min(sweep_points, key=lambda p: p[name + "_gbs"])
                per_op["sweep_min_" + name] = [round(worst[name + "_gbs"], 1), round(worst[name + "_gbs"] / 8000.0, 4),
                                               "T=%d bs=%d %s" % (worst["chunk_tokens"], worst["block_size"], worst["codec"])]
            per_op["sweep_points"] = len(sweep_points)
        if shard_points:
            for name in ("store", "retrieve", "compose"):
                worst = min(shard_points, key=lambda p: p[name + "_gbs"])
                per_op["head_shard_min_" + name] = [round(worst[name + "_gbs"], 1), round(worst[name + "_gbs"] / 8000.0, 4),
                                                    "%d of 8 KV heads per GPU, %s" % (worst["kv_heads_per_gpu"], worst["codec"])]
        # the widenings of the 8B leg in the same compact form (outside `value`)
        wide = {}
        for key in ("ops_int4_not_in_value", "ops_per_channel_key_codecs_not_in_value", "ops_keep_list_not_in_value"):
            for n, v in (extras.get(key) or {}).items():
                if isinstance(v, dict) and "gbs" in v:
                    wide[n] = [round(v["gbs"], 1), round(v["gbs"] / 8000.0, 4)]
        for n, v in (extras.get("ops_single_chunk_not_in_value") or {}).items():
            if isinstance(v, dict) and "gbs" in v:
                wide[n] = [round(v["gbs"], 1), round(v["gbs"] / 8000.0, 4)]
        for n, v in (extras.get("ops_token_delta_rice_not_in_value") or {}).items():
            if isinstance(v, dict) and "retrieve_gbs" in v:
                wide["td_" + n] = {"x_smaller": round(v["smaller_than_bf16_by"], 2), "store": round(v["store_gbs"], 1),
                                   "retrieve": round(v["retrieve_gbs"], 1), "compose": round(v["compose_gbs"], 1),
                                   "host_bf16_gbs": round(v["from_host_bf16_gbs_delivered"], 1)}
                if "half_of_the_tokens_kept" in v:
                    wide["td_" + n]["x_smaller_with_half_of_the_tokens_kept"] = round(v["half_of_the_tokens_kept"]["smaller_than_bf16_of_the_whole_span_by"], 2)
        if wide:
            per_op["widenings_8b"] = wide
        frac = gbs[top] / peak
        rec = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16/int8 (fp32 codec and rotation, fp64 angles)", "data": "synthetic",
            "config": {"workload": W["text"], "also_measured": "llama3-70b batch (32x4x2048 tokens), sweep ends and head-sharded pool shapes: roofline.per_op",
                       "l2": "inputs larger than L2 (every op streams >= 1.9 GB once)", "bytes_per_step": step_bytes},
            "tokens_per_s_reloaded": world * reload_tokens / (sum(op_ms[n] for n in NAMES if not n.startswith("store")) * 1e-3),
            "roofline": {"bound": "hbm", "kernel": kernels[top]["kernel"], "op": top, "achieved": gbs[top], "peak": peak,
                         "peak_kind": "of " + peak_kind, "unit": "GB/s", "frac": frac,
                         "frac_of_nominal_8000": gbs[top] / 8000.0, "traffic": traffic,
                         "traffic_source": ("profiler capture of a reduced case, scaled by the units of a launch" if traffic is not None
                                            else "none: the kernels changed since the profiler capture (algorithmic bytes only)"),
                         "note": ("the measured peak is a plain device copy; bulk-copy streams run a little above it, so this "
                                  "fraction says 'at the copy ceiling', not 'headroom left'" if frac > 1.0 else None),
                         "per_op": per_op},
            "e2e": {"value": world * step_bytes / (e2e_ms / e2e_steps * 1e-3) / 1e9, "unit": UNIT,
                    "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e2e_steps,
                    "ms_per_step": e2e_ms / e2e_steps, "what": "whole step, every chunk in page-locked host memory",
                    "host_link_gbs": (h2d + d2h) / (e2e_ms / e2e_steps * 1e-3) / 1e9, "host_link_peak": link,
                    "llama3_70b_side_stream": (r70 or {}).get("side_stream"),
                    "layerwise_one_host_chunk": (r70 or {}).get("layerwise_one_host_chunk")},
            "gpu_launches": int(launches), "clocks": clocks,
            "ops": ops, "llama3_70b": ({"workload": r70["workload"], "steps": r70["steps"], "ms_per_step": r70["ms_per_step"],
                                        "op_ms": r70["op_ms"], "kernels": {n: r70["kernels"][n]["kernel"] for n in NAMES},
                                        "launches": r70["launches"]} if r70 else None),
            "sweep_extract": sweep_points, "head_sharded_shapes": shard_points, **extras,
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
    ap.add_argument("--extras", default=",".join(EXTRAS), help="which of the legs outside `value` to run: " + ",".join(EXTRAS))
    ap.add_argument("--no-70b", action="store_true", help="skip the llama3-70b leg of the default run")
    ap.add_argument("--no-sweep", action="store_true", help="skip the sweep extract of the default run")
    ap.add_argument("--sweep", action="store_true", help="chunk-length / block-size / codec / fragmentation sweep (1 GPU)")
    ap.add_argument("--workload", default="llama3-8b", choices=["llama3-8b", "llama3-70b"],
                    help="llama3-8b (default): the benchmark run, which also times the 70B batch and the sweep ends; "
                         "llama3-70b: only the batched 70B configuration")
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
