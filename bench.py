#!/usr/bin/env python
"""Benchmark of reuse-prefill on B200: one step = one percache_prefill call of the workload.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4_50] [--impl reference] [--no-table]

Prints ONE JSON line.  `value` is context tokens per second (prompt tokens served / time) with inputs
resident in HBM; `e2e` is the same through host buffers (pinned input hidden states copied in, output
rows copied out inside the timed call).  Between steps the chunks the call stored are dropped again
(host-only bookkeeping, untimed) so that every step sees the same cache state.  The line is about the named
workload (default: the long context with half of its chunks cached); at one GPU its key `workloads` also holds one
compact record for each of the other workloads (time per step, tokens/s, per-kernel-class throughput and fraction
of the measured peak, clocks, and the oracle's extrapolated throughput on the host).

With N > 1 every rank runs an independent replica of the workload on its own GPU (the path does not
shard: no collective), and the aggregate is N x tokens / slowest rank.

`--impl reference` times the CPU oracle (the plain definition the tests check against) on the host.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2601_11553_b200 import workloads as wl

METRIC = "reuse_prefill_tokens_per_s"
UNIT = "tokens/s"
DEFAULT_WORKLOAD = "cfg4_50"      # the largest single-GPU workload that uses both halves of the method
TABLE_WORKLOADS = ("cfg0", "cfg1", "cfg2", "cfg3", "cfg4_100", "cfg4_90", "cfg4_50", "cfg4_0", "prefix_cfg1", "paper_cfg1")


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "tflops_burst": d["bf16_tflops"],
                "tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "tflops_burst": 1590.0, "tflops_sustained": 1400.0, "source": "fallback"}


# --------------------------------------------------------------------------- DRAM traffic from ncu
def kernel_traffic(kernel: str, workload: str):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch, taken once under ncu (profiles/dram_traffic.json).

    An entry is only used while the kernel's source file still has the hash recorded with it."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(path):
        return None
    ent = json.load(open(path)).get(workload, {}).get(kernel)
    if not ent:
        return None
    src = os.path.join(ROOT, "paper_2601_11553_b200", "csrc", ent["source"])
    if not os.path.exists(src) or hashlib.sha256(open(src, "rb").read()).hexdigest() != ent["sha256"]:
        return None
    return ent["dram_bytes_per_launch"]


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.02):
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thr = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._dev = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._dev, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None
            return
        self._thr = threading.Thread(target=self._run, daemon=True)
        self._thr.start()

    def _run(self):
        nv = self._nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
                 "hw_power_brake_slowdown": 0x80, "sync_boost": 0x10}
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._dev, nv.NVML_CLOCK_SM)))
                r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._dev))
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop.set()
        if self._thr:
            self._thr.join(timeout=2)
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------- workload accounting
def flops_per_step(w: wl.Workload, new_rows: int, visible_pairs: int):
    s = w.shape
    per_row = {"qkv": 2 * s.d_model * (s.q_dim + 2 * s.kv_dim), "oproj": 2 * s.q_dim * s.d_model,
               "gateup": 2 * s.d_model * 2 * s.d_ffn, "down": 2 * s.d_ffn * s.d_model}
    # paper-faithful mode: only the projections skip the cached rows, the rest of every block runs on all rows
    rows = {k: (w.total_tokens if (w.paper_mode and k != "qkv") else new_rows) for k in per_row}
    out = {k: v * rows[k] * s.n_layers for k, v in per_row.items()}
    out["attn"] = 4 * s.n_q_heads * s.head_dim * visible_pairs * s.n_layers
    return out


# --------------------------------------------------------------------------- CPU oracle leg
def _oracle_cores():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        return os.cpu_count() or 1


def _oracle_model(shape, weights):
    from oracle import reuse_prefill as orc
    return orc.Model(n_layers=shape.n_layers, d_model=shape.d_model, n_q_heads=shape.n_q_heads,
                     n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, d_ffn=shape.d_ffn,
                     rope_theta=shape.rope_theta, rms_eps=shape.rms_eps, layers=weights)


def oracle_sample(w: wl.Workload, n_layers_sample: int):
    """Time the oracle on the first `n_layers_sample` layers of the workload's model (all rows, same prompts)."""
    from oracle import reuse_prefill as orc
    cores = _oracle_cores()
    shape = wl.ModelShape(n_layers=n_layers_sample, **{k: getattr(w.shape, k) for k in
                                                       ("d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn")})
    model = _oracle_model(shape, wl.make_weights(shape, w.seed))
    store = orc.Store()
    ids_lens = {c: l for p in w.prompts for c, l in zip(p.chunk_ids, p.chunk_len)}
    for c in w.cached_ids:     # cached content: seeded integer values (timing does not depend on them)
        n = ids_lens[c]
        k = np.stack([orc.bf16_bits_to_f64(wl.pool_kv_values(w.seed, c, 0, l, n, shape.kv_dim)) for l in range(shape.n_layers)])
        v = np.stack([orc.bf16_bits_to_f64(wl.pool_kv_values(w.seed, c, 1, l, n, shape.kv_dim)) for l in range(shape.n_layers)])
        store.put(c, k.reshape(shape.n_layers, n, shape.n_kv_heads, shape.head_dim),
                  v.reshape(shape.n_layers, n, shape.n_kv_heads, shape.head_dim))
    cached = set(w.cached_ids)
    prompts = []
    for p in w.prompts:
        hid = [None if c in cached else orc.bf16_bits_to_f64(h) for c, h in zip(p.chunk_ids, p.chunk_hidden)] \
            if p.chunk_hidden else [None] * len(p.chunk_ids)
        prompts.append(orc.Prompt(list(p.chunk_ids), list(p.chunk_len), hid, orc.bf16_bits_to_f64(p.query_hidden)))

    def step():
        t0 = time.perf_counter()
        orc.reuse_prefill(model, store, prompts, commit=False)
        return time.perf_counter() - t0
    return step, cores


class OracleBlockSample:
    """The oracle on a bounded sample of a large workload: block 0 of the model through oracle.block_rows, which
    forms K and V for every new row of a prompt (they are the block's context) and the rest of the block for a few
    sampled rows.  Timed at two sample sizes; the time is linear in the number of sampled rows, so the line through
    the two points gives the time of the block for all rows, and the depth multiplies it.  For a batch only every
    `prompt_stride`-th prompt is timed.  Cached K/V are zeros here (their values do not change the time)."""

    def __init__(self, w: wl.Workload, rows=(32, 288), max_prompts: int = 8):
        from oracle import reuse_prefill as orc
        self.orc, self.w, self.rows = orc, w, rows
        shape1 = wl.ModelShape(n_layers=1, **{k: getattr(w.shape, k) for k in
                                              ("d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn")})
        self.model = _oracle_model(shape1, wl.make_weights(shape1, w.seed))
        self.cores = _oracle_cores()
        cached = set(w.cached_ids)
        stride = max(1, -(-len(w.prompts) // max_prompts))
        self.stride = stride
        self.cases = []
        hkv, hd = w.shape.n_kv_heads, w.shape.head_dim
        for p in w.prompts[::stride]:
            new, segs, xs, start = [], [], [], 0
            for i, (c, n) in enumerate(zip(p.chunk_ids, p.chunk_len)):
                if c in cached:
                    z = np.zeros((n, hkv, hd))
                    segs.append((start, z, z))
                else:
                    new.append(np.arange(start, start + n))
                    xs.append(orc.bf16_bits_to_f64(p.chunk_hidden[i]))
                start += n
            new.append(np.arange(start, start + p.n_query))
            xs.append(orc.bf16_bits_to_f64(p.query_hidden))
            self.cases.append((np.concatenate(xs), np.concatenate(new), start + p.n_query, segs))
        self.m_sampled = sum(c[0].shape[0] for c in self.cases)
        self.slope = None

    def _time(self, n_rows: int) -> float:
        t0 = time.perf_counter()
        for x, new, T, segs in self.cases:
            m = x.shape[0]
            rows = np.unique(np.linspace(0, m - 1, min(n_rows, m)).astype(np.int64))
            self.orc.block_rows(self.model, 0, x, new, T, segs, rows)
        return time.perf_counter() - t0

    def step(self) -> float:
        """One bounded sample; returns the extrapolated seconds of one whole step of the workload."""
        if self.slope is None:
            self._time(self.rows[0])    # untimed first pass: pages in the weights and the BLAS threads
        t_small = self._time(self.rows[0])
        if self.slope is None:          # seconds per sampled row and case, measured once
            t_big = self._time(self.rows[1])
            self.slope = max(0.0, (t_big - t_small) / (self.rows[1] - self.rows[0]) / len(self.cases))
        per_case_rows = [c[0].shape[0] for c in self.cases]
        full_block = t_small + self.slope * sum(max(0, m - min(self.rows[0], m)) for m in per_case_rows)
        return full_block * (self.w.new_rows() / max(self.m_sampled, 1)) * self.w.shape.n_layers

    def describe(self, t_step: float) -> str:
        return (f"block 0 of {self.w.shape.n_layers} of {self.w.name} via oracle.block_rows: K/V of all new rows of "
                f"{len(self.cases)} of {len(self.w.prompts)} prompts + {self.rows[0]} (and once {self.rows[1]}) sampled "
                f"rows each; linear in rows -> all {self.w.new_rows()} new rows, x {self.w.shape.n_layers} blocks: "
                f"EXTRAPOLATED to {t_step:.0f} s per step")


def cpu_baseline_for(w: wl.Workload):
    """Oracle tokens/s on the host for workload w: a whole run where it takes seconds, else the bounded block sample."""
    tokens = w.total_tokens
    if w.paper_mode:                                       # the paper-faithful oracle, a few layers of the real call
        from oracle import paper_mode as pm
        from oracle import reuse_prefill as orc
        n_sample = max(1, min(w.shape.n_layers, 2))
        shape = wl.ModelShape(n_layers=n_sample, **{k: getattr(w.shape, k) for k in
                                                    ("d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn")})
        model = _oracle_model(shape, wl.make_weights(shape, w.seed))
        store = pm.PaperStore()
        p = w.prompts[0]
        f64 = orc.bf16_bits_to_f64
        n_c = len(w.cached_ids)
        pm.paper_prefill(model, store, [pm.PaperPrompt(list(p.chunk_ids[:n_c]), list(p.chunk_len[:n_c]),
                                                       [f64(h) for h in p.chunk_hidden[:n_c]], np.zeros((0, shape.d_model)))])
        t0 = time.perf_counter()
        pm.paper_prefill(model, store, [pm.PaperPrompt(list(p.chunk_ids), list(p.chunk_len), [f64(h) for h in p.chunk_hidden],
                                                       f64(p.query_hidden))], commit=False)
        t = time.perf_counter() - t0
        scale = w.shape.n_layers / n_sample
        return {"value": tokens / (t * scale), "unit": UNIT, "cores": _oracle_cores(), "kind": "oracle",
                "sample": f"first {n_sample} of {w.shape.n_layers} layers of {w.name} through oracle.paper_mode, all rows, "
                          f"one call ({t:.1f} s), time x {scale:g}", "extrapolated": True}
    if w.new_rows() * w.shape.n_layers <= 3000:            # cfg0-sized: the whole call
        step, cores = oracle_sample(w, w.shape.n_layers)
        t = step()
        return {"value": tokens / t, "unit": UNIT, "cores": cores, "kind": "oracle",
                "sample": f"the whole {w.name} call ({t:.2f} s)", "extrapolated": False}
    if w.new_rows() <= 1500 and len(w.prompts) == 1:       # cfg1-sized: a few layers of the real call
        n_sample = max(1, min(w.shape.n_layers, 4))
        step, cores = oracle_sample(w, n_sample)
        t = step()
        scale = w.shape.n_layers / n_sample
        return {"value": tokens / (t * scale), "unit": UNIT, "cores": cores, "kind": "oracle",
                "sample": f"first {n_sample} of {w.shape.n_layers} layers of {w.name}, all new rows, one call "
                          f"({t:.1f} s), time x {scale:g}", "extrapolated": True}
    smp = OracleBlockSample(w)
    t = smp.step()
    return {"value": tokens / t, "unit": UNIT, "cores": smp.cores, "kind": "oracle", "sample": smp.describe(t),
            "extrapolated": True}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = wl.by_name(args.workload)
    big = not (w.new_rows() <= 1500 and len(w.prompts) == 1)
    if big:
        smp = OracleBlockSample(w)
        step = smp.step
        cores = smp.cores
    else:
        n_sample = 1
        raw, cores = oracle_sample(w, n_sample)
        step = lambda: raw() * (w.shape.n_layers / n_sample)
    for _ in range(min(args.warmup, 1)):
        step()
    times = [step() for _ in range(args.steps)]
    ms = 1000.0 * float(np.mean(times))
    value = w.total_tokens / (ms / 1000.0)
    sample = smp.describe(ms / 1000.0) if big else \
        f"layer 0 of {w.shape.n_layers} of {w.name} (all prompts, all new rows), time x {w.shape.n_layers:g}"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": {"workload": w.name, "description": w.description,
                                                        "tokens_per_step": w.total_tokens},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# --------------------------------------------------------------------------- replicas
def max_over_ranks(values, dist, device):
    """Every rank runs an independent replica; the job's time is the slowest rank's (max over ranks of each value)."""
    if dist is None:
        return [float(v) for v in values]
    import torch
    t = torch.tensor([float(v) for v in values], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def aggregate_tokens_per_s(world: int, tokens_per_step: int, steps: int, total_ms: float) -> float:
    """Whole-job throughput of `world` replicas that each did `steps` steps within total_ms (the slowest rank's)."""
    return world * tokens_per_step * steps / (total_ms / 1000.0)


def replica_launch_command(args, port: int):
    """The command that starts one rank per GPU of this node when bench.py itself is asked for N > 1 GPUs without a
    launcher around it (no WORLD_SIZE in the environment)."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)]
    return cmd + list(args.forward)


# --------------------------------------------------------------------------- GPU leg
KERNEL_OF = {"attn": "umma_attention_kernel", "gather": "gather_rerope_kernel"}


def pick_peak(peaks, timed_s: float, reasons):
    """The tensor-core denominator for a run: the sustained figure when the timed region lasts seconds or the power
    cap was active while it ran, else the burst figure."""
    if timed_s >= 1.0 or "sw_power_cap" in reasons:
        return peaks["tflops_sustained"], "sustained"
    return peaks["tflops_burst"], "burst"


class Bench:
    """One model on one GPU and the workloads that run on it."""

    def __init__(self, shape, seed, workloads, local, torch, pcb):
        self.torch, self.pcb = torch, pcb
        self.paper_mode = workloads[0].paper_mode
        self.dev = torch.device("cuda", local)
        self.local = local
        self.shape = shape
        self.stream = torch.cuda.current_stream(self.dev)
        weights_np = wl.make_weights(shape, seed)
        weights = [{k: torch.from_numpy(v.view(np.int16)).to(self.dev).view(torch.bfloat16) for k, v in lw.items()}
                   for lw in weights_np]
        ids_lens = {}
        for w in workloads:
            ids_lens.update({c: l for p in w.prompts for c, l in zip(p.chunk_ids, p.chunk_len)})
        self.ids_lens = ids_lens
        max_tokens = max(w.total_tokens for w in workloads)
        self.h = pcb.PerCache(n_layers=shape.n_layers, d_model=shape.d_model, n_q_heads=shape.n_q_heads,
                              n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, d_ffn=shape.d_ffn, weights=weights,
                              pool_pages=2 * sum((l + 15) // 16 for l in ids_lens.values()) + 256,
                              max_prompt_tokens=max(p.n_total for w in workloads for p in w.prompts),
                              max_batch_prompts=max(len(w.prompts) for w in workloads),
                              max_batch_ctx_tokens=max_tokens, max_batch_new_rows=max_tokens, device=local,
                              stream=self.stream.cuda_stream, flags=pcb.FLAG_PAPER_MODE if self.paper_mode else 0)

    def close(self):
        self.h.close()

    def set_cache_state(self, w: wl.Workload):
        """Exactly w.cached_ids of the workload's chunks are stored: missing ones are produced (a prefill of the chunk
        alone through the library itself, or the seeded integer pool), others of the workload are dropped."""
        h, pcb = self.h, self.pcb
        cached = set(w.cached_ids)
        if w.match_prefix:       # the cached chain: one prefill of exactly that prefix, stored under its path keys
            p = w.prompts[0]
            n = len(w.cached_ids)
            if n and h.has_chunk(pcb.path_key(list(p.chunk_ids[:n]))) is None:
                h.prefill([pcb.PromptSpec(list(p.chunk_ids[:n]), list(p.chunk_len[:n]), list(p.chunk_hidden[:n]), None, 0,
                                          match_prefix=True)])
            return
        for c in w.cached_ids:
            if h.has_chunk(c) is not None:
                continue
            if w.cache_source == "integer_pool":
                h.put_chunk_synthetic(c, self.ids_lens[c], w.seed)
            else:
                hid = wl.chunk_hidden_for(w.seed, c, self.ids_lens[c], self.shape.d_model)
                h.prefill([pcb.PromptSpec([c], [self.ids_lens[c]], [hid], None, 0)])
        for p in w.prompts:
            for c in p.chunk_ids:
                if c not in cached and h.has_chunk(c) is not None:
                    h.drop_chunk(c)

    def measure(self, w: wl.Workload, steps: int, warmup: int, flags: int, full: bool, barrier, dist):
        """Times the workload.  full: also the end-to-end pass through host buffers."""
        torch, pcb, h, dev, stream, shape = self.torch, self.pcb, self.h, self.dev, self.stream, self.shape
        self.set_cache_state(w)
        cached = set(w.cached_ids)
        missed = sorted({c for p in w.prompts for c in p.chunk_ids if c not in cached})
        if w.match_prefix:       # nodes are stored under the key of their path
            missed = [pcb.path_key(list(p.chunk_ids[: i + 1])) for p in w.prompts
                      for i, c in enumerate(p.chunk_ids) if c not in cached]

        def to_dev(a):
            return torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)

        def to_pinned(a):
            return torch.from_numpy(a.view(np.int16)).pin_memory().view(torch.bfloat16)

        def specs(conv):
            out = []
            for p in w.prompts:
                hid = [None if (c in cached and not w.paper_mode) else conv(hh)
                       for c, hh in zip(p.chunk_ids, p.chunk_hidden)] if p.chunk_hidden else None
                out.append(pcb.PromptSpec(list(p.chunk_ids), list(p.chunk_len), hid, conv(p.query_hidden), p.n_query,
                                          match_prefix=w.match_prefix))
            return out

        n_new = [p.n_query + sum(l for c, l in zip(p.chunk_ids, p.chunk_len) if c not in cached) for p in w.prompts]
        if w.paper_mode:         # every row of the prompt comes back
            n_new = [p.n_total for p in w.prompts]
        specs_dev = specs(to_dev)
        out_dev = [torch.empty((n, shape.d_model), dtype=torch.float32, device=dev) for n in n_new]

        def timed(spec_list, outs, n):
            ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
            phases = {k: 0.0 for k in pcb.PHASES}
            launches = {k: 0 for k in pcb.PHASES}
            dev_us, st = 0.0, None
            for i in range(n):
                ev[i][0].record(stream)
                h.prefill(spec_list, out=outs)
                ev[i][1].record(stream)
                st = h.stats()
                dev_us += st["device_us"]
                for k in pcb.PHASES:
                    phases[k] += st["phase_us"][k]
                    launches[k] += st["phase_launches"][k]
                for c in missed:           # host-only bookkeeping, untimed: every step starts from the same cache state
                    h.drop_chunk(c)
            torch.cuda.synchronize(dev)
            return [a.elapsed_time(b) for a, b in ev], phases, launches, dev_us, st

        h.set_flags(flags)
        timed(specs_dev, out_dev, max(warmup, 3))
        sampler = ClockSampler(self.local)
        barrier()
        sampler.start()
        ms, _, launches, dev_us, st = timed(specs_dev, out_dev, steps)
        barrier()
        clocks = sampler.stop()
        total_ms = float(sum(ms))
        # the same steps with CUDA events around every kernel class (a separate pass: the events cost a few per cent)
        h.set_flags(flags | pcb.FLAG_PHASE_TIMING)
        timed(specs_dev, out_dev, 2)
        ph_steps = steps if full else max(2, min(steps, 5))
        ms_ph, phases, launches_ph, _, _ = timed(specs_dev, out_dev, ph_steps)
        h.set_flags(flags)
        e2e_ms = None
        if full:     # end to end: pinned host hidden states in, host rows out, inside the timed call
            specs_host = specs(to_pinned)
            out_host = [torch.empty((n, shape.d_model), dtype=torch.float32).pin_memory() for n in n_new]
            timed(specs_host, out_host, 3)
            barrier()
            ms_e2e, _, _, _, _ = timed(specs_host, out_host, steps)
            barrier()
            e2e_ms = float(sum(ms_e2e))
        vals = max_over_ranks([total_ms] + ([e2e_ms] if full else []), dist, dev)
        total_ms = vals[0]
        if full:
            e2e_ms = vals[1]

        peaks = load_peaks()
        new_rows = int(st["new_rows"])
        fl = flops_per_step(w, new_rows, int(st["attn_visible_pairs"]))
        gather_bytes = int(st["hit_tokens"]) * shape.n_layers * shape.kv_dim * 2 * 2 * 2
        tensor_peak, which_peak = pick_peak(peaks, total_ms / 1000.0, clocks["reasons"])
        weight_bytes_layer = shape.params_per_layer * 2
        per_phase = {}
        for k in ("qkv", "attn", "oproj", "gateup", "down"):
            n = launches_ph[k]
            if n:
                us = phases[k] / n
                tf = fl[k] / shape.n_layers / us / 1e6
                per_phase[k] = {"us_per_launch": us, "launches_per_step": n // ph_steps, "tflops": tf,
                                "frac_of_tensor_peak": tf / tensor_peak}
        if launches_ph["gather"]:
            us = phases["gather"] / launches_ph["gather"]
            gbs = gather_bytes / us / 1e3
            per_phase["gather"] = {"us_per_launch": us, "launches_per_step": 1, "gbs": gbs,
                                   "frac_of_hbm_peak": gbs / peaks["hbm_gbs"]}
        if launches_ph["norm"]:
            per_phase["norm"] = {"us_per_launch": phases["norm"] / launches_ph["norm"],
                                 "launches_per_step": launches_ph["norm"] // ph_steps}
        return {"w": w, "ms": ms, "total_ms": total_ms, "e2e_ms": e2e_ms, "clocks": clocks, "st": st, "phases": phases,
                "launches": launches, "launches_ph": launches_ph, "per_phase": per_phase, "fl": fl, "dev_us": dev_us,
                "gather_bytes": gather_bytes, "new_rows": new_rows, "tensor_peak": tensor_peak, "which_peak": which_peak,
                "peaks": peaks, "ms_ph": ms_ph, "ph_steps": ph_steps, "weight_bytes_layer": weight_bytes_layer}


def table_row(r, world, steps):
    """Compact record of one workload for the per-workload table."""
    w = r["w"]
    row = {"workload": w.name, "form": "gather-free" if r["st"].get("gather_free") else "gather",
           "ms_per_step": r["total_ms"] / steps,
           "tokens_per_s": aggregate_tokens_per_s(world, w.total_tokens, steps, r["total_ms"]),
           "new_rows": r["new_rows"], "hit_tokens": int(r["st"]["hit_tokens"]), "steps": steps,
           "tensor_peak": {"tflops": r["tensor_peak"], "which": r["which_peak"]},
           "clocks": {k: r["clocks"][k] for k in ("sm_mhz", "sm_max_mhz", "reasons")}, "kernels": {}}
    for k, v in r["per_phase"].items():
        if "tflops" in v:
            row["kernels"][k] = {"tflops": round(v["tflops"], 1), "frac": round(v["frac_of_tensor_peak"], 3)}
        elif "gbs" in v:
            row["kernels"][k] = {"gbs": round(v["gbs"], 1), "frac": round(v["frac_of_hbm_peak"], 3)}
    # whole step against the roofline of its algorithmic work: tensor flops, or weight + gather bytes when the call has
    # too few rows to reach the tensor roof (the ridge is ~210 flops per byte)
    flops = sum(r["fl"].values())
    t_s = r["total_ms"] / steps / 1000.0
    row["step_tflops"] = flops / t_s / 1e12
    row["step_frac_of_tensor_peak"] = row["step_tflops"] / r["tensor_peak"]
    hbm_bytes = r["weight_bytes_layer"] * w.shape.n_layers + r["gather_bytes"]
    row["step_hbm_floor_ms"] = hbm_bytes / r["peaks"]["hbm_gbs"] / 1e6
    return row


def run_gpu(args):
    import torch
    from paper_2601_11553_b200 import percache as pcb

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)

    def barrier():
        torch.cuda.synchronize(dev)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    main_w = wl.by_name(args.workload)
    if args.layers > 0:
        main_w.shape = wl.ModelShape(n_layers=args.layers, **{k: getattr(main_w.shape, k) for k in
                                                              ("d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn")})
        main_w.name += f"@{args.layers}layers"
        args.no_table = True
    # Workloads that share the main one's model run on the same handle (the long-context sweep: one model, four hit
    # rates with nested hit sets, run from the fullest cache to the emptiest); the others get a handle each.
    table_names = [] if (args.no_table or world > 1) else [n for n in TABLE_WORKLOADS if n != main_w.name]
    groups = {}
    for name in [main_w.name] + table_names:
        w = main_w if name == main_w.name else wl.by_name(name)
        groups.setdefault((w.seed, w.shape, w.paper_mode), []).append(w)
    rows, main = [], None
    for (seed, shape, _paper), ws in groups.items():
        ws.sort(key=lambda w: -len(w.cached_ids))
        b = Bench(shape, seed, ws, local, torch, pcb)
        for w in ws:
            is_main = w.name == main_w.name
            steps = args.steps if is_main else max(3, min(args.steps, 10))
            r = b.measure(w, steps, args.warmup, args.flags, is_main, barrier, dist)
            if is_main:
                main = r
            elif rank == 0:
                row = table_row(r, world, steps)
                if not args.no_cpu_baseline:
                    row["cpu_baseline"] = cpu_baseline_for(w)
                rows.append(row)
            # a workload the library serves in its gather-free form is also timed in the form that assembles the
            # context, so that the fetch kernel's bandwidth is on record for it
            if r["st"].get("gather_free") and not w.paper_mode and not (args.flags & pcb.FLAG_ALWAYS_GATHER) and not args.no_table:
                r2 = b.measure(w, max(3, min(steps, 10)), args.warmup, args.flags | pcb.FLAG_ALWAYS_GATHER, False, barrier, dist)
                if rank == 0:
                    row2 = table_row(r2, world, max(3, min(steps, 10)))
                    row2["workload"] = w.name + " (gather form)"
                    rows.append(row2)
        b.close()
        del b
        torch.cuda.empty_cache()
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank != 0:
        return

    r, w, shape = main, main_w, main_w.shape
    peaks, st, per_phase, fl = r["peaks"], r["st"], r["per_phase"], r["fl"]
    tokens, new_rows = w.total_tokens, r["new_rows"]
    value = aggregate_tokens_per_s(world, tokens, args.steps, r["total_ms"])
    e2e_value = aggregate_tokens_per_s(world, tokens, args.steps, r["e2e_ms"])
    dom = max(("qkv", "attn", "oproj", "gateup", "down", "gather"), key=lambda k: r["phases"][k])
    if dom == "gather":
        roof = {"bound": "hbm", "achieved": per_phase[dom]["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": per_phase[dom]["gbs"] / peaks["hbm_gbs"], "traffic": None, "kernel": "gather_rerope_kernel",
                "peak_source": f"{peaks['source']} copy bandwidth"}
    else:
        roof = {"bound": "tensor", "achieved": per_phase[dom]["tflops"], "peak": r["tensor_peak"], "unit": "TFLOP/s",
                "frac": per_phase[dom]["tflops"] / r["tensor_peak"], "traffic": None,
                "kernel": KERNEL_OF.get(dom, f"umma_gemm_kernel<{dom}>"),
                "peak_source": f"{peaks['source']} {r['which_peak']} bf16 figure x 1.0 (nominal fp16 : bf16 ratio); "
                               f"{r['which_peak']} because the timed region lasted {r['total_ms'] / 1000.0:.2f} s with "
                               f"throttle reasons {r['clocks']['reasons']}"}
    roof["share_of_step"] = r["phases"][dom] / max(sum(r["phases"].values()), 1e-9)
    traffic = kernel_traffic(roof["kernel"], w.name)
    roof["traffic"] = traffic
    roof["traffic_source"] = None if traffic is None else "stored: one ncu capture of this kernel (profiles/dram_traffic.json), not this run"
    roof["algorithmic_per_launch"] = r["gather_bytes"] if dom == "gather" else fl[dom] / shape.n_layers
    kernels_per_step = (sum(r["launches"][k] for k in pcb.PHASES if k != "io") // args.steps) + 1
    main_row = table_row(r, world, args.steps)

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline_for(w)
        main_row["cpu_baseline"] = cpu

    print(json.dumps({
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": r["total_ms"] / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16", "data": "synthetic",
        "config": {"workload": w.name, "form": "gather-free" if st.get("gather_free") else "gather",
                   "reduced_depth": args.layers > 0, "description": w.description,
                   "tokens_per_step": tokens, "new_rows_per_step": new_rows, "hit_tokens_per_step": int(st["hit_tokens"]),
                   "prompts_per_step": len(w.prompts), "ms_per_prompt": r["total_ms"] / args.steps / len(w.prompts),
                   "computed_rows_per_s": world * new_rows * args.steps / (r["total_ms"] / 1000.0),
                   "l2": f"inputs exceed L2: {shape.params_per_layer * shape.n_layers * 2 / 1e6:.0f} MB of weights are "
                         "streamed every step", "multi_gpu": "independent replicas, no collective",
                   "cache_state": "chunks stored by a step are dropped again before the next (untimed host bookkeeping)",
                   "device_ms_per_step_kernels_only": r["dev_us"] / args.steps / 1000.0,
                   "host_plan_us": st["host_plan_us"], "phase_pass_ms_per_step": float(sum(r["ms_ph"])) / r["ph_steps"]},
        "clocks": r["clocks"],
        "e2e": {"value": e2e_value, "unit": UNIT,
                "h2d_bytes_per_step": (tokens if w.paper_mode else new_rows) * shape.d_model * 2,
                "d2h_bytes_per_step": (tokens if w.paper_mode else new_rows) * shape.d_model * 4,
                "ms_per_step": r["e2e_ms"] / args.steps},
        "gpu_launches": kernels_per_step * args.steps,
        "roofline": roof, "kernels": per_phase, "cpu_baseline": cpu,
        "step_tflops": main_row["step_tflops"], "step_frac_of_tensor_peak": main_row["step_frac_of_tensor_peak"],
        "workloads": rows}))


def run_qa_bank(args):
    """QA-bank lookup (cosine top-1 over all stored query embeddings): streams the bank once per call."""
    import torch
    from paper_2601_11553_b200 import percache as pcb
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    n, dim = 65536, 1024                       # 268 MB of fp32 embeddings: larger than L2
    g = torch.Generator(device=dev).manual_seed(5)
    bank = torch.randn((n, dim), generator=g, device=dev, dtype=torch.float32)
    peaks = load_peaks()
    out = {}
    for nq in (1, 8):
        queries = bank[:nq] * 1.5 + 0.1 * torch.randn((nq, dim), generator=g, device=dev)
        queries = queries.contiguous()
        stream = torch.cuda.current_stream(dev)
        for _ in range(max(args.warmup, 3)):
            pcb.qa_top1(bank, queries, 0.85, device=dev.index, stream=stream.cuda_stream)
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        kus = []
        for a, b in ev:
            a.record(stream)
            idx, score, hit, us = pcb.qa_top1(bank, queries, 0.85, device=dev.index, stream=stream.cuda_stream, timing=True)
            b.record(stream)
            kus.append(us)
        torch.cuda.synchronize(dev)
        ms = float(np.median([a.elapsed_time(b) for a, b in ev]))
        kms = float(np.median(kus)) / 1000.0
        out[nq] = {"ms_per_call": ms, "kernel_ms": kms, "gbs": n * dim * 4 / kms / 1e6, "top1": idx.tolist()[:2]}
    print(json.dumps({"metric": "qa_bank_lookup_gbs", "value": out[1]["gbs"], "unit": "GB/s", "n_gpus": 1,
                      "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": out[1]["ms_per_call"], "kernel_ms": out[1]["kernel_ms"],
                      "higher_is_better": True, "dtype": "f32", "data": "synthetic",
                      "config": {"workload": "qa_bank", "entries": n, "dim": dim, "bytes_per_call": n * dim * 4,
                                 "l2": "bank (268 MB) exceeds L2"},
                      "roofline": {"bound": "hbm", "achieved": out[1]["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                   "frac": out[1]["gbs"] / peaks["hbm_gbs"], "traffic": None, "kernel": "qa_top1_kernel<1>",
                                   "peak_source": peaks["source"]},
                      "batch_of_8_queries": out[8]}))


def run_decode(args):
    """Decode steps after a reuse-prefill of the named workload: one token per prompt and step.

    HBM-bound: every step streams all weights once and every prompt's assembled K/V once."""
    import torch
    from paper_2601_11553_b200 import percache as pcb
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    w = wl.by_name(args.workload[len("decode_"):])
    shape = w.shape
    weights_np = wl.make_weights(shape, w.seed)
    weights = [{k: torch.from_numpy(v.view(np.int16)).to(dev).view(torch.bfloat16) for k, v in lw.items()}
               for lw in weights_np]
    ids_lens = {c: l for p in w.prompts for c, l in zip(p.chunk_ids, p.chunk_len)}
    steps, warm = args.steps, max(args.warmup, 3)
    reserve = warm + 2 * steps + 8
    B = len(w.prompts)
    stream = torch.cuda.current_stream(dev)
    h = pcb.PerCache(n_layers=shape.n_layers, d_model=shape.d_model, n_q_heads=shape.n_q_heads,
                     n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, d_ffn=shape.d_ffn, weights=weights,
                     # + pages lent to the query rows and to the decoded tokens when the prefill runs gather-free
                     pool_pages=sum((l + 15) // 16 for l in ids_lens.values()) + 64
                     + sum((p.n_query + reserve + 15) // 16 + 2 for p in w.prompts),
                     max_prompt_tokens=max(p.n_total for p in w.prompts) + reserve, max_batch_prompts=B,
                     max_batch_ctx_tokens=w.total_tokens + B * reserve, max_batch_new_rows=w.total_tokens, device=local,
                     stream=stream.cuda_stream)
    del weights
    h.set_decode_reserve(reserve)
    h.set_flags(args.flags)
    cached = set(w.cached_ids)
    for c in w.cached_ids:
        if w.cache_source == "integer_pool":
            h.put_chunk_synthetic(c, ids_lens[c], w.seed)
        else:
            h.prefill([pcb.PromptSpec([c], [ids_lens[c]], [wl.chunk_hidden_for(w.seed, c, ids_lens[c], shape.d_model)], None, 0)])

    def to_dev(a):
        return torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)
    specs = []
    for p in w.prompts:
        hid = [None if c in cached else to_dev(hh) for c, hh in zip(p.chunk_ids, p.chunk_hidden)] if p.chunk_hidden else None
        specs.append(pcb.PromptSpec(list(p.chunk_ids), list(p.chunk_len), hid, to_dev(p.query_hidden), p.n_query))
    h.prefill(specs)
    tok_dev = to_dev(wl.make_hidden(w.seed, (9, 0), B, shape.d_model))
    tok_host = torch.from_numpy(wl.make_hidden(w.seed, (9, 0), B, shape.d_model).view(np.int16)).pin_memory().view(torch.bfloat16)
    out_dev = torch.empty((B, shape.d_model), dtype=torch.float32, device=dev)
    out_host = torch.empty((B, shape.d_model), dtype=torch.float32).pin_memory()

    def timed(tok, out, n):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        ctx, dev_us = 0, 0.0
        for a, b in ev:
            a.record(stream)
            h.decode(tok, out=out)
            b.record(stream)
            st = h.stats()
            ctx += st["ctx_tokens"]
            dev_us += st["device_us"]
        torch.cuda.synchronize(dev)
        timed.device_ms = dev_us / 1000.0 / n
        return [a.elapsed_time(b) for a, b in ev], ctx
    timed(tok_dev, out_dev, warm)
    sampler = ClockSampler(local)
    sampler.start()
    ms, ctx_tokens = timed(tok_dev, out_dev, steps)
    device_ms = timed.device_ms
    clocks = sampler.stop()
    ms_e2e, _ = timed(tok_host, out_host, steps)
    launches = sum(h.stats()["phase_launches"].values())
    # per-kernel-class durations from a separate pass with events around every class
    h.set_flags(args.flags | pcb.FLAG_PHASE_TIMING)
    h.decode(tok_dev, out=out_dev)
    h.decode(tok_dev, out=out_dev)
    st = h.stats()
    h.set_flags(args.flags)
    per_phase = {k: {"us_per_launch": st["phase_us"][k] / st["phase_launches"][k], "launches_per_step": st["phase_launches"][k]}
                 for k in pcb.PHASES if st["phase_launches"][k]}
    total_ms, e2e_ms = float(sum(ms)), float(sum(ms_e2e))
    peaks = load_peaks()
    weight_bytes = shape.params_per_layer * shape.n_layers * 2
    kv_bytes = ctx_tokens / steps * shape.kv_dim * 2 * 2 * shape.n_layers          # fp16 K and V of every slot, every layer
    gbs = (weight_bytes + kv_bytes) / (total_ms / steps) / 1e6
    print(json.dumps({
        "metric": "decode_tokens_per_s", "value": B * steps / (total_ms / 1000.0), "unit": "tokens/s", "n_gpus": 1,
        "steps": steps, "warmup": warm, "ms_per_step": total_ms / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f16", "data": "synthetic",
        "config": {"workload": args.workload, "description": "one decoded token per prompt and step after the prefill of "
                   + w.description, "prompts": B, "ctx_tokens": ctx_tokens / steps,
                   "device_ms_per_step_kernels_only": device_ms,
                   "l2": f"weights ({weight_bytes / 1e6:.0f} MB) exceed L2"},
        "clocks": clocks,
        "e2e": {"value": B * steps / (e2e_ms / 1000.0), "unit": "tokens/s", "h2d_bytes_per_step": B * shape.d_model * 2,
                "d2h_bytes_per_step": B * shape.d_model * 4, "ms_per_step": e2e_ms / steps},
        "gpu_launches": launches * steps,
        "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                     "traffic": None, "kernel": "whole decode step (weights + assembled K/V streamed once)",
                     "peak_source": peaks["source"], "algorithmic_per_launch": weight_bytes + kv_bytes},
        "kernels": per_phase}))
    h.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--impl", default="percache", choices=["percache", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-table", action="store_true", help="time the named workload only, not the per-workload table")
    ap.add_argument("--flags", type=int, default=0, help="PERCACHE_FLAG_* bits kept set during the timed passes")
    ap.add_argument("--layers", type=int, default=0,
                    help="profiling aid: run the workload on a model cut to this many layers (every launch keeps its shape, "
                         "a profiler capture stays small); the line then says reduced_depth and is not a result")
    args = ap.parse_args()
    args.forward = sys.argv[1:]
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        # asked for N GPUs without a launcher around us: start one rank per GPU ourselves (independent replicas;
        # the only thing they exchange is the maximum of their times)
        import socket
        import subprocess
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        raise SystemExit(subprocess.call(replica_launch_command(args, port)))
    if args.workload == "qa_bank":
        run_qa_bank(args)
    elif args.workload.startswith("decode_"):
        run_decode(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
