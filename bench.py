#!/usr/bin/env python
"""Benchmark of reuse-prefill on B200: one step = one percache_prefill call of the workload.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg1] [--impl reference]

Prints ONE JSON line.  `value` is context tokens per second (prompt tokens served / time) with inputs
resident in HBM; `e2e` is the same through host buffers (pinned input hidden states copied in, output
rows copied out inside the timed call).  Between steps the chunks the call stored are dropped again
(host-only bookkeeping, untimed) so that every step sees the same cache state.

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
    out = {k: v * new_rows * s.n_layers for k, v in per_row.items()}
    out["attn"] = 4 * s.n_q_heads * s.head_dim * visible_pairs * s.n_layers
    return out


# --------------------------------------------------------------------------- CPU oracle leg
def oracle_sample(w: wl.Workload, n_layers_sample: int):
    """Time the oracle on the first `n_layers_sample` layers of the workload's model (all rows, same prompts)."""
    from oracle import reuse_prefill as orc
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        cores = os.cpu_count() or 1
    shape = wl.ModelShape(n_layers=n_layers_sample, **{k: getattr(w.shape, k) for k in
                                                       ("d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn")})
    weights = wl.make_weights(shape, w.seed)
    model = orc.Model(n_layers=shape.n_layers, d_model=shape.d_model, n_q_heads=shape.n_q_heads,
                      n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, d_ffn=shape.d_ffn,
                      rope_theta=shape.rope_theta, rms_eps=shape.rms_eps, layers=weights)
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


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = wl.by_name(args.workload)
    n_sample = 1
    step, cores = oracle_sample(w, n_sample)
    for _ in range(min(args.warmup, 1)):
        step()
    times = [step() for _ in range(args.steps)]
    scale = w.shape.n_layers / n_sample
    ms = 1000.0 * float(np.mean(times)) * scale
    value = w.total_tokens / (ms / 1000.0)
    sample = f"layer 0 of {w.shape.n_layers} of {w.name} (all prompts, all new rows), time x {scale:g}"
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


# --------------------------------------------------------------------------- GPU leg
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

    w = wl.by_name(args.workload)
    shape = w.shape
    weights_np = wl.make_weights(shape, w.seed)
    weights = [{k: torch.from_numpy(v.view(np.int16)).to(dev).view(torch.bfloat16) for k, v in lw.items()}
               for lw in weights_np]
    ids_lens = {c: l for p in w.prompts for c, l in zip(p.chunk_ids, p.chunk_len)}
    pool_pages = sum((l + 15) // 16 for l in ids_lens.values()) + 64
    stream = torch.cuda.current_stream(dev)
    h = pcb.PerCache(n_layers=shape.n_layers, d_model=shape.d_model, n_q_heads=shape.n_q_heads,
                     n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, d_ffn=shape.d_ffn, weights=weights,
                     pool_pages=pool_pages, max_prompt_tokens=max(p.n_total for p in w.prompts),
                     max_batch_prompts=len(w.prompts), max_batch_ctx_tokens=w.total_tokens,
                     max_batch_new_rows=w.total_tokens, device=local, stream=stream.cuda_stream)
    del weights
    # ---- cache state before every step
    cached = set(w.cached_ids)
    if w.cache_source == "integer_pool":
        for c in w.cached_ids:
            h.put_chunk_synthetic(c, ids_lens[c], w.seed)
    else:   # prefill every cached chunk alone through the library itself
        for c in w.cached_ids:
            hid = wl.chunk_hidden_for(w.seed, c, ids_lens[c], shape.d_model)
            h.prefill([pcb.PromptSpec([c], [ids_lens[c]], [hid], None, 0)])
    missed = sorted({c for p in w.prompts for c in p.chunk_ids if c not in cached})

    def to_dev(a):
        return torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)

    def to_pinned(a):
        return torch.from_numpy(a.view(np.int16)).pin_memory().view(torch.bfloat16)

    def specs(conv):
        out = []
        for p in w.prompts:
            hid = [None if c in cached else conv(hh) for c, hh in zip(p.chunk_ids, p.chunk_hidden)] \
                if p.chunk_hidden else None
            out.append(pcb.PromptSpec(list(p.chunk_ids), list(p.chunk_len), hid, conv(p.query_hidden), p.n_query))
        return out

    specs_dev, specs_host = specs(to_dev), specs(to_pinned)
    n_new = [p.n_query + sum(l for c, l in zip(p.chunk_ids, p.chunk_len) if c not in cached) for p in w.prompts]
    out_dev = [torch.empty((n, shape.d_model), dtype=torch.float32, device=dev) for n in n_new]
    out_host = [torch.empty((n, shape.d_model), dtype=torch.float32).pin_memory() for n in n_new]

    def restore():
        for c in missed:
            h.drop_chunk(c)

    def timed(spec_list, outs, steps, collect_phases=False):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        phases = {k: 0.0 for k in pcb.PHASES}
        launches = {k: 0 for k in pcb.PHASES}
        dev_us = 0.0
        for i in range(steps):
            ev[i][0].record(stream)
            h.prefill(spec_list, out=outs)
            ev[i][1].record(stream)
            st = h.stats()
            dev_us += st["device_us"]
            for k in pcb.PHASES:
                phases[k] += st["phase_us"][k]
                launches[k] += st["phase_launches"][k]
            restore()
        torch.cuda.synchronize(dev)
        ms = [a.elapsed_time(b) for a, b in ev]
        return ms, phases, launches, dev_us, st

    def barrier():
        torch.cuda.synchronize(dev)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    # ---- warm-up, then the timed region (device-resident inputs), max over ranks
    h.set_flags(args.flags)
    timed(specs_dev, out_dev, max(args.warmup, 3))
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    ms, _, launches, dev_us, st = timed(specs_dev, out_dev, args.steps)
    barrier()
    clocks = sampler.stop()
    total_ms = float(sum(ms))
    # ---- same steps with per-kernel-class events (separate pass: the extra events cost a few percent)
    h.set_flags(args.flags | pcb.FLAG_PHASE_TIMING)
    timed(specs_dev, out_dev, 2)
    ms_ph, phases, launches_ph, _, _ = timed(specs_dev, out_dev, args.steps)
    h.set_flags(args.flags)
    # ---- end to end through host buffers
    timed(specs_host, out_host, 3)
    barrier()
    ms_e2e, _, _, _, _ = timed(specs_host, out_host, args.steps)
    barrier()
    e2e_ms = float(sum(ms_e2e))
    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], dist, dev)
    if rank != 0:
        return

    peaks = load_peaks()
    tokens = w.total_tokens
    new_rows = int(st["new_rows"])
    value = aggregate_tokens_per_s(world, tokens, args.steps, total_ms)
    e2e_value = aggregate_tokens_per_s(world, tokens, args.steps, e2e_ms)
    fl = flops_per_step(w, new_rows, int(st["attn_visible_pairs"]))
    gather_bytes = int(st["hit_tokens"]) * shape.n_layers * shape.kv_dim * 2 * 2 * 2
    per_phase = {}
    for k in ("qkv", "attn", "oproj", "gateup", "down"):
        n = launches_ph[k]
        if n:
            us = phases[k] / n
            per_phase[k] = {"us_per_launch": us, "launches_per_step": n // args.steps,
                            "tflops": fl[k] / shape.n_layers / us / 1e6}
    if launches_ph["gather"]:
        us = phases["gather"] / launches_ph["gather"]
        per_phase["gather"] = {"us_per_launch": us, "launches_per_step": 1, "gbs": gather_bytes / us / 1e3}
    if launches_ph["norm"]:
        per_phase["norm"] = {"us_per_launch": phases["norm"] / launches_ph["norm"],
                             "launches_per_step": launches_ph["norm"] // args.steps}
    dom = max(("qkv", "attn", "oproj", "gateup", "down", "gather"), key=lambda k: phases[k])
    if dom == "gather":
        roof = {"bound": "hbm", "achieved": per_phase[dom]["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": per_phase[dom]["gbs"] / peaks["hbm_gbs"], "traffic": None, "kernel": "gather_rerope_kernel"}
    else:
        roof = {"bound": "tensor", "achieved": per_phase[dom]["tflops"], "peak": peaks["tflops_sustained"],
                "unit": "TFLOP/s", "frac": per_phase[dom]["tflops"] / peaks["tflops_sustained"], "traffic": None,
                "kernel": {"attn": "umma_attention_kernel"}.get(dom, f"umma_gemm_kernel<{dom}>")}
    roof["peak_source"] = f"{peaks['source']} (sustained bf16 figure x 1.0 nominal fp16/bf16 ratio)" \
        if roof["bound"] == "tensor" else peaks["source"]
    roof["share_of_step"] = phases[dom] / max(sum(phases.values()), 1e-9)
    roof["traffic"] = kernel_traffic(roof["kernel"], w.name)
    roof["algorithmic_per_launch"] = gather_bytes if dom == "gather" else fl[dom] / shape.n_layers
    kernels_per_step = (sum(launches[k] for k in pcb.PHASES if k != "io") // args.steps) + 1

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        n_sample = max(1, min(shape.n_layers, 7))
        step, cores = oracle_sample(w, n_sample)
        t = step()
        scale = shape.n_layers / n_sample
        cpu = {"value": tokens / (t * scale), "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"first {n_sample} of {shape.n_layers} layers of {w.name}, all new rows, one call "
                         f"({t:.1f} s), time x {scale:g}"}

    print(json.dumps({
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16", "data": "synthetic",
        "config": {"workload": w.name, "description": w.description, "tokens_per_step": tokens,
                   "new_rows_per_step": new_rows, "hit_tokens_per_step": int(st["hit_tokens"]),
                   "prompts_per_step": len(w.prompts), "ms_per_prompt": total_ms / args.steps / len(w.prompts),
                   "computed_rows_per_s": world * new_rows * args.steps / (total_ms / 1000.0),
                   "l2": f"inputs exceed L2: {shape.params_per_layer * shape.n_layers * 2 / 1e6:.0f} MB of weights are "
                         "streamed every step", "multi_gpu": "independent replicas, no collective",
                   "cache_state": "chunks stored by a step are dropped again before the next (untimed host bookkeeping)",
                   "device_ms_per_step_kernels_only": dev_us / args.steps / 1000.0,
                   "host_plan_us": st["host_plan_us"], "phase_pass_ms_per_step": float(sum(ms_ph)) / args.steps},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": new_rows * shape.d_model * 2,
                "d2h_bytes_per_step": new_rows * shape.d_model * 4, "ms_per_step": e2e_ms / args.steps},
        "gpu_launches": kernels_per_step * args.steps,
        "roofline": roof, "kernels": per_phase, "cpu_baseline": cpu}))
    h.close()
    if dist is not None:
        dist.destroy_process_group()


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
                     pool_pages=sum((l + 15) // 16 for l in ids_lens.values()) + 64,
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
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="cfg1")
    ap.add_argument("--impl", default="percache", choices=["percache", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--flags", type=int, default=0, help="PERCACHE_FLAG_* bits kept set during the timed passes")
    args = ap.parse_args()
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
