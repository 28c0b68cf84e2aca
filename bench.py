#!/usr/bin/env python
"""Benchmark of the GLIDE hybrid-attention decode step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl glide|reference]

A step is one glide_decode_step: one token for every layer and sequence of the workload, the
fused launch covering ring append/eviction, phi, state fold, window attention, linear readout
and the shared-normaliser merge.  The state the steps start from is built (untimed) by
glide_prefill over the synthetic prompt.  Default workload: Llama-3-8B-shaped stack, batch 1,
32K context (configs.C1).  Prints ONE JSON line.

Timing: CUDA events on the launching stream around exactly K steps, repeated until at least half a
second of timed work has accumulated while NVML samples the clocks; the median repetition is
reported.  Consecutive steps rotate over several independent copies of the sequence state (total
footprint well above the 126 MB L2), so no step finds its window or state in L2 from the step
before.  `value` is the back-to-back throughput (the launches of consecutive steps overlap by
programmatic dependent launch); `per_step_attention_latency_us` is the median of steps timed one
by one between their own events.  After the headline workload the other configurations and the two
controls (uniform window, full-KV softmax) are timed the same way and reported under `workloads`.

N > 1 (torchrun): the path does not shard -- every rank runs an independent replica of the
workload on its own GPU, no collective on the data path; value = tokens of all ranks / max time.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2607_24788_b200 import configs, synth  # noqa: E402

L2_BYTES = 126e6
# dram__bytes_read.sum + dram__bytes_write.sum per decode launch from the committed ncu capture
# (profiles/), keyed by workload name; None until a capture exists for that workload.
NCU_TRAFFIC_BYTES = {"c1_llama8b_b1_32k": 142.1e6}   # profiles/decode_stream_c1.md
MIN_TIMED_S = 0.5     # the K-step region is repeated until this much timed work has accumulated
MAX_REPS = 4000
KERNEL_KNOBS = {}   # tuning overrides from the command line (decode_chunk, decode_state_splits, decode_impl)
PHI = {"kind": 0}   # --phi 1: the learned feature map (d x d projections with N(0, 1/d) weights, 2d features)
_phi_weights = {}


def glide_kwargs(shape, device):
    """Keyword arguments of glide.Glide / make_config for this run: the kernel knobs and, for --phi 1, the feature
    map's projections (seeded, one set per shape and device, shared by every context built for it)."""
    kw = dict(KERNEL_KNOBS)
    if PHI["kind"]:
        key = (shape.name, str(device))
        if key not in _phi_weights:
            gen = torch.Generator().manual_seed(shape.seed + 77)
            d, dt = shape.head_dim, torch_dtype(shape)
            wq = (torch.randn((shape.n_layers, shape.n_q_heads, d, d), generator=gen) / math.sqrt(d)).to(dt)
            wk = (torch.randn((shape.n_layers, shape.n_kv_heads, d, d), generator=gen) / math.sqrt(d)).to(dt)
            _phi_weights[key] = (wq.to(device), wk.to(device))
        kw.update(phi=PHI["kind"], phi_wq=_phi_weights[key][0], phi_wk=_phi_weights[key][1])
    return kw


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for name, bit in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.01)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def torch_dtype(shape):
    return torch.float32 if shape.dtype == "f32" else torch.bfloat16


def value_scale(shape):
    """Standard deviation of the q and k entries."""
    if shape.value_scales is not None:
        return shape.value_scales[0]
    return synth.default_value_scale(shape.head_dim, shape.unit_variance)


def make_workload(shape):
    """The seeded input generator of a configuration."""
    return synth.Workload(shape.seed, shape.n_layers, shape.batch, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                          torch_dtype(shape), value_scale(shape),
                          v_scale=None if shape.value_scales is None else shape.value_scales[1])


# ---------------------------------------------------------------------------------------------
# CPU oracle leg (cpu_baseline and --impl reference)
# ---------------------------------------------------------------------------------------------
def oracle_decode_rate(shape, steps: int, warmup: int, single_steps: int = 0):
    """Times the oracle's decode step on the host cores on a bounded sample of the workload: one layer of
    every distinct window size, sequence 0, state built by the oracle's own prefill of the full prompt.
    Per-layer-class times are scaled by the number of layers and sequences of each class."""
    from oracle import glide_oracle as orc
    import numpy as np
    dt = torch_dtype(shape)
    wl = make_workload(shape)
    scale = float(np.float32(1.0) / np.sqrt(np.float32(shape.head_dim)))
    classes = {}
    for l, w in enumerate(shape.windows):
        classes.setdefault(w, []).append(l)
    per_class_s = {}
    threads = orc.max_threads()
    used = 1
    single_s = {}
    for w, layers in classes.items():
        l = layers[0]
        okw = {}
        if PHI["kind"]:
            gen = torch.Generator().manual_seed(shape.seed + 77 + l)
            d = shape.head_dim
            okw = dict(phi=PHI["kind"],
                       wq=[(torch.randn((shape.n_q_heads, d, d), generator=gen) / math.sqrt(d)).to(dt).double().numpy()],
                       wk=[(torch.randn((shape.n_kv_heads, d, d), generator=gen) / math.sqrt(d)).to(dt).double().numpy()])
        stack = orc.Stack([w], 1, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, scale, merge=KERNEL_KNOBS.get("merge", 0),
                          **okw)
        # only the tokens that can still matter are absorbed one piece at a time
        piece = 2048
        for pos in range(0, shape.context, piece):
            k, v = wl.kv([l], [0], range(pos, min(pos + piece, shape.context)))
            stack.prefill(None, k.double().numpy(), v.double().numpy(), outputs=False)
        times = []
        for s in range(warmup + steps):
            q, k, v = wl.qkv([l], [0], [shape.context + s])
            q, k, v = (x[:, :, 0].double().numpy() for x in (q, k, v))
            t0 = time.perf_counter()
            stack.decode(q, k, v, threads=threads)
            t1 = time.perf_counter()
            used = max(used, stack.threads_used)
            if s >= warmup:
                times.append(t1 - t0)
        per_class_s[w] = statistics.median(times)
        times = []
        for s in range(single_steps):   # the same stack, one thread
            q, k, v = wl.qkv([l], [0], [shape.context + warmup + steps + s])
            q, k, v = (x[:, :, 0].double().numpy() for x in (q, k, v))
            t0 = time.perf_counter()
            stack.decode(q, k, v, threads=1)
            times.append(time.perf_counter() - t0)
        if times:
            single_s[w] = statistics.median(times)
    if single_steps:
        oracle_decode_rate.single_thread_step_s = sum(single_s[w] * len(layers) for w, layers in classes.items()) * shape.batch
    step_s = sum(per_class_s[w] * len(layers) for w, layers in classes.items()) * shape.batch
    sample = (f"layers {sorted(v[0] for v in classes.values())} (one per distinct window), sequence 0, "
              f"{steps} decode steps each after the oracle's own {shape.context}-token prefill; "
              f"per-class median step time x layers of the class x batch")
    return shape.batch / step_s, step_s, used, sample


def workload_config(shape, extra=None):
    """The `config` object of a bench line: what was run, the same keys for both arms."""
    cfg = {"workload": shape.name, "batch": shape.batch, "context": shape.context, "n_layers": shape.n_layers,
           "sum_windows": sum(shape.windows), "q_heads": shape.n_q_heads, "kv_heads": shape.n_kv_heads,
           "head_dim": shape.head_dim, "multi_gpu": "replicas only", "merge": KERNEL_KNOBS.get("merge", 0),
           "phi": "softmax over the features (d)" if not PHI["kind"] else "learned projection, two softmax halves (2d)"}
    if extra:
        cfg.update(extra)
    return cfg


def run_reference(args, shape):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = min(args.steps, 16)
    tok_s, step_s, cores, sample = oracle_decode_rate(shape, steps, min(args.warmup, 2))
    line = {
        "impl": "reference", "metric": "hybrid-attn decode tokens/s", "value": tok_s, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_s * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(shape, {"l2": "host memory (the oracle runs on the host cores)",
                                          "timing": f"{steps} oracle steps per distinct window size, see cpu_baseline.sample"}),
        "cpu_baseline": {"value": tok_s, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": tok_s, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------
# GPU leg
# ---------------------------------------------------------------------------------------------
def build_states(shape, n_replicas: int, extra_tokens: int, device):
    from paper_2607_24788_b200 import glide
    dt = torch_dtype(shape)
    wl = make_workload(shape)
    max_tokens = shape.context + extra_tokens
    ctxs = [glide.Glide(shape.windows, shape.batch, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, max_tokens,
                        dtype=dt, device=device, prefill_chunk=shape.prefill_chunk, **glide_kwargs(shape, device))
             for _ in range(n_replicas)]
    g0 = ctxs[0]
    # prompt -> state (no outputs needed for a decode benchmark); layers in groups to bound the k/v buffers
    budget_elems = 256 << 20
    per_token_layer = shape.batch * shape.n_kv_heads * shape.head_dim
    piece = 4096
    lgroup = max(1, min(shape.n_layers, budget_elems // (piece * per_token_layer)))
    for lb in range(0, shape.n_layers, lgroup):
        lc = min(lgroup, shape.n_layers - lb)
        for pos in range(0, shape.context, piece):
            k, v = wl.kv(range(lb, lb + lc), range(shape.batch), range(pos, min(pos + piece, shape.context)), device)
            g0.glide_prefill(None, k, v, None, layer_begin=lb, layer_count=lc)
            del k, v
    torch.cuda.synchronize()
    for g in ctxs[1:]:
        for l in range(shape.n_layers):
            rk, rv, S, z = g0.glide_export_state(l)
            cap = g0.capacity(l)
            g.glide_import_state(l, shape.context, rk if cap else None, rv if cap else None, S, z)
        torch.cuda.synchronize()
    return ctxs, wl


def decode_kernel_name(shape) -> str:
    """The kernel glide_create selects for this shape and these knobs (see include/glide.h)."""
    impl, merge = KERNEL_KNOBS.get("decode_impl", 0), KERNEL_KNOBS.get("merge", 0)
    if shape.dtype == "f32" or impl == 2:
        return "glide_decode_kernel"
    if shape.head_dim == 128 and impl in (0, 3):
        return "glide_decode_stream_kernel"
    return "glide_decode_mma_kernel" if merge == 0 else "glide_decode_kernel"


def max_over_ranks(values, dist, device):
    """Replicas only: every rank times its own independent copy of the workload; the job's time is the
    slowest rank's (max over ranks).  `dist` is torch.distributed or None for a single process."""
    if dist is None:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def whole_job_tokens_per_s(world: int, batch: int, steps: int, ms: float) -> float:
    """Aggregate over all replicas: every rank decodes `batch` sequences for `steps` steps in `ms`."""
    return world * batch * steps / (ms * 1e-3)


def roofline_bytes(shape):
    """(the benchmark spec's bytes, bytes with the step's own q/k/v/out rows and the ring append) of one decode step.  With
    the learned feature map the state is twice as large and the step also reads the projections once."""
    fm = 2 if PHI["kind"] else 1
    extra = 0
    if PHI["kind"]:
        extra = shape.n_layers * (shape.n_q_heads + shape.n_kv_heads) * shape.head_dim ** 2 * shape.elem_bytes
    return (configs.decode_step_stream_bytes(shape, shape.context, fm),
            configs.decode_step_bytes(shape, shape.context, fm) + extra)


class DecodeBench:
    """The decode-step measurement of one workload: state copies built by glide_prefill, inputs resident in HBM,
    K back-to-back steps between two CUDA events, repeated; steps rotate over the state copies."""

    def __init__(self, shape, K, W, device, dist, prefill_tokens=0):
        self.shape, self.K, self.W, self.device, self.dist = shape, K, max(W, 3), device, dist
        self.bytes_stream, self.bytes_io = roofline_bytes(shape)
        self.prefill_tokens = prefill_tokens
        free_b, _ = torch.cuda.mem_get_info(device)
        n_rep = max(1, min(16, math.ceil(8 * L2_BYTES / self.bytes_io)))
        # positions a state copy may advance before it is rewound (and room for the prefill measurement at the end)
        self.slack = max(256, 8 * K + 64) + 3 * prefill_tokens
        cfg_probe = self._workspace_bytes(shape, self.slack)
        n_rep = max(1, min(n_rep, int(0.8 * free_b // max(cfg_probe, 1))))
        self.n_rep = n_rep
        self.ctxs, self.wl = build_states(shape, n_rep, self.slack, device)
        L, B, H, Hkv, d = shape.n_layers, shape.batch, shape.n_q_heads, shape.n_kv_heads, shape.head_dim
        self.dt = torch_dtype(shape)
        # inputs of the timed steps, resident in HBM: one buffer per step holding q | k | v
        self.n_in = min(K, 64)
        self.nq, self.nk = L * B * H * d, L * B * Hkv * d
        self.dev_in = torch.empty((self.n_in, self.nq + 2 * self.nk), dtype=self.dt, device=device)
        for i in range(self.n_in):
            q, k, v = self.wl.decode_qkv(shape.context + i, device)
            self.dev_in[i, :self.nq] = q.reshape(-1)
            self.dev_in[i, self.nq:self.nq + self.nk] = k.reshape(-1)
            self.dev_in[i, self.nq + self.nk:] = v.reshape(-1)
        self.outs = [torch.empty((L, B, H, d), dtype=self.dt, device=device) for _ in range(2)]
        self.step_no = 0
        self.advanced = [0] * n_rep              # steps each copy has taken since it was last rewound

    @staticmethod
    def _workspace_bytes(shape, slack):
        from paper_2607_24788_b200 import glide
        cfg, keep = glide.make_config(shape.windows, shape.batch, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                                      shape.context + slack, dtype=torch_dtype(shape), prefill_chunk=shape.prefill_chunk,
                                      **glide_kwargs(shape, "cuda"))
        return glide.glide_workspace_bytes(cfg)

    def views(self, buf):
        L, B, H, Hkv, d = (self.shape.n_layers, self.shape.batch, self.shape.n_q_heads, self.shape.n_kv_heads,
                           self.shape.head_dim)
        nq, nk = self.nq, self.nk
        return (buf[:nq].view(L, B, H, d), buf[nq:nq + nk].view(L, B, Hkv, d), buf[nq + nk:].view(L, B, Hkv, d))

    def one_step(self, buf, ctx_index=None):
        i = self.step_no
        self.step_no += 1
        c = i % self.n_rep if ctx_index is None else ctx_index
        q, k, v = self.views(buf)
        self.ctxs[c].glide_decode_step(q, k, v, self.outs[i & 1])
        self.advanced[c] += 1

    def make_room(self, steps_per_ctx):
        """Rewinds the position counters of copies that could not take `steps_per_ctx` more steps (untimed; ring, S
        and z stay as they are: the time of a step does not depend on the values)."""
        for c in range(len(self.ctxs)):
            if self.advanced[c] + steps_per_ctx + 2 > self.slack - 3 * self.prefill_tokens:
                self.rewind(c)

    def rewind(self, c):
        for l in range(self.shape.n_layers):
            self.ctxs[c].glide_import_state(l, self.shape.context, None, None, None, None)
        self.advanced[c] = 0

    def barrier(self):
        torch.cuda.synchronize()
        if self.dist is not None:
            self.dist.barrier()
            torch.cuda.synchronize()

    def warm_up(self):
        for i in range(self.W):
            self.one_step(self.dev_in[i % self.n_in])
        self.barrier()

    def back_to_back(self, reps, local_rank):
        """Median time of K back-to-back steps; repeated `reps` times at least and until MIN_TIMED_S of timed work."""
        K = self.K
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        times_ms, total = [], 0.0
        per_ctx = math.ceil(K / self.n_rep) + 1
        with ClockSampler(local_rank) as clocks:
            while len(times_ms) < reps or (total < MIN_TIMED_S * 1e3 and len(times_ms) < MAX_REPS):
                self.make_room(per_ctx)
                self.barrier()
                ev0.record()
                for i in range(K):
                    self.one_step(self.dev_in[i % self.n_in])
                ev1.record()
                self.barrier()
                times_ms.append(ev0.elapsed_time(ev1))
                total += times_ms[-1]
        return statistics.median(times_ms), len(times_ms), clocks.summary()

    def isolated(self, n_steps):
        """Every step between its own pair of events (rotating state copies as above): an event between two launches
        keeps the next launch from overlapping the previous one's tail.  Sorted microseconds."""
        self.make_room(math.ceil(n_steps / self.n_rep) + 1)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_steps)]
        self.barrier()
        for i in range(n_steps):
            evs[i][0].record()
            self.one_step(self.dev_in[i % self.n_in])
            evs[i][1].record()
        self.barrier()
        return sorted(a.elapsed_time(b) * 1e3 for a, b in evs)

    def close(self):
        self.ctxs, self.dev_in, self.outs = None, None, None
        torch.cuda.empty_cache()


def latency_summary(lat_us):
    return {"median": lat_us[len(lat_us) // 2], "p10": lat_us[len(lat_us) // 10], "p90": lat_us[(len(lat_us) * 9) // 10],
            "steps": len(lat_us),
            "note": "each step between its own two events (no overlap with the neighbours), rank 0"}


def side_workload(shape, K, W, device, local_rank, prefill_tokens=0):
    """One entry of `workloads`: the same decode measurement on another configuration or control."""
    peak, peak_kind = load_peaks()
    b = DecodeBench(shape, K, W, device, None, prefill_tokens)
    b.warm_up()
    t_ms, n_reps, clocks = b.back_to_back(3, local_rank)
    lat = b.isolated(max(K, 16))
    us = t_ms * 1e3 / K
    entry = {"us_per_step": us, "tokens_per_s": shape.batch / (us * 1e-6), "isolated_step_us": latency_summary(lat)["median"],
             "algorithmic_bytes_per_launch": b.bytes_stream, "algorithmic_bytes_incl_io": b.bytes_io,
             "achieved_gbs": b.bytes_stream / (us * 1e-6) / 1e9, "frac": b.bytes_stream / (us * 1e-6) / 1e9 / peak,
             "frac_incl_io": b.bytes_io / (us * 1e-6) / 1e9 / peak, "peak_kind": f"of {peak_kind}",
             "state_copies": b.n_rep, "repetitions": n_reps, "steps_per_repetition": K, "clocks": clocks,
             "kernel": decode_kernel_name(shape), "sum_windows": sum(shape.windows), "batch": shape.batch,
             "context": shape.context}
    if prefill_tokens > 0:
        b.rewind(b.n_rep - 1)
        entry["prefill"] = measure_prefill(b.ctxs[-1], b.wl, shape, prefill_tokens, device)
    b.close()
    return entry


SIDE_WORKLOADS = ("c2_llama8b_b16_16k", "c2_control_uniform_w1024", "c3_llama8b_b4_128k", "c3_control_full_kv",
                  "c4_mistral7b_b8_8k_chunked", "p1_blockwise_0_half_w")


def run_glide(args, shape):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the GLIDE path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    K, W = args.steps, args.warmup
    b = DecodeBench(shape, K, W, device, dist, args.prefill_tokens)
    L, B, H, Hkv, d = shape.n_layers, shape.batch, shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    dt, nq, nk, n_in = b.dt, b.nq, b.nk, b.n_in
    b.warm_up()
    t_ms, n_reps, clocks = b.back_to_back(args.reps, local_rank)
    lat_us = b.isolated(max(K, 32))

    # same context every step: window and state of the previous step may still sit in L2
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    hot_ms = []
    for _ in range(5):
        b.make_room(K + 1)
        b.barrier()
        ev0.record()
        for i in range(K):
            b.one_step(b.dev_in[i % n_in], ctx_index=0)
        ev1.record()
        b.barrier()
        hot_ms.append(ev0.elapsed_time(ev1))
    hot_ms = statistics.median(hot_ms)

    # end to end through the public call with HOST buffers: pinned q|k|v -> device, step, out -> pinned host
    host_in = torch.empty((n_in, nq + 2 * nk), dtype=dt).pin_memory()
    host_in.copy_(b.dev_in.cpu())
    host_out = torch.empty((L, B, H, d), dtype=dt).pin_memory()
    stage = torch.empty((nq + 2 * nk,), dtype=dt, device=device)
    e2e_steps = K

    def e2e_step(i):
        stage.copy_(host_in[i % n_in], non_blocking=True)
        b.one_step(stage)
        host_out.copy_(b.outs[(b.step_no - 1) & 1], non_blocking=True)
        torch.cuda.current_stream().synchronize()   # the next token depends on this result

    b.make_room(3)
    for i in range(3):
        e2e_step(i)
    e2e_ms = []
    for _ in range(5):
        b.make_room(math.ceil(e2e_steps / b.n_rep) + 1)
        b.barrier()
        ev0.record()
        for i in range(e2e_steps):
            e2e_step(i)
        ev1.record()
        b.barrier()
        e2e_ms.append(ev0.elapsed_time(ev1))
    e2e_t = statistics.median(e2e_ms)

    per_layer = None
    if world == 1 and b.bytes_io <= (8 << 30):
        b.make_room(3 * K + 8)   # the per-layer pass steps a clone of copy 0 forward 3 + 3 K times
        per_layer = measure_per_layer_launch(b.ctxs[0], shape, b.views(b.dev_in[0]), b.outs[0], K, device)

    t_ms, hot_ms, e2e_t = max_over_ranks([t_ms, hot_ms, e2e_t], dist, device)

    if rank == 0:
        peak, peak_kind = load_peaks()
        launch_s = t_ms * 1e-3 / K
        achieved = b.bytes_stream / launch_s / 1e9
        info = b.ctxs[0].glide_decode_launch_info()
        elem = shape.elem_bytes
        lat = latency_summary(lat_us)
        line = {
            "metric": "hybrid-attn decode tokens/s", "value": whole_job_tokens_per_s(world, B, K, t_ms), "unit": "tokens/s",
            "n_gpus": world, "steps": K, "warmup": b.W, "ms_per_step": t_ms / K, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32" if shape.dtype == "f32" else "bf16+f32state",
            "data": "synthetic",
            "config": workload_config(shape, {
                "l2": f"steps rotate over {b.n_rep} independent state copies ({b.n_rep * b.bytes_io / 1e6:.0f} MB per "
                      f"rotation > 126 MB L2)",
                "timing": f"value = back-to-back throughput: K steps between two events, consecutive launches overlap by "
                          f"programmatic dependent launch; median of {n_reps} repetitions (>= {MIN_TIMED_S} s of timed "
                          f"work); the isolated-step latency is per_step_attention_latency_us"}),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": None if PHI["kind"] else NCU_TRAFFIC_BYTES.get(shape.name), "peak_kind": f"of {peak_kind}",
                         "kernel": decode_kernel_name(shape), "algorithmic_bytes_per_launch": b.bytes_stream,
                         "bytes_formula": "sum over layers and sequences of 2 w H_kv d 2B (window) + S,z read and written",
                         "algorithmic_bytes_incl_io": b.bytes_io,
                         "frac_incl_io": b.bytes_io / launch_s / 1e9 / peak,
                         "frac_of_nominal_8TBps": achieved / 8000.0,
                         "isolated_step_frac": b.bytes_stream / (lat["median"] * 1e-6) / 1e9 / peak},
            "per_step_attention_latency_us": lat["median"],
            "back_to_back_us_per_step": launch_s * 1e6,
            "step_latency_us": lat,
            "hot_l2": {"tokens_per_s": world * B * K / (hot_ms * 1e-3), "us_per_step": hot_ms * 1e3 / K,
                       "note": "same sequence state every step (L2 may hold part of it)"},
            "e2e": {"value": world * B * e2e_steps / (e2e_t * 1e-3), "unit": "tokens/s",
                    "h2d_bytes_per_step": (nq + 2 * nk) * elem, "d2h_bytes_per_step": nq * elem,
                    "us_per_step": e2e_t * 1e3 / e2e_steps},
            "gpu_launches": K * info["launches"],
            "decode_launch": info,
            "clocks": clocks,
        }
        if per_layer is not None:
            per_layer["vs_one_launch_hot_l2"] = per_layer["us_per_step"] / (hot_ms * 1e3 / K)
            line["per_layer_launch"] = per_layer
        if args.prefill_tokens > 0:
            b.rewind(b.n_rep - 1)
            line["prefill"] = measure_prefill(b.ctxs[-1], b.wl, shape, args.prefill_tokens, device)
        b.close()
        if world == 1 and args.side_workloads != "none":
            names = SIDE_WORKLOADS if args.side_workloads == "all" else tuple(args.side_workloads.split(","))
            line["workloads"] = {}
            for name in names:
                if name == shape.name:
                    continue
                try:
                    line["workloads"][name] = side_workload(configs.ALL[name], K, W, device, local_rank,
                                                            prefill_tokens=256 if name.startswith("c3_llama") else 0)
                except torch.OutOfMemoryError as e:   # a device with less memory than the control needs
                    line["workloads"][name] = {"skipped": f"out of device memory: {str(e)[:80]}"}
                    torch.cuda.empty_cache()
        if world == 1 and not args.no_cpu_baseline:
            tok_s, step_s, cores, sample = oracle_decode_rate(shape, 4, 1, single_steps=2)
            line["cpu_baseline"] = {"value": tok_s, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                                    "sample": sample, "ms_per_step": step_s * 1e3}
            step1 = oracle_decode_rate.single_thread_step_s
            line["cpu_baseline"]["single_thread"] = {"value": B / step1, "unit": "tokens/s", "cores": 1,
                                                     "ms_per_step": step1 * 1e3}
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def measure_per_layer_launch(g0, shape, qkv, out, steps, device):
    """The same decode step issued layer by layer through glide_decode_step_layers (one launch per layer, each with
    its own schedule) instead of one launch for the whole stack: what a model pays whose layers depend on each
    other, and what the per-launch overhead costs when the windows are small.  Same sequence state every step,
    so it compares with the one-launch `hot_l2` figure."""
    from paper_2607_24788_b200 import glide
    import ctypes
    L = shape.n_layers
    dt = torch_dtype(shape)
    n = g0.glide_layer_info(0)["n"]
    g = glide.Glide(shape.windows, shape.batch, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, g0.max_tokens,
                    dtype=dt, device=device, prefill_chunk=shape.prefill_chunk, **glide_kwargs(shape, device))
    for l in range(L):
        rk, rv, S, z = g0.glide_export_state(l)
        cap = g.capacity(l)
        g.glide_import_state(l, n, rk if cap else None, rv if cap else None, S, z)
    torch.cuda.synchronize()
    q, k, v = qkv
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # the C entry point with pointers resolved once: the binding's per-call argument checks (tens of microseconds)
    # would otherwise be what is measured
    vp = ctypes.c_void_p
    sptr = vp(torch.cuda.current_stream().cuda_stream or None)
    fn = g.lib.glide_decode_step_layers
    calls = [(l, vp(q[l].data_ptr()), vp(k[l].data_ptr()), vp(v[l].data_ptr()), vp(out[l].data_ptr())) for l in range(L)]

    def launch(l):
        _, a, b, c, o = calls[l]
        if fn(g._h, l, 1, a, b, c, o, sptr) != 0:
            raise RuntimeError("glide_decode_step_layers failed in per-layer mode")

    def step():
        for l in range(L):
            launch(l)

    for _ in range(3):
        step()
    torch.cuda.synchronize()
    res = []
    host_us = []
    for _ in range(3):
        ev0.record()
        h0 = time.perf_counter()
        for _ in range(steps):
            step()
        h1 = time.perf_counter()
        ev1.record()
        torch.cuda.synchronize()
        res.append(ev0.elapsed_time(ev1) * 1e3 / steps)
        host_us.append((h1 - h0) * 1e6 / steps)
    del g
    return {"us_per_step": statistics.median(res), "launches_per_step": L,
            "host_issue_us_per_step": statistics.median(host_us),
            "note": "glide_decode_step_layers, one layer per call, issued back to back; when host_issue_us_per_step is "
                    "about us_per_step the figure is bound by the host issuing launches"}


def measure_prefill(ctx, wl, shape, n_tokens, device):
    """glide_prefill with outputs for n_tokens more tokens on every layer (best of 3, CUDA events)."""
    L, B, H, d = shape.n_layers, shape.batch, shape.n_q_heads, shape.head_dim
    n = ctx.glide_layer_info(0)["n"]
    if n + 3 * n_tokens > ctx.max_tokens:
        return None
    q, k, v = wl.qkv(range(L), range(B), range(n, n + n_tokens), device=device)
    out = torch.empty_like(q)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    best = None
    for _ in range(3):
        ev0.record()
        ctx.glide_prefill(q, k, v, out)
        ev1.record()
        torch.cuda.synchronize()
        ms = ev0.elapsed_time(ev1)
        best = ms if best is None else min(best, ms)
    flops = sum(4.0 * d * H * B * sum(min(w, n + i + 1) for i in range(n_tokens)) for w in shape.windows)
    return {"tokens": n_tokens, "context_before": n, "ms": best, "tokens_per_s": B * n_tokens / (best * 1e-3),
            "window_tflops": flops / (best * 1e-3) / 1e12, "note": "glide_prefill with outputs, all layers, chunked"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--reps", type=int, default=15,
                    help="least number of repetitions of the K-step timed region (median reported; repeated further "
                         "until half a second of timed work has accumulated)")
    ap.add_argument("--min-time", type=float, default=MIN_TIMED_S,
                    help="seconds of timed work a figure accumulates at least (0: just --reps repetitions, for "
                         "profiler captures)")
    ap.add_argument("--side-workloads", default="all",
                    help="'all', 'none' or a comma-separated list: the other configurations and controls timed after "
                         "the headline workload (one GPU only)")
    ap.add_argument("--workload", default=configs.C1.name, choices=sorted(configs.ALL))
    ap.add_argument("--impl", default="glide", choices=["glide", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--prefill-tokens", type=int, default=1024,
                    help="tokens appended by glide_prefill WITH outputs after the decode measurement (0: skip)")
    ap.add_argument("--decode-chunk", type=int, default=0, help="window slots per split-K work item (0: library default)")
    ap.add_argument("--state-splits", type=int, default=0, help="row blocks per state update (0: library default)")
    ap.add_argument("--decode-impl", type=int, default=0,
                    help="0 auto, 1 per-item tensor-core/TMA kernel, 2 CUDA-core kernel, 3 streaming tensor-core/TMA kernel")
    ap.add_argument("--prefill-impl", type=int, default=0, help="0 auto, 1 mma.sync, 2 tcgen05 + TMEM, 3 CUDA cores")
    ap.add_argument("--phi", type=int, default=0,
                    help="0 softmax over the head features (the paper's default), 1 the learned map: d x d projections "
                         "with N(0, 1/d) weights, 2d features")
    ap.add_argument("--merge", type=int, default=0,
                    help="0 shared normaliser (the paper's default), 1 / 2 the appendix' sums of two normalised terms "
                         "(evicted-token / all-token state)")
    args = ap.parse_args()
    shape = configs.ALL[args.workload]
    KERNEL_KNOBS.update(decode_chunk=args.decode_chunk, decode_state_splits=args.state_splits,
                        decode_impl=args.decode_impl, prefill_impl=args.prefill_impl, merge=args.merge)
    PHI["kind"] = args.phi
    globals()["MIN_TIMED_S"] = args.min_time
    if args.impl == "reference":
        run_reference(args, shape)
    else:
        run_glide(args, shape)


if __name__ == "__main__":
    main()
