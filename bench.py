#!/usr/bin/env python
"""Benchmark of the libsdllm hot path: cached-KV tokens/s per layer (refresh + sparse attention).

A "step" is one decoding block of the workload's attention stack: for every layer one refresh
(dense block attention + saliency + pooling, top-k, K/V compaction) followed by the block's
cache-reuse steps (sparse block attention over [K_c ; K_n]), issued in model order (step-major,
layer-minor), so consecutive calls touch different layers' K/V and caches. The dense step 0 of each
block (cache_state 0) is not part of this path; `--phase dense` times it on its own, with its own metric. "Cached-KV tokens" of a call are the
key/value positions it consumes: L for a refresh, n + b for a reuse step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2_llada] [--impl ours|reference]

Prints ONE JSON line (rank 0). `--impl reference` times the CPU oracle on a bounded sample instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2508_02558_b200 import workloads as W

METRIC = "cached_kv_tokens_per_s_per_layer"
UNIT = "tokens/s"
PROFILES = os.path.join(ROOT, "profiles")


def ncu_traffic(kernel: str, workload: str, batch: int):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of the reuse-step kernel `kernel` on `workload`, read from
    the ncu summary under profiles/ (a line "traffic_bytes_per_launch: N"); None when no capture of that kernel on that
    workload exists."""
    stem = kernel.replace("_bf16_kernel", "").replace("_kernel", "")
    path = os.path.join(PROFILES, "%s_%s%s_sparse.txt" % (stem, workload, "_b%d" % batch if batch > 1 else ""))
    if not os.path.exists(path):
        return None, None
    for line in open(path):
        if line.startswith("traffic_bytes_per_launch:"):
            try:
                return int(line.split(":")[1].split()[0]), os.path.relpath(path, ROOT)
            except ValueError:
                return None, None
    return None, None


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2_llada",
                    choices=["c2_llada", "c3_dream", "c4_long", "c5_serving", "c6_gen512", "c7_long4k"])
    ap.add_argument("--retention", type=float, default=None, help="override the workload's retention ratio r")
    ap.add_argument("--pool-window", type=int, default=None, help="override the workload's pooling kernel size (odd)")
    ap.add_argument("--batch", type=int, default=1, help="sequences per call (c5_serving: ragged prompt lengths)")
    ap.add_argument("--phase", default="all", choices=["all", "refresh", "sparse", "dense"],
                    help="profiling aid: run only the refresh chain or only the reuse steps in the timed step; "
                         "dense: time the full-sequence dense step (cache_state 0) of every layer instead, on its own metric")
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (0 = the workload's)")
    ap.add_argument("--no-graph", action="store_true", help="launch eagerly instead of replaying a CUDA graph")
    ap.add_argument("--tune", action="append", default=[], metavar="NAME=VALUE",
                    help="override one decision of the library's launch planner (sdllm_tuning_set), e.g. --tune splits=4")
    ap.add_argument("--no-legs", action="store_true", help="skip the short legs over the other workloads (key 'workloads')")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    return ap.parse_args()


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return float(json.load(open(path))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def tensor_peaks():
    """(burst, sustained) dense bf16 TFLOP/s of a library GEMM on this machine."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        m = json.load(open(path))
        return float(m["bf16_tflops"]), float(m.get("bf16_tflops_sustained", m["bf16_tflops"])), "measured"
    return 1590.0, 1400.0, "fallback"


# ------------------------------------------------------------------------------------------------ workload
def workload_config(args) -> W.WorkloadConfig:
    """The named workload, with the retention ratio and pooling kernel size overridden when asked (perf sweeps)."""
    import dataclasses
    cfg = W.CONFIGS[args.workload]
    if args.retention is not None:
        cfg = dataclasses.replace(cfg, retention=float(args.retention))
    if args.pool_window is not None:
        cfg = dataclasses.replace(cfg, pool_window=int(args.pool_window))
    return cfg


def block_schedule(cfg: W.WorkloadConfig, state_of=None):
    """(dense, refresh, reuse) step counts of one decoding block: cache states 0, 1, 2 of Algorithm 2 over the block's
    denoising steps. `state_of` is the library's sdllm_cache_state (the closed form min(i, 2) where the library is not
    loaded: the CPU arm)."""
    state_of = state_of or (lambda i: min(i, 2))
    states = [state_of(i) for i in range(cfg.steps_per_block)]
    return states.count(0), states.count(1), states.count(2)


def tokens_per_step(cfg: W.WorkloadConfig, n_layers: int, seq_lens, n_keeps, phase: str = "all") -> int:
    reuse_steps = block_schedule(cfg)[2]
    refresh = sum(seq_lens) if phase in ("all", "refresh") else 0
    sparse = reuse_steps * sum(n + cfg.block_len for n in n_keeps) if phase in ("all", "sparse") else 0
    return n_layers * (refresh + sparse)


def algorithmic_bytes(cfg: W.WorkloadConfig, seq_lens, n_keeps):
    """Bytes each call must move (K and V once, Q and O once, scores / indices), per layer, summed over the batch."""
    e = 2 if cfg.dtype == "bf16" else 4
    b, Hq, Hkv, D = cfg.block_len, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    out = {"refresh": 0, "topk": 0, "compact": 0, "sparse": 0}
    for L, n_keep in zip(seq_lens, n_keeps):
        out["refresh"] += 2 * L * Hkv * D * e + 2 * b * Hq * D * e + 4 * (L - b) * Hkv
        out["topk"] += 4 * (L - b) * Hkv + 4 * n_keep * Hkv
        out["compact"] += 2 * (2 * n_keep * Hkv * D * e) + 4 * n_keep * Hkv
        out["sparse"] += 2 * (n_keep + b) * Hkv * D * e + 2 * b * Hq * D * e
    return out


class ClockSampler:
    """Samples the SM clock and the clock-event (throttle) reasons of one GPU while timed regions run: a thread polls NVML
    every few milliseconds (read-only queries), and only the samples that fall inside a region marked with begin() /
    end() count. Falls back to an `nvidia-smi -lms` child process when the NVML binding is missing."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    BITS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown"}
    active = None                 # the sampler that timed regions report to

    def __init__(self, index: int):
        self.samples, self.windows, self._t0 = [], [], None
        self.proc = self.file = self.thread = None
        self.max_mhz = None
        try:
            import pynvml
            import threading
            pynvml.nvmlInit()
            self.nv = pynvml
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            self._stop = threading.Event()
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
        except Exception:
            self.thread = None
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            try:
                self.proc = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                              "-lms", "100"], stdout=self.file, stderr=subprocess.DEVNULL)
            except OSError:
                self.proc = None
        ClockSampler.active = self

    def _poll(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                mhz = float(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM))
                try:
                    why = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
                except Exception:
                    why = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
                self.samples.append((time.perf_counter(), mhz, why))
            except Exception:
                pass
            self._stop.wait(0.002)

    def begin(self):
        self._t0 = time.perf_counter()

    def end(self):
        if self._t0 is not None:
            self.windows.append((self._t0, time.perf_counter()))
            self._t0 = None

    def stop(self):
        if ClockSampler.active is self:
            ClockSampler.active = None
        if self.thread is not None:
            self._stop.set()
            self.thread.join(timeout=2)
            inside = [(m, w) for (t, m, w) in self.samples if any(a <= t <= b for a, b in self.windows)] if self.windows else \
                     [(m, w) for (_, m, w) in self.samples]
            reasons = sorted({name for _, w in inside for bit, name in self.BITS.items() if w & bit})
            return {"sm_mhz": statistics.median([m for m, _ in inside]) if inside else None, "sm_max_mhz": self.max_mhz,
                    "samples": len(inside), "reasons": reasons, "source": "nvml, polled every 2 ms inside the timed regions"}
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.file.flush(); self.file.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.file.read().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(n)
        os.unlink(self.file.name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons), "source": "nvidia-smi -lms 100"}


# ------------------------------------------------------------------------------------------------ per-call timing
LEGS = [  # (workload, batch, retention override, pool window override, layers rotated so that the working set exceeds L2)
    ("c3_dream", 1, None, None, 28),
    ("c4_long", 1, 0.1, 3, 3), ("c4_long", 1, 0.25, 3, 3), ("c4_long", 1, 0.5, 3, 3), ("c4_long", 1, 0.5, 1, 3), ("c4_long", 1, 0.5, 7, 3),
    ("c5_serving", 1, None, None, 8), ("c5_serving", 4, None, None, 2), ("c5_serving", 16, None, None, 1),
]


def time_calls(torch, dev, cfg, Bn, n_layers, rank, peak, steps=5, n_step_sets=4, sampler_index=None):
    """Times every call of the path on its own for one workload: the refresh-step attention, top-k, compaction, the two
    fused in one call, the whole refresh chain and the reuse step, each replayed from a CUDA graph over `n_layers` sets
    of buffers (together larger than L2). Returns microseconds per call and the fraction of the HBM roof."""
    import dataclasses
    from paper_2508_02558_b200 import binding as B
    from paper_2508_02558_b200.session import LayerCache
    Hq, Hkv, D, b = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.block_len
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    bdt = B.BF16 if cfg.dtype == "bf16" else B.F32

    def to_dev(x):
        if cfg.dtype == "bf16":
            return torch.from_numpy(W.f32_to_bf16_bits(x).reshape(x.shape).view(np.int16)).view(torch.bfloat16).to(dev)
        return torch.from_numpy(x).to(dev)
    prompt_lens = W.serving_prompt_lengths(Bn, seed=5 + rank) if cfg.name == "c5_serving" else [cfg.prompt_len] * Bn
    seq_lens = [p_ + cfg.gen_len for p_ in prompt_lens]
    L = max(seq_lens)
    caches, Ks, Vs, Qr, Qs, Kn, Vn = [], [], [], [], [], [], []
    gen = torch.Generator(device=dev); gen.manual_seed(99 + rank)
    drift = cfg.drift_std / np.sqrt(D)
    for l in range(n_layers):
        bw = W.make_batch(cfg, prompt_lens, seed=rank, layer=l, block=0)
        q, k, v = bw.refresh_inputs(1)
        Ks.append(to_dev(k)); Vs.append(to_dev(v)); Qr.append(to_dev(q))
        caches.append(LayerCache(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, seq_len_max=L, block_len=b, dtype=bdt,
                                 retention=cfg.retention, pool_window=cfg.pool_window, device=str(dev),
                                 share_scratch_with=caches[0] if caches else None))
        rows = torch.stack([torch.arange(o_, o_ + b, device=dev) for o_ in prompt_lens])
        gather = rows[:, None, :, None].expand(Bn, Hkv, b, D)
        kb, vb = Ks[l].gather(2, gather).float(), Vs[l].gather(2, gather).float()
        Qs.append([(Qr[l].float() + drift * torch.randn(Qr[l].shape, device=dev, generator=gen)).to(tdt) for _ in range(n_step_sets)])
        Kn.append([(kb + drift * torch.randn(kb.shape, device=dev, generator=gen)).to(tdt) for _ in range(n_step_sets)])
        Vn.append([(vb + drift * torch.randn(vb.shape, device=dev, generator=gen)).to(tdt) for _ in range(n_step_sets)])
    d0 = caches[0].desc
    n_keeps = [B.keep_count(d0, Li, pi)[0] for Li, pi in zip(seq_lens, prompt_lens)]
    sl = torch.tensor(seq_lens, dtype=torch.int32, device=dev)
    bo = torch.tensor(prompt_lens, dtype=torch.int32, device=dev)
    out_r = [torch.empty((Bn, Hq, b, D), dtype=tdt, device=dev) for _ in range(n_layers)]
    out_s = [torch.empty((Bn, Hq, b, D), dtype=tdt, device=dev) for _ in range(n_layers)]
    stream = torch.cuda.Stream(device=dev)
    torch.cuda.synchronize(dev)

    def graph_time(fn, calls):
        with torch.cuda.stream(stream):
            fn()
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            fn()
        with torch.cuda.stream(stream):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(3):
                g.replay()
            e1.record(stream)
            stream.synchronize()
            # at least `steps` replays, and enough of them for about 30 ms: the clock sampler polls every few milliseconds
            n_rep = max(steps, min(2000, int(0.03 / max(e0.elapsed_time(e1) / 3e3, 1e-6)) + 1))
            if ClockSampler.active:
                ClockSampler.active.begin()
            e0.record(stream)
            for _ in range(n_rep):
                g.replay()
            e1.record(stream)
            stream.synchronize()
            if ClockSampler.active:
                ClockSampler.active.end()
        return e0.elapsed_time(e1) * 1e3 / n_rep / calls

    c = caches
    ops = {
        "refresh_chain": (lambda: [c[l].refresh(Qr[l], Ks[l], Vs[l], sl, bo, out=out_r[l], stream=stream) for l in range(n_layers)], n_layers),
        "refresh": (lambda: [B.refresh_scores(c[l].desc, Qr[l], Ks[l], Vs[l], sl, bo, out_r[l], None, c[l].pooled, c[l].workspace, stream)
                             for l in range(n_layers)], n_layers),
        "topk": (lambda: [B.select_topk(c[l].desc, c[l].pooled, sl, bo, c[l].kept_idx, c[l].kept_cnt, None, stream) for l in range(n_layers)], n_layers),
        "compact": (lambda: [B.compact_kv(c[l].desc, Ks[l], Vs[l], c[l].kept_idx, c[l].kept_cnt, c[l].k_c, c[l].v_c, stream)
                             for l in range(n_layers)], n_layers),
        "select_compact": (lambda: [B.select_compact(c[l].desc, c[l].pooled, sl, bo, Ks[l], Vs[l], c[l].kept_idx, c[l].kept_cnt, c[l].k_c,
                                                     c[l].v_c, stream) for l in range(n_layers)], n_layers),
        "reuse": (lambda: [c[l].sparse_step(Qs[l][t], Kn[l][t], Vn[l][t], out_s[l], stream=stream)
                           for t in range(n_step_sets) for l in range(n_layers)], n_layers * n_step_sets),
    }
    sampler = ClockSampler(sampler_index) if sampler_index is not None else None
    us = {}
    for name in ("refresh_chain", "refresh", "topk", "compact", "select_compact", "reuse"):   # the chain first: it fills every cache
        us[name] = graph_time(*ops[name])
    clocks = sampler.stop() if sampler else None
    ab = algorithmic_bytes(cfg, seq_lens, n_keeps)
    ab["refresh_chain"] = ab["refresh"] + ab["topk"] + ab["compact"]
    ab["select_compact"] = ab["topk"] + ab["compact"]
    ab["reuse"] = ab["sparse"]
    rec = {"workload": cfg.name, "batch": Bn, "retention": cfg.retention, "pool_window": cfg.pool_window, "layers_rotated": n_layers,
           "seq_len_max": L, "n_keep_max": max(n_keeps), "fused_select_compact": B.launch_count(d0, B.OP_SELECT_COMPACT) == 1}
    for name in us:
        rec[name + "_us"] = round(us[name], 3)
        rec["frac_" + name] = round(ab[name] / (us[name] * 1e-6) / 1e9 / peak, 4)
    rec["clocks"] = clocks
    del caches, Ks, Vs, Qr, Qs, Kn, Vn
    torch.cuda.empty_cache()
    return rec


def run_legs(torch, dev, rank, peak, local):
    """Short legs over the workloads that are not the headline: one record per (workload, batch, retention, window)."""
    import dataclasses
    out = []
    for name, Bn, r, s_, layers in LEGS:
        cfg = W.CONFIGS[name]
        if r is not None:
            cfg = dataclasses.replace(cfg, retention=r)
        if s_ is not None:
            cfg = dataclasses.replace(cfg, pool_window=s_)
        out.append(time_calls(torch, dev, cfg, Bn, layers, rank, peak, sampler_index=local))
    return out


# ------------------------------------------------------------------------------------------------ CPU oracle arm
def oracle_block_sample(cfg: W.WorkloadConfig, seed: int):
    """One layer x one decoding block through the CPU oracle: 1 refresh + the block's reuse steps. Returns (tokens, seconds)."""
    import oracle
    s = W.make_sequence(cfg, seed=seed, layer=0, block=0)
    q, k, v = s.refresh_inputs(1)
    steps = [s.sparse_inputs(i) for i in range(2, cfg.steps_per_block)]
    t0 = time.perf_counter()
    r = oracle.refresh(q, k, v, s.block_off, cfg.retention, cfg.pool_window)
    k_c, v_c = oracle.gather_rows(k, r.kept_idx), oracle.gather_rows(v, r.kept_idx)
    for q2, kn, vn in steps:
        oracle.sparse_block_attention(q2, k_c, v_c, kn, vn)
    dt = time.perf_counter() - t0
    return cfg.seq_len + len(steps) * (r.n_keep + cfg.block_len), dt


def oracle_one_thread(workload: str):
    """The same bounded oracle sample on ONE host thread (a child process with OMP_NUM_THREADS=1, the oracle untouched)."""
    env = dict(os.environ, OMP_NUM_THREADS="1")
    try:
        res = subprocess.run([sys.executable, os.path.abspath(__file__), "--impl", "reference", "--workload", workload, "--steps", "1",
                              "--warmup", "1"], env=env, capture_output=True, text=True, timeout=240)
        line = json.loads(res.stdout.strip().splitlines()[-1])
        return {"value": line["value"], "unit": UNIT, "cores": 1, "sample": line["config"]["sample"]}
    except Exception as e:                      # the figure is reported context: never let it take the run down
        return {"value": None, "error": repr(e)[:200]}


def oracle_other_workloads():
    """Bounded oracle samples of the other configurations: the tiny config whole, one refresh + 2 reuse steps of one
    long-context point and of the serving batches (cached-KV tokens per second, all host threads)."""
    import dataclasses
    import oracle
    out = []
    jobs = [("c1_tiny", 1, None, 3), ("c3_dream", 1, None, 2), ("c4_long", 1, 0.5, 2), ("c5_serving", 1, None, 2), ("c5_serving", 4, None, 2),
            ("c5_serving", 16, None, 1)]
    for name, Bn, r, n_reuse in jobs:
        cfg = W.CONFIGS[name]
        if r is not None:
            cfg = dataclasses.replace(cfg, retention=r)
        lens = W.serving_prompt_lengths(Bn, seed=5) if name == "c5_serving" else [cfg.prompt_len] * Bn
        bw = W.make_batch(cfg, lens, seed=0)
        steps = [bw.sparse_inputs(i) for i in range(2, 2 + n_reuse)]
        q, k, v = bw.refresh_inputs(1)
        tok, t0 = 0, time.perf_counter()
        for i, sq in enumerate(bw.seqs):
            Li, o = sq.seq_len, sq.block_off
            res = oracle.refresh(q[i], k[i, :, :Li], v[i, :, :Li], o, cfg.retention, cfg.pool_window)
            k_c, v_c = oracle.gather_rows(k[i, :, :Li], res.kept_idx), oracle.gather_rows(v[i, :, :Li], res.kept_idx)
            tok += Li
            for q2, kn, vn in steps:
                oracle.sparse_block_attention(q2[i], k_c, v_c, kn[i], vn[i])
                tok += res.n_keep + cfg.block_len
        sec = time.perf_counter() - t0
        out.append({"workload": name, "batch": Bn, "retention": cfg.retention, "value": tok / sec, "unit": UNIT, "cores": omp_threads(),
                    "seconds": round(sec, 3), "sample": "1 layer: 1 refresh + %d reuse steps" % n_reuse})
    return out


def omp_threads() -> int:
    env = os.environ.get("OMP_NUM_THREADS")
    return int(env) if env else len(os.sched_getaffinity(0))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = workload_config(args)
    import oracle
    oracle.build()
    for i in range(args.warmup):
        oracle_block_sample(cfg, seed=1000 + i) if i == 0 else None      # one warm pass is enough for a CPU loop
    tok, sec = 0, 0.0
    for i in range(args.steps):
        t, s = oracle_block_sample(cfg, seed=i)
        tok += t; sec += s
    value = tok / sec
    sample = "per step: 1 layer x 1 block (1 refresh + %d reuse steps) of %s" % (cfg.steps_per_block - 2, cfg.name)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * sec / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": omp_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------------------------------------ replicas over ranks
def slowest_rank_seconds(sec: float, device=None) -> float:
    """Timed seconds of the slowest rank (the ranks run independent replicas: no data-path collective)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return sec
    t = torch.tensor([sec], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(tokens_per_rank: float, world: int, slowest_sec: float) -> float:
    """Whole-job throughput: every rank processed tokens_per_rank in at most slowest_sec."""
    return world * tokens_per_rank / slowest_sec


# ------------------------------------------------------------------------------------------------ CUDA arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2508_02558_b200 import binding as B
    from paper_2508_02558_b200.session import LayerCache

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: libsdllm has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    B.lib()
    for item in args.tune:
        name, _, val = item.partition("=")
        B.tuning_set(name, int(val))

    cfg = workload_config(args)
    n_layers = args.layers or cfg.n_layers
    Hq, Hkv, D, b = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.block_len
    n_dense, n_refresh, reuse_steps = block_schedule(cfg, B.cache_state)      # Algorithm 2: 1 dense, 1 refresh, 30 reuse
    assert n_refresh == 1
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    bdt = B.BF16 if cfg.dtype == "bf16" else B.F32

    def to_dev(x):
        if cfg.dtype == "bf16":
            return torch.from_numpy(W.f32_to_bf16_bits(x).reshape(x.shape).view(np.int16)).view(torch.bfloat16).to(dev)
        return torch.from_numpy(x).to(dev)

    # ---- inputs: base tensors from the seeded host generator (one (layer, block=0) each); per-step drift on the device
    Bn = max(1, args.batch)
    if cfg.name == "c5_serving":
        prompt_lens = W.serving_prompt_lengths(Bn, seed=5 + rank)
    else:
        prompt_lens = [cfg.prompt_len] * Bn
    seq_lens = [p_ + cfg.gen_len for p_ in prompt_lens]
    L = max(seq_lens)
    caches, Ks, Vs, Qr = [], [], [], []
    gen = torch.Generator(device=dev); gen.manual_seed(1234 + rank)
    for l in range(n_layers):
        bw = W.make_batch(cfg, prompt_lens, seed=rank, layer=l, block=0)
        q, k, v = bw.refresh_inputs(1)
        Ks.append(to_dev(k)); Vs.append(to_dev(v)); Qr.append(to_dev(q))
        caches.append(LayerCache(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, seq_len_max=L, block_len=b, dtype=bdt,
                                 retention=cfg.retention, pool_window=cfg.pool_window, device=str(dev),
                                 share_scratch_with=caches[0] if caches else None))
    # one allocation per kind, the per-layer tensors are views of it: the end-to-end leg refills them with one copy each
    K_all, V_all, Q_all = torch.stack(Ks), torch.stack(Vs), torch.stack(Qr)
    Ks, Vs, Qr = list(K_all.unbind(0)), list(V_all.unbind(0)), list(Q_all.unbind(0))
    n_keeps = [B.keep_count(caches[0].desc, Li, pi)[0] for Li, pi in zip(seq_lens, prompt_lens)]
    n_keep = max(n_keeps)
    seq_len_t = torch.tensor(seq_lens, dtype=torch.int32, device=dev)
    block_off = torch.tensor(prompt_lens, dtype=torch.int32, device=dev)
    drift = cfg.drift_std / np.sqrt(D)
    # fresh block rows for every (reuse step, layer): Q_b', K_n, V_n = base + drift, rounded to the compute dtype
    Qs = torch.empty((reuse_steps, n_layers, Bn, Hq, b, D), dtype=tdt, device=dev)
    Kn = torch.empty((reuse_steps, n_layers, Bn, Hkv, b, D), dtype=tdt, device=dev)
    Vn = torch.empty_like(Kn)
    rows = torch.stack([torch.arange(o_, o_ + b, device=dev) for o_ in prompt_lens])          # [B, b] block positions
    gather = rows[:, None, :, None].expand(Bn, Hkv, b, D)
    for l in range(n_layers):
        kb, vb = Ks[l].gather(2, gather).float(), Vs[l].gather(2, gather).float()
        for t in range(reuse_steps):
            Qs[t, l] = (Qr[l].float() + drift * torch.randn(Qr[l].shape, device=dev, generator=gen)).to(tdt)
            Kn[t, l] = (kb + drift * torch.randn((Bn, Hkv, b, D), device=dev, generator=gen)).to(tdt)
            Vn[t, l] = (vb + drift * torch.randn((Bn, Hkv, b, D), device=dev, generator=gen)).to(tdt)
    out_r = torch.empty((n_layers, Bn, Hq, b, D), dtype=tdt, device=dev)
    out_s = torch.empty((reuse_steps, n_layers, Bn, Hq, b, D), dtype=tdt, device=dev)

    stream = torch.cuda.Stream(device=dev)
    torch.cuda.synchronize(dev)                     # the inputs above were produced on the default stream

    def one_step():
        """One decoding block: refresh every layer, then every reuse step over every layer (model order)."""
        for l in range(n_layers):
            caches[l].refresh(Qr[l], Ks[l], Vs[l], seq_len_t, block_off, out=out_r[l], stream=stream)
        for t in range(reuse_steps):
            for l in range(n_layers):
                caches[l].sparse_step(Qs[t, l], Kn[t, l], Vn[t, l], out_s[t, l], stream=stream)

    def sparse_only():
        for t in range(reuse_steps):
            for l in range(n_layers):
                caches[l].sparse_step(Qs[t, l], Kn[t, l], Vn[t, l], out_s[t, l], stream=stream)

    def refresh_only():
        for l in range(n_layers):
            caches[l].refresh(Qr[l], Ks[l], Vs[l], seq_len_t, block_off, out=out_r[l], stream=stream)

    def make_runner(fn):
        if args.no_graph:
            return fn
        with torch.cuda.stream(stream):
            fn()                                    # first eager call sets kernel attributes outside the capture
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            fn()
        return graph.replay

    def timed(runner, iters, warm):
        with torch.cuda.stream(stream):
            for _ in range(warm):
                runner()
            stream.synchronize()
            if world > 1:
                dist.barrier()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            if ClockSampler.active:
                ClockSampler.active.begin()
            e0.record(stream)
            for _ in range(iters):
                runner()
            e1.record(stream)
            torch.cuda.synchronize()
            if ClockSampler.active:
                ClockSampler.active.end()
            if world > 1:
                dist.barrier()
        return e0.elapsed_time(e1) / 1e3

    if args.phase == "dense":
        # ---- the dense step on its own: every row of every sequence over all of its keys, layer after layer
        nq = min(n_layers, max(1, int(4e9 // (2 * Bn * Hq * L * D * 2))))        # distinct Q / output sets (a few GB)
        inv = 1.0 / np.sqrt(D)
        Qf = [(torch.randn((Bn, Hq, L, D), device=dev, generator=gen) * inv).to(tdt) for _ in range(nq)]
        Of = [torch.empty((Bn, Hq, L, D), dtype=tdt, device=dev) for _ in range(nq)]
        torch.cuda.synchronize(dev)

        def dense_only():
            for l in range(n_layers):
                caches[l].dense_step(Qf[l % nq], Ks[l], Vs[l], seq_len_t, Of[l % nq], stream=stream)
        sampler = ClockSampler(local) if rank == 0 else None
        sec = slowest_rank_seconds(timed(make_runner(dense_only), args.steps, max(args.warmup, 3)), dev)
        clocks = sampler.stop() if sampler else None
        flops = 4.0 * sum(float(x) * x for x in seq_lens) * Hq * D * n_layers
        burst, sustained, kind = tensor_peaks()
        tflops = world * flops * args.steps / sec / 1e12
        per_gpu = tflops / world
        if rank == 0:
            print(json.dumps({
                "metric": "dense_step_query_tokens_per_s_per_layer", "value": whole_job_value(sum(seq_lens) * n_layers * args.steps, world, sec),
                "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": 1e3 * sec / args.steps,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
                "config": {"workload": cfg.name, "batch": Bn, "phase": "dense", "layers": n_layers, "seq_len": L, "n_q_heads": Hq,
                           "n_kv_heads": Hkv, "head_dim": D, "step": "the dense step (all rows x all keys) of %d layers" % n_layers,
                           "launch": "eager" if args.no_graph else "cuda_graph_replay", "parallelism": "replicas" if world > 1 else "1gpu"},
                "roofline": {"bound": "tensor", "kernel": "sdllm_dense_attn (dense_attn_bf16_kernel: tcgen05, two 128-row query tiles per CTA share one pass over K/V)",
                             "achieved": per_gpu, "peak": sustained, "peak_kind": kind + ", sustained library GEMM", "unit": "TFLOP/s",
                             "frac": per_gpu / sustained, "frac_of_burst": per_gpu / burst, "flops_per_step": flops,
                             "us_per_launch": 1e6 * sec / args.steps / n_layers, "traffic": None},
                "clocks": clocks, "gpu_launches": n_layers * B.launch_count(caches[0].desc, B.OP_DENSE_ATTN) * args.steps,
            }))
        if world > 1:
            dist.destroy_process_group()
        return

    with torch.cuda.stream(stream):
        refresh_only()                              # every layer's cache exists before any reuse step runs
    stream.synchronize()
    d0 = caches[0].desc
    refresh_launches = B.launch_count(d0, B.OP_REFRESH_SCORES) + B.launch_count(d0, B.OP_SELECT_COMPACT)
    sparse_launches = reuse_steps * B.launch_count(d0, B.OP_SPARSE_BLOCK_ATTN)
    launches_per_step = n_layers * ((refresh_launches if args.phase in ("all", "refresh") else 0) +
                                    (sparse_launches if args.phase in ("all", "sparse") else 0))
    step_runner = make_runner({"all": one_step, "refresh": refresh_only, "sparse": sparse_only}[args.phase])
    sampler = ClockSampler(local) if rank == 0 else None
    sec = timed(step_runner, args.steps, max(args.warmup, 3))
    clocks = sampler.stop() if sampler else None
    sec = slowest_rank_seconds(sec, dev)
    tok = tokens_per_step(cfg, n_layers, seq_lens, n_keeps, args.phase)
    value = whole_job_value(tok * args.steps, world, sec)

    # ---- roofline of the dominant call (sparse block attention: 30 of the 31 calls per layer per block)
    ab = algorithmic_bytes(cfg, seq_lens, n_keeps)
    sp_runner = make_runner(sparse_only)
    sp_sec = timed(sp_runner, max(3, args.steps // 2), 3) / max(3, args.steps // 2) / (n_layers * reuse_steps)
    rf_runner = make_runner(refresh_only)
    rf_sec = timed(rf_runner, max(3, args.steps // 2), 3) / max(3, args.steps // 2) / n_layers
    peak, peak_kind = peaks()
    achieved = ab["sparse"] / sp_sec / 1e9
    plan_text = B.plan_describe(caches[0].desc, B.OP_SPARSE_BLOCK_ATTN)      # what the library will launch for this call
    traffic, traffic_file = ncu_traffic(plan_text.split()[0], cfg.name, Bn)
    roofline = {"bound": "hbm", "kernel": "sdllm_sparse_block_attn (%s)" % plan_text,
                "achieved": achieved,
                "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                "frac_of_8TBps": achieved / 8000.0, "algorithmic_bytes_per_launch": ab["sparse"], "us_per_launch": sp_sec * 1e6,
                "traffic": traffic, "traffic_source": traffic_file,
                "refresh_chain": {"us_per_layer": rf_sec * 1e6, "algorithmic_bytes": ab["refresh"] + ab["topk"] + ab["compact"],
                                  "achieved": (ab["refresh"] + ab["topk"] + ab["compact"]) / rf_sec / 1e9,
                                  "frac": (ab["refresh"] + ab["topk"] + ab["compact"]) / rf_sec / 1e9 / peak}}
    # every call of the path on its own, for the headline workload and (default run) for the other configurations
    per_call = None
    legs = None
    if rank == 0 and world == 1 and not args.no_legs:
        per_call = time_calls(torch, dev, cfg, Bn, min(n_layers, 8 if Bn == 1 else 2), rank, peak, sampler_index=local)
        roofline["calls"] = {k: per_call[k] for k in per_call if k.endswith("_us") or k.startswith("frac_")}
        if args.workload == "c2_llada" and args.batch == 1 and args.retention is None and args.pool_window is None:
            legs = run_legs(torch, dev, rank, peak, local)

    # ---- end to end: inputs start in pinned host memory, results are read back, every step
    e2e = None
    if not args.no_e2e:
        hK, hV, hQ = K_all.cpu().pin_memory(), V_all.cpu().pin_memory(), Q_all.cpu().pin_memory()
        hQs, hKn, hVn = Qs.cpu().pin_memory(), Kn.cpu().pin_memory(), Vn.cpu().pin_memory()
        h_out_r, h_out_s = out_r.cpu().pin_memory(), out_s.cpu().pin_memory()

        # Two sets of device buffers: while step i runs from one set, the copy stream fills the other with step i + 1's
        # inputs and a third stream brings step i - 1's outputs back. Every step's inputs still cross PCIe inside the
        # timed region, every output is read back; the library is driven exactly as in the device-resident measurement.
        def fresh_like(t):
            return torch.empty_like(t)
        sets = [dict(Q=Q_all, K=K_all, V=V_all, Qs=Qs, Kn=Kn, Vn=Vn, out_r=out_r, out_s=out_s, run=step_runner)]
        if args.phase == "all":
            s2 = dict(Q=fresh_like(Q_all), K=fresh_like(K_all), V=fresh_like(V_all), Qs=fresh_like(Qs), Kn=fresh_like(Kn), Vn=fresh_like(Vn),
                      out_r=fresh_like(out_r), out_s=fresh_like(out_s))

            def step_on_second_set():
                for l in range(n_layers):
                    caches[l].refresh(s2["Q"][l], s2["K"][l], s2["V"][l], seq_len_t, block_off, out=s2["out_r"][l], stream=stream)
                for t in range(reuse_steps):
                    for l in range(n_layers):
                        caches[l].sparse_step(s2["Qs"][t, l], s2["Kn"][t, l], s2["Vn"][t, l], s2["out_s"][t, l], stream=stream)
            s2["run"] = make_runner(step_on_second_set)
            sets.append(s2)
        h_outs = [(h_out_r, h_out_s)] + [(h_out_r.clone().pin_memory(), h_out_s.clone().pin_memory()) for _ in sets[1:]]
        copy_in, copy_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        ev_in = [torch.cuda.Event() for _ in sets]      # the set's inputs have arrived
        ev_run = [torch.cuda.Event() for _ in sets]     # the step on the set has finished
        ev_out = [torch.cuda.Event() for _ in sets]     # the set's outputs are on the host
        torch.cuda.synchronize(dev)
        step_no = [0]

        def e2e_step():
            i = step_no[0] % len(sets); step_no[0] += 1
            x = sets[i]
            copy_in.wait_event(ev_run[i])                # the set's previous step no longer reads its inputs
            with torch.cuda.stream(copy_in):
                x["Q"].copy_(hQ, non_blocking=True); x["K"].copy_(hK, non_blocking=True); x["V"].copy_(hV, non_blocking=True)
                x["Qs"].copy_(hQs, non_blocking=True); x["Kn"].copy_(hKn, non_blocking=True); x["Vn"].copy_(hVn, non_blocking=True)
                ev_in[i].record(copy_in)
            stream.wait_event(ev_in[i])
            stream.wait_event(ev_out[i])                 # the set's previous outputs have left
            with torch.cuda.stream(stream):
                x["run"]()
                ev_run[i].record(stream)
            copy_out.wait_event(ev_run[i])
            with torch.cuda.stream(copy_out):
                h_outs[i][0].copy_(x["out_r"], non_blocking=True); h_outs[i][1].copy_(x["out_s"], non_blocking=True)
                ev_out[i].record(copy_out)

        def e2e_run(iters):
            copy_in.wait_stream(stream); copy_out.wait_stream(stream)      # nothing starts ahead of the timed region
            for _ in range(iters):
                e2e_step()
            stream.wait_stream(copy_in); stream.wait_stream(copy_out)      # the timed region ends when the last output is back
        e2e_iters = max(2, min(args.steps, 6))
        e2e_run(2)                                       # warm-up: both sets, all three streams
        torch.cuda.synchronize(dev)
        e2e_sec = timed(lambda: e2e_run(e2e_iters), 1, 0)
        e2e_sec = slowest_rank_seconds(e2e_sec, dev)
        esz = Ks[0].element_size()
        h2d = n_layers * Bn * ((2 * Hkv * L * D + Hq * b * D) * esz + reuse_steps * (2 * Hkv * b * D + Hq * b * D) * esz)
        d2h = n_layers * Bn * (1 + reuse_steps) * Hq * b * D * esz
        e2e = {"value": whole_job_value(tok * e2e_iters, world, e2e_sec), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "ms_per_step": 1e3 * e2e_sec / e2e_iters, "steps": e2e_iters,
               "overlap": "double-buffered: copies of step i+1 and i-1 run beside step i" if len(sets) > 1 else "none"}

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        oracle.build()
        oracle_block_sample(cfg, seed=99)            # warm the caches and the OpenMP pool
        ctok, csec = oracle_block_sample(cfg, seed=0)
        cpu_baseline = {"value": ctok / csec, "unit": UNIT, "cores": omp_threads(), "kind": "oracle", "seconds": csec,
                        "sample": "1 layer x 1 block (1 refresh + %d reuse steps) of %s, fp64" % (reuse_steps, cfg.name)}
        if legs is not None:
            cpu_baseline["one_thread"] = oracle_one_thread(cfg.name)
            cpu_baseline["other_workloads"] = oracle_other_workloads()

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": 1e3 * sec / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": cfg.dtype, "data": "synthetic",
            "config": {"workload": cfg.name, "batch": Bn, "phase": args.phase, "layers": n_layers, "seq_len": L, "block_len": b, "n_q_heads": Hq, "n_kv_heads": Hkv,
                       "head_dim": D, "retention": cfg.retention, "pool_window": cfg.pool_window, "n_keep": n_keep,
                       "step": "1 decoding block: %d layers x (1 refresh chain + %d reuse steps)" % (n_layers, reuse_steps),
                       "l2": "no flush: one step streams %.0f MB of K/V and caches across layers, larger than L2" % (
                           n_layers * (ab["refresh"] + ab["compact"] / 2) / 1e6),
                       "launch": "eager" if args.no_graph else "cuda_graph_replay", "parallelism": "replicas" if world > 1 else "1gpu"},
            "block_steps_per_s": world * n_layers * (1 + reuse_steps) * args.steps / sec,
            "roofline": roofline, "workloads": legs, "cpu_baseline": cpu_baseline, "e2e": e2e, "clocks": clocks,
            "gpu_launches": launches_per_step * args.steps,
        }))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
