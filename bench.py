"""Benchmark of the LVSpec verify step on B200.

A "step" is one pass of the whole hot path over one batch of synthetic input:
the verification attention of every layer of the model-shaped config (each
layer with its own K/V cache), then the loose acceptance pass over the target
logits fed by the last layer's visual mass.

    python bench.py --gpus N --steps K --warmup W [--config ID] [--impl reference]

prints one JSON line.  The path does not shard ("replicas only"): with N > 1
every rank runs the same workload on its own GPU, no collective on the data
path; the value is the sum over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "verified draft tokens/sec per verify step"
UNIT = "tokens/s"


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, help="workload config id (1, 2 or 3)")
    ap.add_argument("--kernel", type=int, default=0, help="attention kernel selector (0 = default)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch layer by layer, no CUDA graph")
    ap.add_argument("--fp8-cache", action="store_true",
                    help="run the step on an fp8 (E4M3) cache with one scale per KV head: the config's caches "
                         "quantised on the device, lvspec_verify_attention_fp8 in every layer (the roofline then "
                         "counts one byte per cache element); not the default workload")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the timing of configs 3 and 1 that the default (config 2) run adds to its line")
    ap.add_argument("--no-next-rows", action="store_true",
                    help="skip the timing of the paper's own relevance score (not part of the step)")
    ap.add_argument("--sweep", action="store_true",
                    help="run the head-shape sweep (workload config 4): gamma x KV length x batch, one layer "
                         "per point; the JSON line then carries the per-point table under \"sweep\"")
    ap.add_argument("--lam", type=float, default=None,
                    help="loosening ratio lambda of the rule (the config's 0.7 by default; the paper's "
                         "sensitivity table runs 0.0, 0.2, 0.5, 0.7, 0.9)")
    ap.add_argument("--top-n", type=int, default=10,
                    help="N of the cosine Top-N relevance score timed beside the step (the paper runs 1, 10, 100)")
    ap.add_argument("--layers", type=int, default=0,
                    help="override the config's layer count (a smaller case of the same kernel for "
                         "profiler captures; the line then says so and is not a bench value)")
    return ap.parse_args()


# --------------------------------------------------------------------------- #
# clocks
# --------------------------------------------------------------------------- #
class ClockSampler:
    """Samples the SM clock and the throttle reasons while the timed region runs.
    Reads only: NVML queries every few milliseconds (nvidia-smi as a fallback,
    which is slower per sample)."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int):
        self.index = index
        self.samples = []          # (sm_mhz, max_mhz, [bool per NAMES])
        self._stop = threading.Event()
        self._thread = None
        self._nvml = None
        self._handle = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._handle = self._pick_handle(pynvml, index)
            self._nvml = pynvml
            self._max = float(pynvml.nvmlDeviceGetMaxClockInfo(self._handle, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nvml = None

    @staticmethod
    def _pick_handle(pynvml, index):
        # CUDA_VISIBLE_DEVICES may renumber the devices: go by UUID when it names one
        vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
        ids = [x.strip() for x in vis.split(",") if x.strip()]
        if index < len(ids):
            tok = ids[index]
            if tok.startswith("GPU-"):
                return pynvml.nvmlDeviceGetHandleByUUID(tok)
            if tok.isdigit():
                return pynvml.nvmlDeviceGetHandleByIndex(int(tok))
        return pynvml.nvmlDeviceGetHandleByIndex(index)

    def _once(self):
        try:
            if self._nvml is not None:
                n = self._nvml
                sm = float(n.nvmlDeviceGetClockInfo(self._handle, n.NVML_CLOCK_SM))
                r = int(n.nvmlDeviceGetCurrentClocksEventReasons(self._handle)) \
                    if hasattr(n, "nvmlDeviceGetCurrentClocksEventReasons") \
                    else int(n.nvmlDeviceGetCurrentClocksThrottleReasons(self._handle))
                flags = [bool(r & n.nvmlClocksThrottleReasonHwSlowdown),
                         bool(r & n.nvmlClocksThrottleReasonHwThermalSlowdown),
                         bool(r & n.nvmlClocksThrottleReasonSwThermalSlowdown),
                         bool(r & n.nvmlClocksThrottleReasonSwPowerCap)]
                self.samples.append((sm, self._max, flags))
                return
            out = subprocess.run(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                  "-i", str(self.index)], capture_output=True, text=True, timeout=5).stdout
            parts = [x.strip() for x in out.strip().split(",")]
            if len(parts) >= 6:
                self.samples.append((float(parts[0]), float(parts[1]),
                                     [x.lower() == "active" for x in parts[2:6]]))
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            self._once()
            self._stop.wait(0.002 if self._nvml is not None else 0.1)

    def start(self):
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join(timeout=10)
        if not self.samples:
            self._once()

    def summary(self):
        sm = [s[0] for s in self.samples]
        mx = [s[1] for s in self.samples]
        reasons = [n for i, n in enumerate(self.NAMES) if any(s[2][i] for s in self.samples)]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "sm_mhz_min": min(sm) if sm else None, "reasons": reasons, "samples": len(self.samples),
                "source": "nvml" if self._nvml is not None else "nvidia-smi"}


# --------------------------------------------------------------------------- #
# reference arm: the CPU oracle, as it stands, on a bounded sample
# --------------------------------------------------------------------------- #
_ORACLE_INPUTS = {}


def oracle_sample_step(cfg, sample_layers: int, accept_sets=None, gpu_mass=None):
    """Times the oracle on `sample_layers` layers of attention plus the
    acceptance pass and scales the attention part to the config's layer count.
    Returns (seconds per full step, cores used, accepted lengths).  The sampled
    layers' inputs are drawn once and kept: only the oracle's own work is timed.

    accept_sets: list of (logits, draft) of one step each; the acceptance time is
    the mean over them.  gpu_mass: the visual mass the rule is fed (the bytes the
    GPU's last attention layer wrote, so that both sides judge the same scores);
    without it the oracle's own mass of the last sampled layer."""
    import oracle
    from paper_2604_05650_b200 import workloads as W
    cores = oracle.max_threads()
    t_attn = 0.0
    mass = None
    for layer in range(sample_layers):
        key = (cfg.name, cfg.layers, layer)
        if key not in _ORACLE_INPUTS:
            _ORACLE_INPUTS[key] = W.attention_inputs(cfg, layer=layer)
        q, k, v, kv_len, span = _ORACLE_INPUTS[key]
        t0 = time.perf_counter()
        _, mass = oracle.verify_attention(q, k, v, kv_len, span)
        t_attn += time.perf_counter() - t0
    if accept_sets is None:
        key = (cfg.name, "accept")
        if key not in _ORACLE_INPUTS:
            _ORACLE_INPUTS[key] = [W.accept_inputs(cfg)]
        accept_sets = _ORACLE_INPUTS[key]
    rule_mass = np.ascontiguousarray(mass if gpu_mass is None else gpu_mass, dtype=np.float32)
    lens = []
    t0 = time.perf_counter()
    for logits, draft in accept_sets:
        a, _, _ = oracle.loose_accept(logits, draft, rule_mass, oracle.n_loose(cfg.lam, cfg.gamma),
                                      cfg.shift_window)
        lens.append(a)
    t_acc = (time.perf_counter() - t0) / len(accept_sets)
    return t_attn * cfg.layers / sample_layers + t_acc, cores, lens


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    # a bounded sample per step: two layers, one when many steps are asked for
    sample_layers = 2 if args.steps <= 30 else 1
    for _ in range(max(1, min(args.warmup, 1))):
        oracle_sample_step(cfg, 1)
    times = []
    cores = 1
    for _ in range(max(1, args.steps)):
        t, cores, _ = oracle_sample_step(cfg, sample_layers)
        times.append(t)
    t_step = sum(times) / len(times)
    value = cfg.batch * cfg.gamma / t_step
    sample = (f"each step: {sample_layers} of {cfg.layers} attention layers timed and scaled by layer count, "
              f"plus the full acceptance pass")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_step * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_desc(cfg, args.gpus),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def workload_desc(cfg, n_gpus):
    return {"workload": f"workload config {cfg_id_of(cfg)}: {cfg.name}-shaped verify step, {cfg.layers} layers, "
                        f"batch {cfg.batch}, gamma {cfg.gamma}, heads {cfg.n_q_heads}/{cfg.n_kv_heads}x{cfg.head_dim}, "
                        f"KV {cfg.kv_len} ({cfg.span[1] - cfg.span[0]} visual), vocab {cfg.vocab}",
            "kv_bytes_per_step": cfg.kv_bytes_per_layer * cfg.layers,
            "l2": "inputs larger than L2 (every layer streams its own K/V cache)",
            "parallelism": "replicas only" if n_gpus > 1 else "1 GPU",
            "layers_overridden": cfg.layers != full_layers(cfg)}


def full_layers(cfg):
    from paper_2604_05650_b200 import workloads as W
    return W.CONFIGS[cfg_id_of(cfg)].layers


def cfg_id_of(cfg):
    from paper_2604_05650_b200 import workloads as W
    for i, c in W.CONFIGS.items():
        if c.name == cfg.name:
            return i
    return -1


# --------------------------------------------------------------------------- #
# our arm
# --------------------------------------------------------------------------- #
def slowest_rank_ms(ms_local, world, dist, device):
    """Replicas only: every rank runs the same workload on its own GPU; the job
    takes as long as its slowest rank (MAX over ranks of the device-timed ms)."""
    import torch
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(world, batch, gamma, ms_step):
    """Verified draft tokens per second of the whole job: all ranks' tokens over
    the slowest rank's step time."""
    return world * batch * gamma / (ms_step * 1e-3)


N_ACCEPT_SETS = 16      # distinct (logits, drafts) sets the timed steps rotate over


def device_workload(cfg, dev, torch):
    """Synthetic inputs of the config's recipe drawn on the device (seeded):
    Q, K, V ~ N(0,1) in bf16 with the +0.5 shift of visual keys on 8 coordinates
    per KV head; logits and drafts come from the shared host generator, one set
    per sequence of a batch of N_ACCEPT_SETS x B (the timed steps rotate over the
    sets, so that the accepted length is not one sequence's draw)."""
    from paper_2604_05650_b200 import workloads as W
    gen = torch.Generator(device=dev)
    gen.manual_seed(cfg.seed)
    B, g, Hq, Hkv, D, L = cfg.batch, cfg.gamma, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.kv_len
    vs, ve = cfg.span
    qs, ks, vs_ = [], [], []
    for _ in range(cfg.layers):
        q = torch.randn((B, g, Hq, D), generator=gen, device=dev, dtype=torch.float32)
        k = torch.randn((B, Hkv, L, D), generator=gen, device=dev, dtype=torch.float32)
        v = torch.randn((B, Hkv, L, D), generator=gen, device=dev, dtype=torch.float32)
        for h in range(Hkv):
            dims = torch.randperm(D, generator=gen, device=dev)[:8]
            k[:, h, vs:ve, dims] += 0.5
        qs.append(q.to(torch.bfloat16))
        ks.append(k.to(torch.bfloat16))
        vs_.append(v.to(torch.bfloat16))
        del q, k, v
    logits, draft = W.accept_inputs(cfg, batch=N_ACCEPT_SETS * B)
    sets = [(np.ascontiguousarray(logits[i * B:(i + 1) * B]), np.ascontiguousarray(draft[i * B:(i + 1) * B]))
            for i in range(N_ACCEPT_SETS)]
    return qs, ks, vs_, sets


class VerifyStep:
    """One config's verify step on one GPU: device inputs, the library calls of a step
    (every layer's attention, then the acceptance pass on the last layer's mass), the
    CUDA graphs they are replayed from, and the device-timed loop."""

    def __init__(self, cfg, ctx, stream, dev, torch, kernel=0, use_graph=True, fp8=False):
        from paper_2604_05650_b200 import binding
        self.cfg, self.ctx, self.stream, self.dev, self.torch = cfg, ctx, stream, dev, torch
        self.qs, self.ks, self.vs, self.sets = device_workload(cfg, dev, torch)
        self.fp8 = fp8
        if fp8:
            # E4M3 codes and one scale per (sequence, KV head): the largest magnitude -> 448
            def quantize(t):
                scale = (t.float().abs().amax(dim=(2, 3)) / 448.0).clamp_min(1e-30)
                return (t.float() / scale[:, :, None, None]).to(torch.float8_e4m3fn).view(torch.uint8).contiguous(), \
                    scale.contiguous()
            self.k8 = [quantize(t) for t in self.ks]
            self.v8 = [quantize(t) for t in self.vs]
            self.ks = self.vs = None
            torch.cuda.empty_cache()
        B, g, Hq, Hkv, D, L = cfg.batch, cfg.gamma, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.kv_len
        self.shape = binding.attn_shape(B, g, Hq, Hkv, D, L, 0, kernel)
        self.kv_len = np.full((B,), L, dtype=np.int32)
        self.span = np.tile(np.asarray([cfg.span], dtype=np.int32), (B, 1))
        self.out = torch.empty((B, g, Hq, D), dtype=torch.bfloat16, device=dev)
        self.mass = torch.empty((B, g, Hq), dtype=torch.float32, device=dev)
        self.logits = [torch.from_numpy(l).to(dev) for l, _ in self.sets]
        self.draft = [torch.from_numpy(d).to(dev) for _, d in self.sets]
        self.alen = torch.full((N_ACCEPT_SETS, B), -1, dtype=torch.int32, device=dev)
        torch.cuda.synchronize(dev)
        # scratch for both calls is sized before anything is captured
        ctx.reserve(max(ctx.attention_workspace_bytes(self.shape, L),
                        ctx.accept_workspace_bytes(B, g, cfg.vocab)))
        l0 = ctx.launch_count()
        with torch.cuda.stream(stream):
            self.attention_layers()
            self.accept(0)
        stream.synchronize()
        self.launches_per_step = ctx.launch_count() - l0
        with torch.cuda.stream(stream):
            for i in range(1, N_ACCEPT_SETS):        # every set judged at least once
                self.accept(i)
        stream.synchronize()
        self.graph_attn, self.graph_acc = None, None
        if use_graph:
            self.graph_attn = torch.cuda.CUDAGraph()
            with torch.cuda.graph(self.graph_attn, stream=stream):
                self.attention_layers()
            self.graph_acc = []
            for i in range(N_ACCEPT_SETS):
                gr = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gr, stream=stream):
                    self.accept(i)
                self.graph_acc.append(gr)

    def attention_layers(self):
        for l in range(self.cfg.layers):
            if self.fp8:
                self.ctx.verify_attention_fp8(self.shape, self.qs[l], self.k8[l][0], self.v8[l][0], self.k8[l][1],
                                              self.v8[l][1], self.kv_len, self.span, self.out, self.mass)
            else:
                self.ctx.verify_attention(self.shape, self.qs[l], self.ks[l], self.vs[l], self.kv_len, self.span,
                                          self.out, self.mass)

    def accept(self, i):
        c = self.cfg
        self.ctx.loose_accept(c.batch, c.gamma, c.vocab, c.n_q_heads, self.logits[i], self.draft[i], self.mass,
                              self.alen[i], c.shift_window, lam=c.lam)

    def step(self, i=0, ev_a=None, ev_b=None):
        """Step i on the stream; ev_a / ev_b bracket its attention part."""
        if ev_a is not None:
            ev_a.record(self.stream)
        if self.graph_attn is not None:
            self.graph_attn.replay()
        else:
            self.attention_layers()
        if ev_b is not None:
            ev_b.record(self.stream)
        if self.graph_acc is not None:
            self.graph_acc[i % N_ACCEPT_SETS].replay()
        else:
            self.accept(i % N_ACCEPT_SETS)

    def timed(self, steps, warmup, barrier, clock_index):
        """Device-timed loop: `warmup` untimed steps, then `steps` steps between two
        events, the SM clock sampled meanwhile.  Returns (ms_total, sorted per-step
        attention ms, clock summary)."""
        torch, stream = self.torch, self.stream
        with torch.cuda.stream(stream):
            for i in range(max(warmup, 3)):
                self.step(i)
        stream.synchronize()
        clocks = ClockSampler(clock_index)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        attn_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                   for _ in range(steps)]
        barrier()
        torch.cuda.synchronize(self.dev)
        clocks.start()
        with torch.cuda.stream(stream):
            ev0.record(stream)
            for i in range(steps):
                self.step(i, *attn_ev[i])
            ev1.record(stream)
        stream.synchronize()
        torch.cuda.synchronize(self.dev)
        barrier()
        clocks.stop()
        return ev0.elapsed_time(ev1), sorted(a.elapsed_time(b) for a, b in attn_ev), clocks.summary()

    def accepted_per_step(self, steps):
        """Mean accepted length (summed over the batch) of the steps timed: step i
        judged set i % N_ACCEPT_SETS."""
        a = self.alen.sum(dim=1).cpu().numpy()
        used = [int(a[i % N_ACCEPT_SETS]) for i in range(steps)]
        return sum(used) / max(1, len(used))

    def free(self):
        self.graph_attn = self.graph_acc = None
        self.qs = self.ks = self.vs = self.logits = self.draft = self.k8 = self.v8 = None
        self.torch.cuda.empty_cache()


def hbm_peak():
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        return float(json.load(open(peaks_path))["hbm_gbs"]), "measured", json.load(open(peaks_path))
    return 6650.0, "fallback", {}


def attention_bytes_per_launch(cfg, fp8=False):
    """Algorithmic bytes of one attention call: K and V once (one byte per element and the
    scales with an fp8 cache), q and out, the mass."""
    B, g, Hq, D = cfg.batch, cfg.gamma, cfg.n_q_heads, cfg.head_dim
    kv = cfg.kv_bytes_per_layer // 2 + 2 * B * cfg.n_kv_heads * 4 if fp8 else cfg.kv_bytes_per_layer
    return kv + 2 * (B * g * Hq * D * 2) + B * g * Hq * 4


def time_other_config(cfg_id, ctx, stream, dev, torch, args, barrier, local):
    """Another model-shaped config with the same graph-replay timing as the main one:
    its own device inputs, warm-up, timed steps and clock record."""
    from paper_2604_05650_b200 import workloads as W
    cfg = W.CONFIGS[cfg_id]
    vs = VerifyStep(cfg, ctx, stream, dev, torch, args.kernel, not args.no_graph)
    steps = max(20, min(args.steps, 100))
    ms_total, attn_ms, clocks = vs.timed(steps, args.warmup, barrier, local)
    status = ctx.device_status()
    peak, peak_src, _ = hbm_peak()
    ms_step = ms_total / steps
    us_per_launch = sum(attn_ms) / steps * 1e3 / cfg.layers
    nbytes = attention_bytes_per_launch(cfg)
    gbs = nbytes / (us_per_launch * 1e-6) / 1e9
    res = {"workload": workload_desc(cfg, 1)["workload"], "steps": steps, "ms_per_step": ms_step,
           "value": cfg.batch * cfg.gamma / (ms_step * 1e-3), "unit": UNIT,
           "accepted_tokens_per_s": vs.accepted_per_step(steps) / (ms_step * 1e-3),
           "us_per_launch": us_per_launch, "us_per_launch_median": attn_ms[len(attn_ms) // 2] * 1e3 / cfg.layers,
           "bytes_per_launch": nbytes, "achieved_gbs": gbs, "frac": gbs / peak, "peak": peak,
           "peak_source": peak_src, "splits": ctx.attention_splits(vs.shape, cfg.kv_len),
           "device_status": status, "clocks": clocks}
    vs.free()
    return res


def run_ours(args, cfg):
    import torch
    import torch.distributed as dist
    from paper_2604_05650_b200 import binding, build as _build

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    if rank == 0:
        _build.build()
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist.barrier()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)

    def barrier():
        if world > 1:
            dist.barrier()

    ctx = binding.Context(local)
    stream = torch.cuda.Stream(device=dev)
    ctx.set_stream(stream.cuda_stream)
    vs = VerifyStep(cfg, ctx, stream, dev, torch, args.kernel, not args.no_graph, args.fp8_cache)
    B, g, Hq, Hkv, D, L = cfg.batch, cfg.gamma, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.kv_len

    ms_total, attn_ms, clock_summary = vs.timed(args.steps, args.warmup, barrier, local)
    status = ctx.device_status()
    ms_attn = sum(attn_ms) / args.steps
    ms_total_max = slowest_rank_ms(ms_total, world, dist, dev)
    ms_step = ms_total_max / args.steps
    value = whole_job_tokens_per_s(world, B, g, ms_step)
    accepted = vs.accepted_per_step(args.steps)
    gpu_alen = vs.alen.cpu().numpy()                   # [sets, B], judged on gpu_mass
    gpu_mass = vs.mass.cpu().numpy()                   # the last layer's visual mass

    # roofline of the dominant kernel: one verification-attention launch
    bytes_per_launch = attention_bytes_per_launch(cfg, args.fp8_cache)
    us_per_launch = ms_attn * 1e3 / cfg.layers
    achieved = bytes_per_launch / (us_per_launch * 1e-6) / 1e9
    peak, peak_src, peaks = hbm_peak()
    # DRAM bytes per launch from the committed ncu capture; null once the kernel has changed
    traffic = None
    tr_path = os.path.join(ROOT, "profiles", "traffic.json")
    if os.path.exists(tr_path):
        import hashlib
        tr = json.load(open(tr_path))
        src = os.path.join(ROOT, tr.get("kernel_source", ""))
        if os.path.exists(src) and hashlib.sha256(open(src, "rb").read()).hexdigest() == tr.get("kernel_source_sha256"):
            traffic = tr.get(f"config{cfg_id_of(cfg)}" + ("_fp8" if args.fp8_cache else ""))
    # secondary bounds of the same launch: useful tensor flops (two products, 2 flops per
    # multiply-add) against the measured bf16 GEMM rate, and exponentials against the
    # special-function rate (16 per clock and SM at the sampled clock)
    flops = 4.0 * B * Hq * g * cfg.kv_len * D
    bf16_peak = float(peaks.get("bf16_tflops_sustained", 1400.0))
    exps = float(B * Hq * g * cfg.kv_len)
    sm_mhz = clock_summary.get("sm_mhz") or 1965.0
    n_sm = torch.cuda.get_device_properties(dev).multi_processor_count
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": traffic, "peak_source": peak_src, "kernel": "verify attention (one layer)",
                "us_per_launch": us_per_launch, "bytes_per_launch": bytes_per_launch,
                "us_per_launch_median": attn_ms[len(attn_ms) // 2] * 1e3 / cfg.layers,
                "us_per_launch_min": attn_ms[0] * 1e3 / cfg.layers,
                "frac_of_nominal_8000": achieved / 8000.0,
                "tensor_tflops": flops / (us_per_launch * 1e-6) / 1e12,
                "tensor_frac_of_measured_bf16": flops / (us_per_launch * 1e-6) / 1e12 / bf16_peak,
                "mufu_frac": exps / (us_per_launch * 1e-6) / (16.0 * n_sm * sm_mhz * 1e6)}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": workload_desc(cfg, world), "cache": "e4m3 codes, one scale per KV head" if args.fp8_cache else "bf16",
            "accepted_tokens_per_s": world * accepted / (ms_step * 1e-3),
            "accept_len_mean": accepted, "accept_len_sets": gpu_alen.sum(axis=1).tolist(),
            "accept_sets": f"{N_ACCEPT_SETS} seeded (logits, drafts) sets; step i judges set i mod {N_ACCEPT_SETS}",
            "accept_checked": False,
            "ms_attention_per_step": ms_attn,
            "ms_accept_per_step": ms_step - ms_attn if world == 1 else None,
            "gpu_launches": vs.launches_per_step * args.steps, "device_status": status,
            "cuda_graph": vs.graph_attn is not None,
            "roofline": roofline, "clocks": clock_summary}

    if not args.no_next_rows and world == 1 and not args.fp8_cache:
        line["next_rows"] = {"visual_relevance": time_visual_relevance(cfg, ctx, stream, torch, dev, peak, args.top_n),
                             "fp8_attention": time_fp8_attention(cfg, ctx, stream, vs.ks, vs.vs, vs.qs, torch, dev, peak),
                             "paged_attention": time_paged_attention(cfg, ctx, stream, vs.ks, vs.vs, vs.qs, torch, dev, peak),
                             "several_spans": time_span_layer(cfg, ctx, stream, vs.ks, vs.vs, vs.qs, torch, dev)}

    # end to end through the host-buffer entry points
    if not args.no_e2e and not args.fp8_cache:
        line["e2e"] = run_e2e(args, cfg, ctx, stream, vs, torch, dev, world, barrier, dist)
    sets = vs.sets
    vs.free()
    del vs
    if world == 1 and not args.no_other_configs and cfg_id_of(cfg) == 2 and args.layers == 0 and not args.fp8_cache:
        line["other_configs"] = {str(i): time_other_config(i, ctx, stream, dev, torch, args, barrier, local)
                                 for i in (3, 1)}
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        # the oracle on a bounded sample; its acceptance pass runs on the very inputs of the
        # timed steps and on the GPU's own mass bytes, so its accepted lengths must equal the GPU's
        n_layers = 8 if cfg.layers >= 8 else cfg.layers
        t_cpu, cores, lens = oracle_sample_step(cfg, n_layers, sets, gpu_mass)
        want = np.stack(lens)
        if not (want == gpu_alen).all():
            raise SystemExit(f"accepted lengths differ from the oracle's rule on the same mass bytes: "
                             f"GPU {gpu_alen.tolist()} oracle {want.tolist()}")
        line["accept_checked"] = True
        line["cpu_baseline"] = {"value": B * g / t_cpu, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"{n_layers} of {cfg.layers} attention layers timed once and scaled "
                                          f"by layer count, plus the acceptance pass (mean over the "
                                          f"{N_ACCEPT_SETS} sets, judged on the GPU's mass bytes and compared "
                                          f"with the GPU's accepted lengths)"}
    ctx.close()
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def time_visual_relevance(cfg, ctx, stream, torch, dev, peak, top_n=10):
    """The paper's own relevance score (Eq. 4) on the config's visual span and
    hidden size, N = 10: not part of the verify step this benchmark times (the
    step scores positions by the attention's visual mass), measured beside it.
    HBM-bound on the one pass over H_V; two H_V copies alternate (each > L2)."""
    B, g = cfg.batch, cfg.gamma
    lv, d = cfg.span[1] - cfg.span[0], cfg.n_q_heads * cfg.head_dim
    gen = torch.Generator(device=dev)
    gen.manual_seed(cfg.seed + 77)
    hv = [torch.randn((B, lv, d), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16) for _ in range(2)]
    hd = torch.randn((B, g, d), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    inv = [torch.empty((B, lv), dtype=torch.float32, device=dev) for _ in range(2)]
    rel = torch.empty((B, g), dtype=torch.float32, device=dev)
    with torch.cuda.stream(stream):
        for c in range(2):
            ctx.row_inv_norms(B * lv, d, hv[c], inv[c])
        for c in range(2):
            ctx.visual_relevance(B, g, lv, d, hd, hv[c], inv[c], top_n, rel)
    stream.synchronize()
    reps = 10
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        e0.record(stream)
        for _ in range(reps):
            for c in range(2):
                ctx.visual_relevance(B, g, lv, d, hd, hv[c], inv[c], top_n, rel)
        e1.record(stream)
    stream.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / (2 * reps)
    nbytes = B * lv * d * 2 + B * lv * 4
    gbs = nbytes / (us * 1e-6) / 1e9
    return {"us_per_call": us, "n_visual": lv, "dim": d, "top_n": top_n, "bytes_per_call": nbytes,
            "achieved_gbs": gbs, "frac_of_peak": gbs / peak, "launches_per_call": 2}


def time_span_layer(cfg, ctx, stream, ks, vs_, qs, torch, dev):
    """The last layer's attention with the visual span cut into frames of 196 positions
    with 3 positions of text between them (only the layer whose mass feeds the rule needs
    the union of the spans): time of that one call against the plain call on the hull."""
    from paper_2604_05650_b200 import binding
    B, g, Hq, Hkv, D, L = cfg.batch, cfg.gamma, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.kv_len
    frames, pos = [], cfg.span[0]
    while pos + 196 <= cfg.span[1] and len(frames) < 200:
        frames.append([pos, pos + 196])
        pos += 199
    spans = np.tile(np.asarray([frames], dtype=np.int32), (B, 1, 1))
    hull = np.tile(np.asarray([[frames[0][0], frames[-1][1]]], dtype=np.int32), (B, 1))
    out = torch.empty((B, g, Hq, D), dtype=torch.bfloat16, device=dev)
    mass = torch.empty((B, g, Hq), dtype=torch.float32, device=dev)
    shape = binding.attn_shape(B, g, Hq, Hkv, D, L, 0, 0)
    kv_len = np.full((B,), L, dtype=np.int32)
    n = min(4, len(ks))

    def timed(call):
        with torch.cuda.stream(stream):
            for l in range(n):
                call(l)
            stream.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                ctx.set_stream(torch.cuda.current_stream().cuda_stream)
                for l in range(n):
                    call(l)
            ctx.set_stream(stream.cuda_stream)
            graph.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(5):
                graph.replay()
            e1.record(stream)
        stream.synchronize()
        return e0.elapsed_time(e1) * 1e3 / (5 * n)

    us_spans = timed(lambda l: ctx.verify_attention_spans(shape, qs[l], ks[l], vs_[l], kv_len, spans, out, mass))
    us_hull = timed(lambda l: ctx.verify_attention(shape, qs[l], ks[l], vs_[l], kv_len, hull, out, mass))
    return {"n_spans": len(frames), "gap_positions": 3 * (len(frames) - 1), "us_per_call": us_spans,
            "us_per_call_one_span": us_hull, "note": "graph replays of four layers' calls"}


def time_fp8_attention(cfg, ctx, stream, ks, vs_, qs, torch, dev, peak):
    """The verify attention on an fp8 (E4M3) cache: the first layers' caches of the step
    quantised on the device with one scale per KV head (largest magnitude -> 448), in a
    graph of up to eight layers (each streams its own K/V, more than L2 together).
    Algorithmic bytes: one byte per cache element, q and out in bf16, the mass."""
    from paper_2604_05650_b200 import binding
    B, g, Hq, Hkv, D, L = cfg.batch, cfg.gamma, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.kv_len
    if D != 128 or g * (Hq // Hkv) > 80:
        return None
    n_layers = min(8, len(ks))

    def quantize(t):
        scale = (t.float().abs().amax(dim=(2, 3)) / 448.0).clamp_min(1e-30)
        codes = (t.float() / scale[:, :, None, None]).to(torch.float8_e4m3fn).view(torch.uint8)
        return codes.contiguous(), scale.contiguous()

    k8 = [quantize(ks[l]) for l in range(n_layers)]
    v8 = [quantize(vs_[l]) for l in range(n_layers)]
    out = torch.empty((B, g, Hq, D), dtype=torch.bfloat16, device=dev)
    mass = torch.empty((B, g, Hq), dtype=torch.float32, device=dev)
    shape = binding.attn_shape(B, g, Hq, Hkv, D, L, 0, 0)
    kv_len = np.full((B,), L, dtype=np.int32)
    span = np.tile(np.asarray([cfg.span], dtype=np.int32), (B, 1))

    def layers():
        for l in range(n_layers):
            ctx.verify_attention_fp8(shape, qs[l], k8[l][0], v8[l][0], k8[l][1], v8[l][1], kv_len, span, out, mass)

    with torch.cuda.stream(stream):
        layers()
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            ctx.set_stream(torch.cuda.current_stream().cuda_stream)
            layers()
        ctx.set_stream(stream.cuda_stream)
        for _ in range(3):
            graph.replay()
        reps = 20
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            graph.replay()
        e1.record(stream)
    stream.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / (reps * n_layers)
    nbytes = cfg.kv_bytes_per_layer // 2 + 2 * B * Hkv * 4 + 2 * B * g * Hq * D * 2 + B * g * Hq * 4
    gbs = nbytes / (us * 1e-6) / 1e9
    return {"us_per_layer": us, "layers_in_graph": n_layers, "bytes_per_layer": nbytes, "achieved_gbs": gbs,
            "frac_of_peak": gbs / peak, "splits": ctx.attention_splits(shape, L, fp8=True), "cache": "E4M3, one scale per KV head"}


def time_paged_attention(cfg, ctx, stream, ks, vs_, qs, torch, dev, peak):
    """The verify attention on a paged cache (512-position pages scattered at random
    over a pool): the first layers' caches of the step, re-read as page pools, in a
    graph of up to eight layers (each streams its own 134 MB, more than L2 together)."""
    from paper_2604_05650_b200 import binding
    B, g, Hq, Hkv, D, L = cfg.batch, cfg.gamma, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.kv_len
    page = 512
    if L % page or D != 128:
        return None
    n_layers = min(8, len(ks))
    per_seq = L // page
    n_pages = B * per_seq
    # [B, Hkv, L, D] -> [B * L / page, Hkv, page, D]: logical page j of sequence b sits at
    # pool page b * per_seq + j; then the pool pages are shuffled and the table follows
    gen = torch.Generator(device="cpu")
    gen.manual_seed(cfg.seed + 99)
    perm = torch.randperm(n_pages, generator=gen)
    inv = torch.empty_like(perm)
    inv[perm] = torch.arange(n_pages)
    pools = []
    for l in range(n_layers):
        pk = ks[l].view(B, Hkv, per_seq, page, D).permute(0, 2, 1, 3, 4).reshape(n_pages, Hkv, page, D)
        pv = vs_[l].view(B, Hkv, per_seq, page, D).permute(0, 2, 1, 3, 4).reshape(n_pages, Hkv, page, D)
        pools.append((pk[perm.to(dev)].contiguous(), pv[perm.to(dev)].contiguous()))
    table = inv.view(B, per_seq).to(torch.int32).to(dev)
    out = torch.empty((B, g, Hq, D), dtype=torch.bfloat16, device=dev)
    mass = torch.empty((B, g, Hq), dtype=torch.float32, device=dev)
    shape = binding.attn_shape(B, g, Hq, Hkv, D, L, 0, 0)
    kv_len = np.full((B,), L, dtype=np.int32)
    span = np.tile(np.asarray([cfg.span], dtype=np.int32), (B, 1))

    def layers():
        for l in range(n_layers):
            ctx.verify_attention_paged(shape, page, n_pages, qs[l], pools[l][0], pools[l][1], table,
                                       kv_len, span, out, mass)

    with torch.cuda.stream(stream):
        layers()
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            ctx.set_stream(torch.cuda.current_stream().cuda_stream)
            layers()
        ctx.set_stream(stream.cuda_stream)
        for _ in range(3):
            graph.replay()
        reps = 10
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            graph.replay()
        e1.record(stream)
    stream.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / (reps * n_layers)
    nbytes = cfg.kv_bytes_per_layer + 2 * B * g * Hq * D * 2 + B * g * Hq * 4
    gbs = nbytes / (us * 1e-6) / 1e9
    del pools
    return {"us_per_layer": us, "page_size": page, "n_pages": n_pages, "layers_in_graph": n_layers,
            "bytes_per_layer": nbytes, "achieved_gbs": gbs, "frac_of_peak": gbs / peak}


def run_e2e(args, cfg, ctx, stream, vs, torch, dev, world, barrier, dist):
    """Same step through lvspec_*_host: every input starts in pinned host
    memory (K/V caches included) and the accepted length ends on the host."""
    from paper_2604_05650_b200 import binding
    B, g, Hq, Hkv, D, L = cfg.batch, cfg.gamma, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.kv_len
    pin = lambda t: t.cpu().pin_memory()
    hq = [pin(t) for t in vs.qs]
    hk = [pin(t) for t in vs.ks]
    hv = [pin(t) for t in vs.vs]
    hlog, hdraft = pin(vs.logits[0]), pin(vs.draft[0])
    hout = torch.empty((B, g, Hq, D), dtype=torch.bfloat16).pin_memory()
    hmass = torch.empty((B, g, Hq), dtype=torch.float32).pin_memory()
    hlen = torch.zeros((B,), dtype=torch.int32).pin_memory()
    shape, kv_len, span = vs.shape, vs.kv_len, vs.span

    def step():
        for l in range(cfg.layers):
            ctx.verify_attention_host(shape, hq[l], hk[l], hv[l], kv_len, span, hout, hmass)
        ctx.loose_accept_host(B, g, cfg.vocab, Hq, hlog, hdraft, hmass, hlen, cfg.shift_window, lam=cfg.lam)

    # every layer's caches cross PCIe each step (0.16 s per step on the 32K configs): the
    # steps asked for, up to 30
    steps = max(1, min(args.steps, 30))
    step()
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(dev)
    ev0.record(stream)
    for _ in range(steps):
        step()
    ev1.record(stream)
    stream.synchronize()
    barrier()
    ms = ev0.elapsed_time(ev1) / steps
    ms = slowest_rank_ms(ms, world, dist, dev)
    h2d = cfg.layers * (hq[0].numel() * 2 + 2 * hk[0].numel() * 2) + hlog.numel() * 4 + hdraft.numel() * 4 \
        + hmass.numel() * 4
    d2h = cfg.layers * (hout.numel() * 2 + hmass.numel() * 4) + hlen.numel() * 4
    del hk, hv
    # The same step as a serving loop sees it: the caches are state and stay on the device;
    # what crosses PCIe every step is what the step is given (the draft queries of every
    # layer, the target logits, the draft tokens) and what it returns (the accepted length).
    # The copies run beside the kernels: the first layers' queries go first, the rest of
    # the queries, the logits and the drafts follow on a second stream while the first
    # layers' attention runs; each is joined where it is first read.
    hq_all = torch.stack([t for t in hq]).pin_memory()
    dq_all = torch.empty(hq_all.shape, dtype=hq_all.dtype, device=dev)
    dq = [dq_all[l] for l in range(cfg.layers)]
    dlog, ddraft = torch.empty_like(vs.logits[0]), torch.empty_like(vs.draft[0])
    dout = torch.empty((B, g, Hq, D), dtype=torch.bfloat16, device=dev)
    dmass = torch.empty((B, g, Hq), dtype=torch.float32, device=dev)
    dlen = torch.zeros((B,), dtype=torch.int32, device=dev)
    head = min(4, cfg.layers)            # layers whose queries are copied ahead of the first kernel
    side = torch.cuda.Stream(device=dev)

    def resident_body(main):
        """Everything of one step, enqueued on `main` with the copies forked to `side`."""
        ctx.set_stream(main.cuda_stream)
        with torch.cuda.stream(main):
            dq_all[:head].copy_(hq_all[:head], non_blocking=True)
        side.wait_stream(main)
        with torch.cuda.stream(side):
            if head < cfg.layers:
                dq_all[head:].copy_(hq_all[head:], non_blocking=True)
            ev_q = torch.cuda.Event()
            ev_q.record(side)
            dlog.copy_(hlog, non_blocking=True)
            ddraft.copy_(hdraft, non_blocking=True)
        with torch.cuda.stream(main):
            for l in range(cfg.layers):
                if l == head:
                    main.wait_event(ev_q)
                ctx.verify_attention(shape, dq[l], vs.ks[l], vs.vs[l], kv_len, span, dout, dmass)
            main.wait_stream(side)
            ctx.loose_accept(B, g, cfg.vocab, Hq, dlog, ddraft, dmass, dlen, cfg.shift_window, lam=cfg.lam)
            hlen.copy_(dlen, non_blocking=True)

    step_graph = None
    resident_body(stream)
    stream.synchronize()
    if not args.no_graph:
        step_graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(step_graph, stream=stream):
            resident_body(torch.cuda.current_stream())
    ctx.set_stream(stream.cuda_stream)

    def resident_step():
        if step_graph is not None:
            with torch.cuda.stream(stream):
                step_graph.replay()
        else:
            resident_body(stream)
        stream.synchronize()

    resident_step()
    barrier()
    r_steps = max(3, args.steps)
    torch.cuda.synchronize(dev)
    ev0.record(stream)
    for _ in range(r_steps):
        resident_step()
    ev1.record(stream)
    stream.synchronize()
    barrier()
    ms_res = slowest_rank_ms(ev0.elapsed_time(ev1) / r_steps, world, dist, dev)
    res_h2d = cfg.layers * hq[0].numel() * 2 + hlog.numel() * 4 + hdraft.numel() * 4
    return {"value": whole_job_tokens_per_s(world, B, g, ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": ms, "steps": steps,
            "note": "K/V caches of every layer cross PCIe each step",
            "kv_resident": {"value": whole_job_tokens_per_s(world, B, g, ms_res), "unit": UNIT,
                            "h2d_bytes_per_step": res_h2d, "d2h_bytes_per_step": hlen.numel() * 4,
                            "ms_per_step": ms_res, "steps": r_steps,
                            "note": "caches resident on the device; queries, logits and drafts from pinned host "
                                    "memory (copied beside the attention kernels and joined where first read), "
                                    "accepted length back, a host synchronisation every step; the device part "
                                    "is one CUDA graph unless --no-graph"}}


def run_sweep(args):
    """workload config 4: the 40/8x128 head shape, one layer, gamma x KV length x
    batch.  Per point: time of one attention call and of the acceptance pass,
    achieved HBM GB/s of the attention call against the measured peak, verified
    tokens/s of the single-layer step.  Each point rotates over enough distinct
    K/V buffers (>= 256 MB in total, at least 2) that no call finds its cache in L2."""
    import torch
    from paper_2604_05650_b200 import binding, build as _build, workloads as W
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    _build.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    ctx = binding.Context(0)
    stream = torch.cuda.Stream(device=dev)
    ctx.set_stream(stream.cuda_stream)
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peak = float(json.load(open(peaks_path))["hbm_gbs"]) if os.path.exists(peaks_path) else 6650.0
    gen = torch.Generator(device=dev)
    gen.manual_seed(4)
    points, tok_total, ms_total = [], 0.0, 0.0
    clocks = ClockSampler(0)
    clocks.start()
    idx = 0
    for batch in W.SWEEP_BATCHES:
        for kv in W.SWEEP_KV_LENS:
            kv_bytes = 2 * batch * 8 * kv * 128 * 2
            copies = max(2, -(-(256 << 20) // kv_bytes))
            ks = [torch.randn((batch, 8, kv, 128), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
                  for _ in range(copies)]
            vs_ = [torch.randn((batch, 8, kv, 128), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
                   for _ in range(copies)]
            for gamma in W.SWEEP_GAMMAS:
                cfg = W.sweep_config(gamma=gamma, kv_len=kv, batch=batch, point=idx)
                idx += 1
                logits_h, draft_h = W.accept_inputs(cfg)
                logits, draft = torch.from_numpy(logits_h).to(dev), torch.from_numpy(draft_h).to(dev)
                q = torch.randn((batch, gamma, 40, 128), generator=gen, device=dev).to(torch.bfloat16)
                out = torch.empty_like(q)
                mass = torch.empty((batch, gamma, 40), dtype=torch.float32, device=dev)
                alen = torch.zeros((batch,), dtype=torch.int32, device=dev)
                shape = binding.attn_shape(batch, gamma, 40, 8, 128, kv, 0, args.kernel)
                kv_len = np.full((batch,), kv, dtype=np.int32)
                span = np.tile(np.asarray([cfg.span], dtype=np.int32), (batch, 1))

                def rotation():
                    for c in range(copies):
                        ctx.verify_attention(shape, q, ks[c], vs_[c], kv_len, span, out, mass)

                def accept():
                    ctx.loose_accept(batch, gamma, cfg.vocab, 40, logits, draft, mass, alen,
                                     cfg.shift_window, lam=cfg.lam)

                with torch.cuda.stream(stream):
                    rotation()
                    accept()
                stream.synchronize()
                g_attn, g_acc = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
                with torch.cuda.graph(g_attn, stream=stream):
                    rotation()
                with torch.cuda.graph(g_acc, stream=stream):
                    accept()
                reps = max(3, min(50, int(2000 // copies)))
                e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
                with torch.cuda.stream(stream):
                    for _ in range(3):
                        g_attn.replay()
                        g_acc.replay()
                    e0.record(stream)
                    for _ in range(reps):
                        g_attn.replay()
                    e1.record(stream)
                    for _ in range(reps):
                        g_acc.replay()
                    e2.record(stream)
                stream.synchronize()
                us_attn = e0.elapsed_time(e1) * 1e3 / (reps * copies)
                us_acc = e1.elapsed_time(e2) * 1e3 / reps
                nbytes = kv_bytes + 2 * q.numel() * 2 + mass.numel() * 4
                gbs = nbytes / (us_attn * 1e-6) / 1e9
                tps = batch * gamma / ((us_attn + us_acc) * 1e-6)
                points.append({"batch": batch, "kv_len": kv, "gamma": gamma, "us_attention": round(us_attn, 2),
                               "us_accept": round(us_acc, 2), "hbm_gbs": round(gbs, 1),
                               "frac_of_measured_peak": round(gbs / peak, 4), "tokens_per_s": round(tps, 1),
                               "splits": ctx.attention_splits(shape, kv), "kv_buffers": copies})
                tok_total += batch * gamma
                ms_total += (us_attn + us_acc) * 1e-3
                del g_attn, g_acc
            del ks, vs_
            torch.cuda.empty_cache()
    clocks.stop()
    status = ctx.device_status()
    ctx.close()
    line = {"metric": METRIC, "value": tok_total / (ms_total * 1e-3), "unit": UNIT, "n_gpus": 1,
            "steps": len(points), "warmup": 3, "ms_per_step": ms_total / len(points), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "workload config 4: sweep on the 40/8x128 head shape, one layer per point, "
                                   "gamma {4,8,16} x KV {4K,16K,64K,128K} x batch {1,4,16}, 75% visual",
                       "l2": "each point rotates over >= 256 MB of distinct K/V buffers"},
            "device_status": status,
            "clocks": clocks.summary(), "peak_hbm_gbs": peak, "sweep": points}
    print(json.dumps(line))


def main():
    args = parse()
    if args.sweep:
        run_sweep(args)
        return
    from paper_2604_05650_b200 import workloads as W
    cfg = W.CONFIGS[args.config]
    if args.layers > 0:
        cfg = dataclasses.replace(cfg, layers=args.layers)
    if args.lam is not None:
        cfg = dataclasses.replace(cfg, lam=args.lam)
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
