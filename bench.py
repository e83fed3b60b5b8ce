"""Benchmark of the MoE layer forward pass (one "step" = the whole hot path over one synthetic batch).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl mok|reference]

Prints ONE JSON line.  Default workload: the DeepSeek-V3-like layer (T=32768, H=7168, E=256, k=8, I=2048, one shared
expert of I=2048; about 23 GB of expert weights resident in HBM), synthetic seeded inputs.  The same line carries
`per_config` (the four smaller workloads, each timed the same way) and `sweep` (the default workload at T = 64, 512,
4096 against the HBM weight-read roofline); `--per-config none` / `--no-sweep` leave them out.

With N > 1 (launched by torch.distributed.run) every rank holds a full copy of the weights and its own batch of T
tokens (token-sharded replicas: no data-path collective), the step time is the max over ranks and `value` is the
aggregate tokens/s ("weak" scaling); the sub-records are only produced at N = 1.

`--impl reference` times the CPU oracle (the fp64 definition of the layer) on the host cores on a bounded token
sample of the same workload; it is a deliberately slow baseline, not a target.
"""
import argparse
import datetime
import json
import math
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "moe_layer_fwd_tokens_per_s"
UNIT = "tokens/s"
DEFAULT_WORKLOAD = "deepseek_v3"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes (read + write) of ONE launch of the dominant kernel (routed gate/up grouped GEMM), from the ncu captures
# summarised under profiles/.  The two DRAM byte counters and the duration are one pass per launch (nothing is saved or
# restored), so they are captured on the full-size workloads themselves; `scale` would carry a capture of a scaled
# case (same H, I, k and rows per expert, a fraction of the experts and tokens) to the full size.
NCU_TRAFFIC = {
    # one-pass captures at full size (dram__bytes_read.sum + dram__bytes_write.sum of one launch)
    "deepseek_v3": {"bytes": 20.57e9, "scale": 1, "source": "profiles/gemm_kernels_deepseek_v3.md"},
    # the routed expert FFN as one persistent launch (the default where synchronised tile starts pay)
    "deepseek_v3+one_launch": {"bytes": 38.01e9, "scale": 1, "source": "profiles/gemm_kernels_deepseek_v3.md"},
    "gpt_oss_120b+one_launch": {"bytes": 9.55e9, "scale": 1, "source": "profiles/gemm_kernels_other_workloads.md"},
    "qwen3_30b_a3b": {"bytes": 1.415e9, "scale": 1, "source": "profiles/gemm_kernels_other_workloads.md"},
    "mixtral_8x7b": {"bytes": 3.553e9, "scale": 1, "source": "profiles/gemm_kernels_other_workloads.md"},
    "gpt_oss_120b": {"bytes": 5.136e9, "scale": 1, "source": "profiles/gemm_kernels_other_workloads.md"},
}


def parse():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=20)
    p.add_argument("--warmup", type=int, default=5)
    p.add_argument("--config", default=DEFAULT_WORKLOAD)
    p.add_argument("--impl", default="mok", choices=["mok", "reference"])
    p.add_argument("--tokens", type=int, default=0, help="override T (small-T sweeps)")
    p.add_argument("--experts", type=int, default=0,
                   help="override E: with --tokens, a scaled copy of a workload (same H, I, k and rows per expert) that is "
                        "small enough for a profiler capture")
    p.add_argument("--fused-ffn", type=int, default=0, help="2: routed gate/up + down GEMM as one persistent launch; 3: and the combine")
    p.add_argument("--h-ring", type=int, default=0,
                   help="slots (256 rows each, >= 24) of a ring that holds the gated activation, in the smaller workspace "
                        "that goes with it (0 = a row for every route)")
    p.add_argument("--cpu-sample", type=int, default=0, help="tokens of the CPU-oracle sample (0 = auto)")
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--per-config", default="auto",
                   help="'auto' (the other workloads when the default one is benchmarked on one GPU), 'none', or a "
                        "comma-separated list of workload names")
    p.add_argument("--no-sweep", action="store_true", help="skip the small-T sweep of the default workload")
    p.add_argument("--no-e2e", action="store_true", help="skip the host-buffer (end-to-end) legs")
    p.add_argument("--no-backward", action="store_true", help="skip the backward-pass record of the headline workload")
    p.add_argument("--no-counters", action="store_true", help="skip the device-side counter pass")
    p.add_argument("--cooldown", type=float, default=2.0,
                   help="idle seconds before each workload's warm-up, so that every workload starts from the same board state")
    p.add_argument("--sustain-seconds", type=float, default=2.0,
                   help="length of the extra loop that shows the power-capped steady state (0 = skip)")
    p.add_argument("--gather-mode", type=int, default=0, help="0 auto, 1 fused into the GEMM, 2 separate kernel")
    p.add_argument("--cta-group", type=int, default=0, help="0 default, 1 single CTAs, 2 CTA pairs")
    p.add_argument("--gemm", type=int, default=0, help="0 tcgen05 (tokens on M), 2 tcgen05 (tokens on N), 1 SIMT")
    p.add_argument("--tile-sched", type=int, default=0, help="routed GEMMs: 0 persistent grid, 1 tiles stolen through cluster launch control")
    p.add_argument("--host-chunks", type=int, default=0, help="token chunks of the host-buffer call (0 = auto)")
    p.add_argument("--precision", default="bf16", choices=["bf16", "mxfp8"],
                   help="routed experts in bf16 (the headline workload) or MXFP8 with pre-quantised weights")
    p.add_argument("--comm-ctas", type=int, default=0,
                   help="one-launch expert FFN: CTAs that only stage token rows for the computing CTAs (0 = the gather "
                        "warps of every CTA pull their rows themselves)")
    p.add_argument("--parallelism", default="replicas", choices=["replicas", "ep"],
                   help="replicas: every GPU holds all experts and its own batch (no data-path collective); ep: expert "
                        "parallelism, every GPU holds E / N experts and its own batch of T tokens, rows are pulled from "
                        "the peers' token buffers and combined by the token's owner")
    p.add_argument("--ep-check", action="store_true",
                   help="--parallelism ep with several ranks: compare with the one-rank layer even when that means "
                        "loading all experts on every rank")
    p.add_argument("--pass", dest="which", default="forward", choices=["forward", "backward"],
                   help="forward (the headline metric) or the backward pass of the same workload (bf16)")
    return p.parse_args()


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
    return dict(FALLBACK_PEAKS, source="fallback")


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples with timestamps, taken in the background for the whole run;
    window(t0, t1) summarises the samples that fall into one timed region (host wall-clock seconds)."""
    Q = ("timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.samples = None

    def start(self):
        import tempfile
        self.t_start = time.time()
        # into a file: a pipe that nobody drains fills up after a few hundred lines and stops nvidia-smi
        self.log = tempfile.NamedTemporaryFile("w+", prefix="mok_clocks_", suffix=".csv", delete=False)
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=self.log, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        self.samples = []
        if self.proc is None:
            return
        time.sleep(0.05)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=10)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            self.proc.wait()
        self.log.flush()
        self.log.seek(0)
        out = self.log.read()
        self.log.close()
        try:
            os.unlink(self.log.name)
        except OSError:
            pass
        for line in out.strip().splitlines():
            f = [v.strip() for v in line.split(",")]
            if len(f) < 10:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                self.samples.append((ts, float(f[2]), float(f[3]), float(f[4]),
                                     [n for n, v in zip(self.NAMES, f[6:10]) if v.lower().startswith("active")]))
            except ValueError:
                continue
        # nvidia-smi prints local time and time.time() counts from the UTC epoch: where the two disagree about the
        # time zone the difference is a whole number of quarter hours, which the first sample reveals
        if self.samples:
            off = round((self.samples[0][0] - self.t_start) / 900.0) * 900.0
            if off:
                self.samples = [(s[0] - off,) + s[1:] for s in self.samples]

    def window(self, t0, t1):
        if self.samples is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["clock samples not collected yet"]}
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        note = None
        if not inside:      # a region shorter than the sampling period: take the sample nearest to its middle
            mid = 0.5 * (t0 + t1)
            inside = [min(self.samples, key=lambda s: abs(s[0] - mid))]
            note = "region shorter than the sampling period: nearest sample"
        sm = sorted(s[1] for s in inside)
        reasons = sorted({r for s in inside for r in s[4]})
        out = {"sm_mhz": sm[len(sm) // 2], "sm_min_mhz": sm[0], "sm_max_mhz": max(s[2] for s in inside),
               "power_w_max": max(s[3] for s in inside), "samples": len(inside), "reasons": reasons}
        if note:
            out["note"] = note
        return out


def _median(v):
    v = sorted(v)
    return v[len(v) // 2]


def cpu_oracle_leg(cfg, d, sample, gpu_idx=None, gpu_w=None):
    """The oracle as it stands on the host cores: routing of all T tokens (its per-token share is charged to the
    sample) plus the per-token FFN of `sample` tokens.  Returns (tokens/s, seconds, threads, routing report); the
    report compares the device's top-k ids and weights (when given) with the oracle's, token by token."""
    import numpy as np
    from oracle import mok_ref
    t0 = time.perf_counter()
    idx, w, gap, lg = mok_ref.route(d["x"], d["W_r"], d["bias"], cfg.k)
    t_route = time.perf_counter() - t0
    tokens = np.arange(min(sample, cfg.T), dtype=np.int32)
    t0 = time.perf_counter()
    if d.get("W_gate_up") is not None and len(tokens):
        mok_ref.ffn_tokens(d["x"], d["W_gate_up"], d["W_down"], d["W_sgu"], d["W_sd"], idx, w, tokens)
    t_ffn = time.perf_counter() - t0
    t = t_ffn + t_route * len(tokens) / cfg.T
    report = None
    if gpu_idx is not None:
        sel = np.take_along_axis(lg, idx.astype(np.int64), axis=1)
        inner = np.full(cfg.T, np.inf) if cfg.k == 1 else (sel[:, :-1] - sel[:, 1:]).min(axis=1)
        differs = (gpu_idx != idx).any(axis=1)
        same_set = (np.sort(gpu_idx, axis=1) == np.sort(idx, axis=1)).all(axis=1)
        w_sel = mok_ref.weights(lg, gpu_idx)
        report = {"boundary_near_ties": int((gap < 1e-4).sum()),
                  "order_near_ties": int(((inner < 1e-4) & ~(gap < 1e-4)).sum()),
                  "flipped_tokens": int(differs.sum()), "flipped_sets": int((~same_set).sum()),
                  "flipped_outside_near_ties": int((differs & ~((gap < 1e-4) | (inner < 1e-4))).sum()),
                  "w_max_err": float(np.abs(gpu_w.astype(np.float64) - w_sel).max())}
    return (len(tokens) / t if len(tokens) else 0.0), t_ffn + t_route, mok_ref.num_threads(), report


def fingerprints(d, limit=1 << 28):
    """SHA-256 of each input tensor as generated (tensors above `limit` bytes: of their first `limit` bytes)."""
    import hashlib
    import numpy as np
    out = {"numpy": np.__version__}
    for name in ("x", "W_r", "bias", "W_gate_up", "W_down", "W_sgu", "W_sd"):
        a = d.get(name)
        if a is None:
            continue
        raw = memoryview(np.ascontiguousarray(a)).cast("B")
        part = raw[:limit]
        out[name] = hashlib.sha256(part).hexdigest()[:16] + ("" if len(raw) <= limit else f" (first {limit} bytes)")
    return out


def auto_sample(cfg, cores, seconds=15.0):
    # the scalar oracle sustains about 4 fp64 GFLOP/s per core on the GPU hosts
    per_token = 6.0 * cfg.H * (cfg.k * cfg.I + cfg.I_s)
    n = int(seconds * 4.0e9 * cores / per_token)
    return max(16, min(cfg.T, n))


def run_reference(args, cfg, rank):
    """The CPU oracle as the reference arm.  Rank 0 only."""
    if rank != 0:
        return
    from paper_2609_36070_b200 import inputs
    d = inputs.make_inputs(cfg)
    cores = os.cpu_count() or 1
    steps = max(1, min(args.steps, 3))
    warm = min(args.warmup, 1)
    sample = args.cpu_sample or max(16, auto_sample(cfg, cores) // (steps + warm))
    for _ in range(warm):
        cpu_oracle_leg(cfg, d, sample)
    rates = []
    t_total = 0.0
    for _ in range(steps):
        r, t, threads, _ = cpu_oracle_leg(cfg, d, sample)
        rates.append(r)
        t_total += t
    value = sum(rates) / len(rates)
    line = {"metric": METRIC, "value": value, "unit": UNIT, "impl": "reference", "n_gpus": args.gpus, "steps": steps,
            "warmup": warm, "ms_per_step": 1e3 * t_total / steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "T": cfg.T, "H": cfg.H, "E": cfg.E, "k": cfg.k, "I": cfg.I, "I_shared": cfg.I_s},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": f"routing of all {cfg.T} tokens (charged pro rata) + fp64 FFN of the first {sample} tokens per step"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gflops": value * 6.0 * cfg.H * (cfg.k * cfg.I + cfg.I_s) / 1e9}
    print(json.dumps(line), flush=True)


def backward_record(cfg, g, idx, w, steps, warmup, cta_group=0, sampler=None):
    """Times mok_moe_backward (activation recomputation, dx, router-weight and weight gradients) on tensors already on
    the device; idx / w: the forward pass's routing.  FLOPs are counted as twice the forward pass's (dgrad + wgrad), as
    in the paper's Section 4.1; the recomputed gate/up product and the transposes are extra work that is not counted."""
    import numpy as np
    import torch
    from paper_2609_36070_b200 import inputs, mok
    dev = g["x"].device
    rng = np.random.default_rng(1)
    dout = mok.to_device_bf16(inputs.f32_to_bf16_bits(rng.standard_normal((cfg.T, cfg.H), dtype=np.float32)), dev)
    res = mok.mok_moe_backward(g["x"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], idx, w, dout)
    bws = res["workspace"]
    conf = mok._config(cta_group=cta_group)

    def step():
        mok.mok_moe_backward(g["x"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], idx, w, dout, workspace=bws,
                             config=conf)

    for _ in range(max(warmup, 3)):
        step()
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    t0 = time.time()
    ev[0].record()
    for i in range(steps):
        step()
        ev[i + 1].record()
    torch.cuda.synchronize()
    t1 = time.time()
    per = sorted(ev[i].elapsed_time(ev[i + 1]) for i in range(steps))
    ms = per[len(per) // 2]
    assert mok.mok_read_status(bws) == 0
    flops = 2.0 * cfg.ffn_flops()
    rec = {"ms_per_step": ms, "mean_ms_per_step": ev[0].elapsed_time(ev[steps]) / steps, "steps": steps,
           "tokens_per_s": cfg.T / (ms * 1e-3), "tflops": flops / (ms * 1e-3) / 1e12,
           "flops_counted": "2 x forward (dgrad + wgrad); the recomputed gate/up product is extra work, not counted",
           "pass": "backward (recompute + dgrad + wgrad), bf16", "_window": (t0, t1)}
    del res, bws, dout
    return rec


def run_backward(args, cfg):
    """`--pass backward`: the backward pass of one workload on one GPU, one JSON line."""
    import torch
    from paper_2609_36070_b200 import inputs, mok
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    d = inputs.make_inputs(cfg)
    g = {k: (None if d[k] is None else mok.to_device_bf16(d[k], dev)) for k in ("x", "W_gate_up", "W_down", "W_sgu", "W_sd")}
    W_r = torch.from_numpy(d["W_r"]).to(dev)
    bias = None if d["bias"] is None else torch.from_numpy(d["bias"]).to(dev)
    ws = mok.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, device=dev)
    out, st = mok.mok_moe_forward_ex(g["x"], W_r, bias, g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k, ws,
                                     stages=True)
    sampler = ClockSampler(0)
    sampler.start()
    rec = backward_record(cfg, g, st["topk_idx"], st["topk_w"], args.steps, args.warmup, args.cta_group)
    sampler.stop()
    win = rec.pop("_window")
    print(json.dumps({"metric": "moe_layer_bwd_tokens_per_s", "value": rec["tokens_per_s"], "unit": UNIT, "n_gpus": 1,
                      "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": rec["ms_per_step"],
                      "mean_ms_per_step": rec["mean_ms_per_step"], "higher_is_better": True,
                      "dtype": "bf16", "data": "synthetic", "tflops": rec["tflops"],
                      "config": {"workload": cfg.name, "T": cfg.T, "H": cfg.H, "E": cfg.E, "k": cfg.k, "I": cfg.I,
                                 "I_shared": cfg.I_s, "pass": rec["pass"]},
                      "clocks": sampler.window(*win)}), flush=True)


class Layer:
    """One workload resident on the device, with the calls the benchmark times."""

    def __init__(self, cfg, args, dev, rank=0, d=None, staging=0):
        import torch
        from paper_2609_36070_b200 import inputs, mok, sharding
        self.cfg, self.args, self.dev, self.mok, self.torch = cfg, args, dev, mok, torch
        self.d = d if d is not None else inputs.make_inputs(cfg)
        if rank > 0:
            self.d["x"] = sharding.rank_tokens(cfg, rank)
        d = self.d
        self.g = {k: (None if d[k] is None else mok.to_device_bf16(d[k], dev))
                  for k in ("x", "W_gate_up", "W_down", "W_sgu", "W_sd")}
        self.W_r = torch.from_numpy(d["W_r"]).to(dev)
        self.bias = None if d["bias"] is None else torch.from_numpy(d["bias"]).to(dev)
        self.mx = args.precision == "mxfp8"
        self.prec = mok.MOK_PRECISION_MXFP8 if self.mx else mok.MOK_PRECISION_BF16
        self.mxw = mok.MxWeights(self.g["W_gate_up"], self.g["W_down"]) if self.mx else None
        self.ws = mok.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, device=dev, host_staging=staging,
                                      mx=self.mx, h_ring_tiles=args.h_ring)
        # the router weights are split once, as a caller of the library would do at load time
        try:
            self.split = mok.mok_router_prepare(self.W_r, cfg.k, self.conf())
        except mok.MokError:
            self.split = None
        self.out = torch.empty_like(self.g["x"])

    def conf(self, **kw):
        a = self.args
        base = dict(impl=a.gemm, gather_mode=a.gather_mode, cta_group=a.cta_group, precision=self.prec,
                    tile_sched=a.tile_sched, fused_ffn=a.fused_ffn, h_ring_tiles=a.h_ring, comm_ctas=a.comm_ctas)
        base.update(kw)
        return self.mok._config(**base)

    def view(self, T):
        """The same weights with the first T tokens (the small-T sweep)."""
        import copy
        v = copy.copy(self)
        v.cfg = self.cfg.with_tokens(T)
        v.g = dict(self.g, x=self.g["x"][:T].contiguous())
        v.out = self.out[:T]
        return v

    def step(self, conf, stages=False):
        g, cfg = self.g, self.cfg
        return self.mok.mok_moe_forward_ex(g["x"], self.W_r, self.bias, g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"],
                                           cfg.k, self.ws, out=self.out, config=conf, mx_weights=self.mxw, stages=stages,
                                           router_split=self.split)

    def check_status(self):
        status = self.mok.mok_read_status(self.ws)
        assert status == 0, self.mok.mok_status_string(status)

    def timed_steps(self, conf, steps, barrier):
        """K steps bracketed by a barrier + synchronize on both sides, with one CUDA event between consecutive steps.
        Returns (total ms, per-step ms list, host wall-clock window)."""
        torch = self.torch
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        barrier()
        t0 = time.time()
        ev[0].record()
        for i in range(steps):
            self.step(conf)
            ev[i + 1].record()
        barrier()
        t1 = time.time()
        return ev[0].elapsed_time(ev[steps]), [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)], (t0, t1)

    def stage_times(self, steps, second_half=False):
        """Per-stage CUDA-event times (events recorded by the library around every stage) of a loop of its own, so
        that the events are not part of the headline loop.  Returns {stage: (mean, median)} in ms and the window;
        second_half: statistics over the second half of the loop only (the steady state of a long loop)."""
        mok = self.mok
        conf = self.conf(profile=1)
        mok.mok_profile_begin(steps)
        self.torch.cuda.synchronize()
        t0 = time.time()
        for _ in range(steps):
            self.step(conf)
        stage = mok.mok_profile_end(steps)
        self.torch.cuda.synchronize()
        t1 = time.time()
        if second_half:
            stage = stage[len(stage) // 2:]
            t0 = 0.5 * (t0 + t1)
        res = {s: (sum(c[s] for c in stage) / len(stage), _median([c[s] for c in stage]), min(c[s] for c in stage))
               for s in mok.STAGES}
        return res, (t0, t1)

    def one_launch_ab(self, rounds=3, block_s=0.3):
        """The routed expert FFN as two launches (gate/up GEMM, down GEMM) against ONE persistent launch
        (config.fused_ffn = 2), alternating in blocks of about `block_s` seconds so that both see the same board state.
        Returns mean step times in ms (first round dropped), or None where the one-launch kernel does not apply."""
        torch = self.torch
        a = self.args
        if self.mx or a.gemm != 0 or a.cta_group in (1, 2) or a.tile_sched == 1 or (self.cfg.I + 127) // 128 > 32:
            return None
        confs = {"two_launches": self.conf(fused_ffn=1), "one_launch": self.conf(fused_ffn=2)}
        for c in confs.values():
            self.step(c)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        self.step(confs["two_launches"])
        e1.record()
        torch.cuda.synchronize()
        n = int(max(3, min(500, block_s * 1e3 / max(e0.elapsed_time(e1), 1e-3))))
        acc = {k: [] for k in confs}
        for r in range(rounds + 1):
            for name, c in confs.items():
                e0.record()
                for _ in range(n):
                    self.step(c)
                e1.record()
                torch.cuda.synchronize()
                if r > 0:
                    acc[name].append(e0.elapsed_time(e1) / n)
        self.check_status()
        out = {k + "_ms": sum(v) / len(v) for k, v in acc.items()}
        out.update({"rounds": rounds, "steps_per_block": n,
                    "how": "blocks of the two variants alternate in one process; whole-step time, mean over the rounds"})
        return out

    def counters(self):
        """Device-side counters of the GEMM kernels (one extra step with config.debug = 1), reduced to the figures the
        roofline discussion uses."""
        conf = self.conf(debug=1)
        self.step(conf)
        raw = self.mok.mok_debug_counters(self.ws)
        out = {}
        for name, c in raw.items():
            if name == "fused" and c["ctas"]:      # the one-launch expert FFN: whole-kernel clock and imbalance
                out[name] = {"sm_ghz_in_kernel": c["mma_total"] / max(1, c["mma_total_ns"]),
                             "busiest_cta_over_mean": c["mma_total_max_cta"] / (c["mma_total"] / c["ctas"]), "ctas": c["ctas"],
                             "producer_wait_for_rows_share": raw["gemm2"]["producer_wait_stage"] / max(1, c["mma_total"])}
                continue
            if not c["ctas"] or not c["k_blocks"]:
                continue
            units = c["k_blocks"]               # 128-row x 64-column-of-K MMA units: 512 tensor-pipe cycles each
            r = {"sm_ghz_in_kernel": c["mma_total"] / max(1, c["mma_total_ns"]),
                 "cycles_per_unit": c["mma_total"] / units,
                 "wait_operands_per_unit": c["mma_wait_operands"] / units,
                 "wait_accumulator_per_unit": c["mma_wait_accumulator"] / units,
                 "busiest_cta_over_mean": c["mma_total_max_cta"] / (c["mma_total"] / c["ctas"]),
                 "ctas": c["ctas"]}
            if c["valid_rows_x_k_blocks"]:
                r["pad_row_share_of_mma_work"] = 1.0 - c["valid_rows_x_k_blocks"] / (128.0 * units)
            out[name] = r
        return out


def roofline_fracs(tflops, pk, mx, region_s, clocks):
    """achieved / peak against both measured bf16 peaks; `frac` is the one that fits the run: the burst figure for a
    kernel timed at full clocks in a short region, the sustained one when the timed region lasts seconds or the SM
    clock sampled during it sits well under the maximum (the board is then in its power-capped steady state)."""
    scale = 2.0 if mx else 1.0   # fp8 tensor peak = measured bf16 peak x the nominal 2:1 ratio (4.5 vs 2.25 PFLOP/s dense)
    burst, sust = scale * pk["bf16_tflops"], scale * pk.get("bf16_tflops_sustained", pk["bf16_tflops"])
    sm, smx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    sustained = region_s > 2.0 or (sm is not None and smx and sm < 0.9 * smx)
    peak = sust if sustained else burst
    return {"achieved": tflops, "peak": peak, "unit": "TFLOP/s", "frac": tflops / peak,
            "frac_of_burst": tflops / burst, "frac_of_sustained": tflops / sust,
            "peak_source": f"{pk['source']} " + ("bf16_tflops_sustained" if sustained else "bf16_tflops (burst)") +
                           (" x 2 (nominal fp8 : bf16 ratio)" if mx else "") +
                           (": timed region of %.1f s at a median %s MHz of %s" % (region_s, sm, smx))}


def measure(layer, steps, warmup, barrier, sampler_windows, pk, with_counters):
    """Headline loop, stage loop and counters of one workload on this rank.  Clock windows are resolved later, when
    the sampler has been stopped; `sampler_windows` collects (record, key, window) for that."""
    cfg, mok = layer.cfg, layer.mok
    conf = layer.conf()

    def rest_and_warm():
        if layer.args.cooldown > 0:
            layer.torch.cuda.synchronize()
            time.sleep(layer.args.cooldown)
        for _ in range(warmup):
            layer.step(conf)
        barrier()
        layer.check_status()

    # Two short loops, each from the same rested board state (the board throttles within ~0.1 s of load, so a loop
    # that simply followed the other would run in a different regime): per-stage events first, then the headline loop.
    rest_and_warm()
    stage_steps = max(3, min(steps, 10))
    stages, swin = layer.stage_times(stage_steps)
    layer.check_status()
    rest_and_warm()
    total_ms, per_step, win = layer.timed_steps(conf, steps, barrier)
    layer.check_status()
    rec = {"ms_per_step": _median(per_step), "mean_ms_per_step": total_ms / steps, "min_ms_per_step": min(per_step),
           "steps": steps, "stage_ms": {s: stages[s][1] for s in mok.STAGES},
           "stage_ms_mean": {s: stages[s][0] for s in mok.STAGES}, "stage_ms_min": {s: stages[s][2] for s in mok.STAGES},
           "_region_s": total_ms * 1e-3,
           "_stage_region_s": swin[1] - swin[0]}
    sampler_windows.append((rec, "clocks", win))
    sampler_windows.append((rec, "clocks_stage_loop", swin))
    # The steady state under the board's power cap: a loop of a few seconds, statistics over its second half, and the
    # device-side counters (in-kernel SM clock) right behind it while the board is still in that state.
    secs = layer.args.sustain_seconds
    if secs > 0:
        n = int(max(10, min(5000, secs * 1e3 / rec["ms_per_step"])))
        sstages, ssw = layer.stage_times(n, second_half=True)
        layer.check_status()
        srec = {"steps": n, "stage_ms": {s: sstages[s][0] for s in mok.STAGES}}
        srec["ms_per_step"] = sum(srec["stage_ms"].values())
        rec["sustained"] = srec
        sampler_windows.append((srec, "clocks", ssw))
    if rec["ms_per_step"] < 0.3 and not layer.mx:
        # a launch-bound layer: the same call recorded once into a CUDA graph and replayed (what a caller with a fixed
        # shape would do), so that the number shows the GPU's time and not the host's launch rate
        torch = layer.torch
        try:
            layer.step(conf)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                layer.step(conf)
            for _ in range(5):
                graph.replay()
            torch.cuda.synchronize()
            n = 200
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(n):
                graph.replay()
            e1.record()
            torch.cuda.synchronize()
            layer.check_status()
            rec["cuda_graph_replay_ms"] = e0.elapsed_time(e1) / n
            del graph
        except Exception as ex:                      # (informational: never fails the run)
            rec["cuda_graph_replay_ms"] = None
            rec["cuda_graph_note"] = str(ex)[:200]
    if with_counters and not layer.mx and layer.args.gemm == 0:
        rec["counters"] = layer.counters()
        layer.check_status()
        ab = layer.one_launch_ab()
        if ab is not None:
            rec["one_launch_ffn"] = ab
    return rec


def finish_record(rec, cfg, pk, mx, world=1):
    """Derived figures of one workload's record (after the clock windows have been filled in)."""
    ms = rec["ms_per_step"]
    flops = cfg.ffn_flops()
    st = rec["stage_ms"]
    rec["tokens_per_s"] = world * cfg.T / (ms * 1e-3)
    rec["tflops"] = world * flops / (ms * 1e-3) / 1e12
    ffn_ms = st["gemm1"] + st["gemm2"] + st["shared_gemm1"] + st["shared_gemm2"]
    ffn_tf = flops / (ffn_ms * 1e-3) / 1e12
    scale = 2.0 if mx else 1.0
    rec["ffn_phase"] = {"ms": ffn_ms, "tflops": ffn_tf, "frac_of_burst": ffn_tf / (scale * pk["bf16_tflops"]),
                        "frac_of_sustained": ffn_tf / (scale * pk.get("bf16_tflops_sustained", pk["bf16_tflops"]))}
    # The dominant kernel: the routed gate/up grouped GEMM -- or, where the library runs the routed expert FFN as ONE
    # persistent launch (its default for large expert matrices), that kernel, which holds the gate/up AND the down
    # tiles (the stage events then show the whole launch under gemm1 and nothing under gemm2).
    one_launch = st["gemm2"] < 0.01 * st["gemm1"]
    g1_flops = (6.0 if one_launch else 4.0) * cfg.T * cfg.k * cfg.H * cfg.I
    g1_tf = g1_flops / (st["gemm1"] * 1e-3) / 1e12
    clk = rec.get("clocks_stage_loop") or {}
    dom = roofline_fracs(g1_tf, pk, mx, rec.pop("_stage_region_s"), clk)
    dom["ms"] = st["gemm1"]
    dom["kernel"] = ("routed expert FFN in one persistent launch: gate/up tiles + SwiGLU and down tiles, token gather fused "
                     "(fused_ffn_kernel)") if one_launch else \
                    "routed gate/up grouped GEMM + SwiGLU, token gather fused (gemm_m2_kernel<EPI_SWIGLU, GATHER>)"
    dom["algorithmic_flops_per_launch"] = g1_flops
    # the fastest single launch of the loop against the burst peak (itself the best of ten single launches)
    best = rec.pop("stage_ms_min")["gemm1"]
    dom["best_launch_ms"] = best
    dom["best_launch_frac_of_burst"] = g1_flops / (best * 1e-3) / 1e12 / (scale * pk["bf16_tflops"])
    if clk.get("sm_mhz"):
        dom["sm_cycles"] = st["gemm1"] * 1e-3 * clk["sm_mhz"] * 1e6       # kernel time x median sampled SM clock
    ck = "fused" if one_launch else "gemm1"
    if "counters" in rec and ck in rec["counters"]:
        dom["sm_cycles_device"] = st["gemm1"] * 1e-3 * rec["counters"][ck]["sm_ghz_in_kernel"] * 1e9
    tr = NCU_TRAFFIC.get(cfg.name + ("+one_launch" if one_launch else ""))
    # weights once per expert, rows gathered once per route, h written (and, in the one launch, read back from L2), y written
    dom["algorithmic_bytes"] = 2.0 * (2 * cfg.I * cfg.H * cfg.E + cfg.T * cfg.k * (cfg.H + cfg.I)) + \
        (2.0 * (cfg.I * cfg.H * cfg.E + cfg.T * cfg.k * cfg.H) if one_launch else 0.0)
    dom["traffic"] = None if (mx or tr is None) else tr["bytes"] * tr["scale"]
    if tr is not None and not mx:
        dom["traffic_source"] = f"{tr['source']} (ncu capture x {tr['scale']})"
    rec["dominant_kernel"] = dom
    rec.pop("_region_s", None)
    if "sustained" in rec:
        s = rec["sustained"]
        sst = s["stage_ms"]
        sffn = sst["gemm1"] + sst["gemm2"] + sst["shared_gemm1"] + sst["shared_gemm2"]
        sust_peak = scale * pk.get("bf16_tflops_sustained", pk["bf16_tflops"])
        s["tokens_per_s"] = world * cfg.T / (s["ms_per_step"] * 1e-3)
        s["tflops"] = world * flops / (s["ms_per_step"] * 1e-3) / 1e12
        s["ffn_phase"] = {"ms": sffn, "tflops": flops / (sffn * 1e-3) / 1e12,
                          "frac_of_sustained": flops / (sffn * 1e-3) / 1e12 / sust_peak,
                          "frac_of_burst": flops / (sffn * 1e-3) / 1e12 / (scale * pk["bf16_tflops"])}
        s_flops = (6.0 if sst["gemm2"] < 0.01 * sst["gemm1"] else 4.0) * cfg.T * cfg.k * cfg.H * cfg.I
        s["dominant_kernel"] = {"ms": sst["gemm1"], "tflops": s_flops / (sst["gemm1"] * 1e-3) / 1e12,
                                "frac_of_sustained": s_flops / (sst["gemm1"] * 1e-3) / 1e12 / sust_peak}
    return rec


def run_ep(args, cfg, rank, local_rank, world):
    """`--parallelism ep`: the expert-parallel layer (Sections 2.1, 3.1-3.3) with one process per GPU.  Every rank keeps
    T tokens of its own (weak scaling: N * T tokens per step in total) and E / N experts; per step it routes its tokens,
    all-gathers the routes, builds Algorithm 1's schedule for its experts, runs their FFNs on rows pulled from the
    owners' token buffers, and after one barrier combines its own tokens' rows from the serving ranks' buffers.
    Same timing rules and JSON line as the replicated mode; `value` = N * T / the slowest rank's median step time."""
    import statistics
    import torch
    import torch.distributed as dist
    from paper_2609_36070_b200 import ep, inputs, mok, sharding
    assert args.warmup >= 3, "timing rules: at least 3 warm-up steps"
    assert cfg.E % world == 0, "the experts must divide over the ranks"
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29543")
    os.environ.setdefault("TORCH_SYMM_MEM_DISABLE_MULTICAST", "1")     # plain peer pointers only
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    pk = peaks()
    mx = args.precision == "mxfp8"
    L = cfg.E // world
    d = inputs.make_inputs(cfg, expert_range=(rank * L, (rank + 1) * L))
    if rank > 0:
        d["x"] = sharding.rank_tokens(cfg, rank)
    g = {k: (None if d[k] is None else mok.to_device_bf16(d[k], dev)) for k in ("x", "W_gate_up", "W_down", "W_sgu", "W_sd")}
    W_r = torch.from_numpy(d["W_r"]).to(dev)
    bias = None if d["bias"] is None else torch.from_numpy(d["bias"]).to(dev)
    mxw = mok.MxWeights(g["W_gate_up"], g["W_down"]) if mx else None
    layer = ep.DistributedLayer(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, dev, mx=mx)
    out = torch.empty_like(g["x"])
    conf = mok._config(cta_group=args.cta_group, comm_ctas=args.comm_ctas, fused_ffn=args.fused_ffn,
                       tile_sched=args.tile_sched)

    def step(x, timeline=None):
        layer.forward(x, W_r, bias, g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], out=out, config=conf,
                      mx_weights=mxw, timeline=timeline)

    def barrier():
        dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        barrier()
        t0 = time.time()
        ev[0].record()
        for i in range(steps):
            fn(i)
            ev[i + 1].record()
        barrier()
        return [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)], (t0, time.time())

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    for _ in range(args.warmup):
        step(g["x"])
    per, win = timed(lambda i: step(g["x"]), args.steps)
    ms = sharding.max_over_ranks(statistics.median(per), dist, dev)
    mean_ms = sharding.max_over_ranks(sum(per) / len(per), dist, dev)
    assert layer.status() == 0, mok.mok_status_string(layer.status())
    # phases, from a loop of their own with an event after each
    phases = {}
    n_ph = max(3, min(args.steps, 10))
    for _ in range(n_ph):
        tl = []
        step(g["x"], tl)
        torch.cuda.synchronize()
        for (_, a), (name, b) in zip(tl, tl[1:]):
            phases.setdefault(name, []).append(a.elapsed_time(b))
    phases = {k: sharding.max_over_ranks(statistics.median(v), dist, dev) for k, v in phases.items()}
    # end to end: the rank's tokens start in pinned host memory and its output ends there, every step
    xh = g["x"].cpu().pin_memory()
    oh = torch.empty_like(xh).pin_memory()

    def e2e_step(i):
        step(xh)
        oh.copy_(out, non_blocking=True)

    for _ in range(3):
        e2e_step(0)
    e2e_steps = max(5, min(args.steps, 50))
    per_e, _ = timed(e2e_step, e2e_steps)
    e2e_ms = sharding.max_over_ranks(statistics.median(per_e), dist, dev)
    same_bits = bool(torch.equal(oh.view(torch.int16), out.cpu().view(torch.int16)))
    # the bits of the one-rank layer: a token's output depends only on its own row and the weights, so every rank can
    # run the replicated layer on its own tokens with all experts and compare.  Needs all experts on every rank, so
    # with more than one rank it runs for workloads of at most 8 GB of expert weights, or when asked for.
    bits_equal = None
    w_bytes = 6.0 * cfg.E * cfg.H * cfg.I
    if not mx and (world == 1 or args.ep_check or w_bytes <= 8e9):
        full = g if world == 1 else {k: (None if v is None else mok.to_device_bf16(v, dev)) for k, v in
                                     inputs.make_inputs(cfg).items() if k in ("W_gate_up", "W_down")}
        ws1 = mok.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, device=dev)
        step(g["x"])
        one = mok.mok_moe_forward_ex(g["x"], W_r, bias, full["W_gate_up"], full["W_down"], g["W_sgu"], g["W_sd"], cfg.k, ws1)
        ok = torch.tensor([int(torch.equal(out.view(torch.int16), one.view(torch.int16)) and mok.mok_read_status(ws1) == 0)],
                          device=dev)
        dist.all_reduce(ok, op=dist.ReduceOp.MIN)
        bits_equal = bool(ok.item())
        del full, ws1, one
    sampler.stop() if rank == 0 else None
    if rank == 0:
        flops = 6.0 * cfg.T * cfg.H * (cfg.k * cfg.I + cfg.I_s)          # per rank: its experts serve N*T*k/N rows on average
        peak = (2.0 if mx else 1.0) * pk["bf16_tflops"]
        ffn_ms = phases["expert_ffn"]
        act = 2 * cfg.T * cfg.H
        clocks = sampler.window(*win)
        line = {
            "metric": METRIC, "value": world * cfg.T / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "mean_ms_per_step": mean_ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "mxfp8 routed experts (fp32 accumulate), bf16 elsewhere" if mx else "bf16", "data": "synthetic",
            "config": {"workload": cfg.name, "T_per_gpu": cfg.T, "T_total": world * cfg.T, "H": cfg.H, "E": cfg.E,
                       "experts_per_gpu": L, "k": cfg.k, "I": cfg.I, "I_shared": cfg.I_s, "routing": cfg.bias,
                       "parallelism": f"ep{world}", "comm_ctas": args.comm_ctas,
                       "l2": "inputs larger than L2 (weights + activations >> 126 MB), no explicit flush",
                       "timing": "ms_per_step = median of the per-step CUDA-event times of one bracketed loop (max over "
                                 "ranks); phase times come from a second loop with an event after every phase"},
            "tflops": world * flops / (ms * 1e-3) / 1e12,
            "bitwise_equal_to_one_rank_layer": bits_equal,
            "phase_ms": phases,
            "roofline": {"kernel": "the rank's expert FFN call (Algorithm 1 schedule, routed gate/up with the pull gather "
                                   "fused, down, shared expert)", "bound": "tensor",
                         "achieved": flops / (ffn_ms * 1e-3) / 1e12, "peak": peak, "unit": "TFLOP/s",
                         "frac": flops / (ffn_ms * 1e-3) / 1e12 / peak, "peak_kind": "burst (of measured)"
                         if pk["source"] == "measured" else "burst (of fallback)", "traffic": None, "ms": ffn_ms},
            "gpu_launches": args.steps * (mok.mok_launch_count(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, conf) + 1),
            "clocks": clocks,
            "e2e": {"value": world * cfg.T / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms, "steps": e2e_steps,
                    "h2d_bytes_per_step": act, "d2h_bytes_per_step": act,
                    "mode": "per step: pinned host x -> the rank's peer-visible token buffer, the expert-parallel layer, "
                            "out -> pinned host", "result_bits_equal_device_call": same_bits},
        }
        print(json.dumps(line), flush=True)
    dist.barrier()
    dist.destroy_process_group()


def main():
    args = parse()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    from paper_2609_36070_b200 import inputs
    cfg = inputs.CONFIGS[args.config]
    if args.tokens:
        cfg = cfg.with_tokens(args.tokens)
    if args.experts:
        import dataclasses
        cfg = dataclasses.replace(cfg, E=args.experts, name=f"{cfg.name}_E{args.experts}")
    if args.impl == "reference":
        run_reference(args, cfg, rank)
        return
    if args.which == "backward":
        if rank == 0:
            run_backward(args, cfg)
        return
    if args.parallelism == "ep":
        run_ep(args, cfg, rank, local_rank, world)
        return

    import gc
    import numpy as np
    import torch
    from paper_2609_36070_b200 import mok, sharding
    assert args.warmup >= 3, "timing rules: at least 3 warm-up steps"
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    pk = peaks()
    mx = args.precision == "mxfp8"
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    windows = []

    # ------------------------------------------------------------------ the headline workload
    # every rank: same weights, its own batch (seed offset by rank)
    layer = Layer(cfg, args, dev, rank=rank, staging=0 if args.no_e2e else 2)
    main_rec = measure(layer, args.steps, args.warmup, barrier, windows, pk, with_counters=not args.no_counters and rank == 0)
    ms_per_step = sharding.max_over_ranks(main_rec["ms_per_step"], dist, dev)
    mean_ms = sharding.max_over_ranks(main_rec["mean_ms_per_step"], dist, dev)
    main_rec["ms_per_step"], main_rec["mean_ms_per_step"] = ms_per_step, mean_ms

    ws_bytes = (mok.mok_workspace_bytes_ring(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, args.h_ring) if args.h_ring else
                mok.mok_workspace_bytes(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k))
    # device's routing of this batch (for the comparison inside the cpu-baseline leg); outside every timed region
    gpu_idx = gpu_w = counts = None
    if rank == 0:
        _, st = layer.step(layer.conf(), stages=True)
        layer.check_status()
        gpu_idx, gpu_w = st["topk_idx"].cpu().numpy(), st["topk_w"].cpu().numpy()
        counts = st["counts"].cpu().numpy()
        del st

    # End to end through the host-buffer entry points: pinned host x -> device, layer, result -> pinned host, every step.
    # Throughput (`e2e.value`): a stream of batches through the asynchronous call, whose two staging slots let the upload
    # of step i+1 and the download of step i-1 overlap the layer of step i; the timed region ends when the last result
    # has arrived in host memory.  Latency of ONE isolated batch (`e2e.single_call_ms`): the blocking call, which cuts
    # the batch into token chunks to overlap its own copies.
    e2e = None
    if not args.no_e2e:
        g = layer.g
        xh = g["x"].cpu().pin_memory()
        oh = [torch.empty_like(xh).pin_memory() for _ in range(2)]
        conf0 = layer.conf(host_chunks=args.host_chunks)

        def e2e_submit(i):
            mok.mok_moe_forward_host_async(xh, oh[i & 1], layer.W_r, layer.bias, g["W_gate_up"], g["W_down"], g["W_sgu"],
                                           g["W_sd"], cfg.k, layer.ws, config=conf0, mx_weights=layer.mxw)

        def single_call():
            mok.mok_moe_forward_host(xh, oh[0], layer.W_r, layer.bias, g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"],
                                     cfg.k, layer.ws, config=conf0, mx_weights=layer.mxw)

        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e2e_steps = max(5, min(args.steps, 50))
        for i in range(3):
            e2e_submit(i)
        mok.mok_host_wait()
        barrier()
        ev0.record()
        for i in range(e2e_steps):
            e2e_submit(i)
        mok.mok_host_wait()               # the host blocks until the last download has landed ...
        ev1.record()                      # ... so this event closes the region after every copy of every step
        barrier()
        layer.check_status()
        e2e_ms = sharding.max_over_ranks(ev0.elapsed_time(ev1) / e2e_steps, dist, dev)
        for _ in range(2):
            single_call()
        barrier()
        ev0.record()
        for _ in range(3):
            single_call()
        ev1.record()
        barrier()
        single_ms = sharding.max_over_ranks(ev0.elapsed_time(ev1) / 3, dist, dev)
        act_bytes = 2 * cfg.T * cfg.H
        same_bits = bool(torch.equal(oh[(e2e_steps - 1) & 1].view(torch.int16), layer.out.cpu().view(torch.int16)))
        e2e = {"value": world * cfg.T / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms, "steps": e2e_steps,
               "h2d_bytes_per_step": act_bytes, "d2h_bytes_per_step": act_bytes,
               "mode": "stream of batches through mok_moe_forward_host_async (two staging slots), timed until the last "
                       "result is in host memory",
               "single_call_ms": single_ms, "result_bits_equal_device_call": same_bits}
        del xh, oh

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ------------------------------------------------------------------ backward pass of the headline workload (N = 1)
    backward = None
    if world == 1 and not args.no_backward and not mx and gpu_idx is not None:
        free, _ = torch.cuda.mem_get_info()
        need = (mok.mok_bwd_workspace_bytes(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k) +
                6.0 * cfg.E * cfg.H * cfg.I + 6.0 * cfg.H * cfg.I_s + 4.0 * cfg.T * cfg.H + (2 << 30))
        if free > need:
            _, stb = layer.step(layer.conf(), stages=True)
            time.sleep(args.cooldown)
            backward = backward_record(cfg, layer.g, stb["topk_idx"], stb["topk_w"], max(5, min(args.steps, 10)), 3,
                                       args.cta_group)
            windows.append((backward, "clocks", backward.pop("_window")))
            del stb
            gc.collect()
            torch.cuda.empty_cache()
        else:
            backward = {"skipped": f"needs {need / 2**30:.0f} GiB of free device memory, {free / 2**30:.0f} free"}

    # ------------------------------------------------------------------ small-T sweep of the default workload (N = 1)
    sweep = None
    if world == 1 and not args.no_sweep and args.config == DEFAULT_WORKLOAD and not args.tokens and not args.experts:
        sweep = []
        for T in (64, 512, 4096):
            v = layer.view(T)
            keep = args.sustain_seconds
            args.sustain_seconds = 0.0
            rec = measure(v, 30, 5, barrier, windows, pk, with_counters=False)
            args.sustain_seconds = keep
            _, st = v.step(v.conf(), stages=True)
            v.check_status()
            active = int((st["counts"].cpu().numpy() > 0).sum())
            wbytes = 2.0 * 3 * cfg.H * (active * cfg.I + cfg.I_s)          # every active expert's weights, read once
            roof_ms = wbytes / (pk["hbm_gbs"] * 1e9) * 1e3
            # the same bound GEMM by GEMM, with each GEMM's tensor time where that is the larger one (from a few
            # thousand tokens on, the shared expert's two GEMMs are bound by arithmetic, not by their 88 MB of weights)
            def gemm_bound_ms(w_bytes, flops):
                return max(w_bytes / (pk["hbm_gbs"] * 1e9), flops / (pk["bf16_tflops"] * 1e12)) * 1e3
            rows = int(st["counts"].cpu().numpy().sum())
            roof2_ms = (gemm_bound_ms(4.0 * cfg.H * cfg.I * active, 4.0 * rows * cfg.H * cfg.I) +
                        gemm_bound_ms(2.0 * cfg.H * cfg.I * active, 2.0 * rows * cfg.H * cfg.I))
            if cfg.I_s:
                roof2_ms += (gemm_bound_ms(4.0 * cfg.H * cfg.I_s, 4.0 * T * cfg.H * cfg.I_s) +
                             gemm_bound_ms(2.0 * cfg.H * cfg.I_s, 2.0 * T * cfg.H * cfg.I_s))
            sm = rec["stage_ms"]
            gemm_ms = sm["gemm1"] + sm["gemm2"] + sm["shared_gemm1"] + sm["shared_gemm2"]
            rec.update({"T": T, "active_experts": active, "weight_bytes": wbytes, "hbm_roofline_ms": roof_ms,
                        "gemm_ms": gemm_ms, "gemm_frac_of_hbm_roofline": roof_ms / gemm_ms,
                        "per_gemm_roofline_ms": roof2_ms, "gemm_frac_of_per_gemm_roofline": roof2_ms / gemm_ms,
                        "step_frac_of_hbm_roofline": roof_ms / rec["ms_per_step"],
                        "tokens_per_s": T / (rec["ms_per_step"] * 1e-3)})
            rec.pop("_region_s", None)
            rec.pop("_stage_region_s", None)
            rec.pop("stage_ms_mean", None)
            rec.pop("stage_ms_min", None)
            sweep.append(rec)
            del st

    # ------------------------------------------------------------------ the other workloads (N = 1)
    names = []
    if args.per_config == "auto":
        if world == 1 and args.config == DEFAULT_WORKLOAD and not args.tokens and not args.experts:
            names = [n for n in inputs.CONFIG_ORDER if n != args.config]
    elif args.per_config != "none":
        names = [n for n in args.per_config.split(",") if n]
    main_d = layer.d
    main_counts = counts
    fp = fingerprints(main_d)
    # keep the host copy of the headline inputs for the cpu-baseline leg; release the device copy before loading others
    if names:
        del layer
        gc.collect()
        torch.cuda.empty_cache()
    per_config = {}
    for n in names:
        c = inputs.CONFIGS[n]
        lay = Layer(c, args, dev)
        est = None
        for _ in range(3):
            lay.step(lay.conf())
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        lay.step(lay.conf())
        e1.record()
        torch.cuda.synchronize()
        est = max(e0.elapsed_time(e1), 1e-3)
        steps = int(min(200, max(20, math.ceil(50.0 / est))))           # a short timed region: about 50 ms or 20 steps
        rec = measure(lay, steps, 5, barrier, windows, pk, with_counters=not args.no_counters)
        _, st = lay.step(lay.conf(), stages=True)
        lay.check_status()
        rec["config"] = {"workload": c.name, "T": c.T, "H": c.H, "E": c.E, "k": c.k, "I": c.I, "I_shared": c.I_s,
                         "routing": c.bias}
        cnt = st["counts"].cpu().numpy()
        rec["load"] = {"max_count": int(cnt.max()), "empty_experts": int((cnt == 0).sum()),
                       "rows_padded_to_128": int(((cnt + 127) // 128 * 128).sum()), "rows": int(cnt.sum())}
        if not args.no_cpu_baseline:   # the cpu-baseline leg of this workload: routing in full, a short FFN sample
            cores = os.cpu_count() or 1
            r, s, th, rp = cpu_oracle_leg(c, lay.d, auto_sample(c, cores, seconds=1.0), st["topk_idx"].cpu().numpy(),
                                          st["topk_w"].cpu().numpy())
            rec["cpu_baseline"] = {"value": r, "unit": UNIT, "cores": th, "kind": "oracle", "seconds": s}
            rec["routing_check"] = rp
        per_config[n] = rec
        del lay, st
        gc.collect()
        torch.cuda.empty_cache()

    sampler.stop()
    for rec, key, win in windows:
        rec[key] = sampler.window(*win)
    region_s = main_rec["_region_s"]
    finish_record(main_rec, cfg, pk, mx, world)
    for n, rec in per_config.items():
        finish_record(rec, inputs.CONFIGS[n], pk, mx)
        rec.pop("stage_ms_mean", None)
    if sweep:
        for rec in sweep:
            rec.pop("clocks_stage_loop", None)

    dom = main_rec.pop("dominant_kernel")
    roofline = {"kernel": dom.pop("kernel"), "bound": "tensor"}
    if mx:
        roofline["kernel"] = ("routed gate/up grouped GEMM on MXFP8 operands + SwiGLU + activation quantisation, token gather "
                              "fused (gemm_mx_kernel<EPI_SWIGLU, GATHER>)")
    roofline.update(dom)
    if "sustained" in main_rec:
        roofline["sustained_run"] = main_rec["sustained"]["dominant_kernel"]
    conf = mok._config(impl=args.gemm, gather_mode=args.gather_mode, cta_group=args.cta_group, fused_ffn=args.fused_ffn,
                       h_ring_tiles=args.h_ring,
                       precision=mok.MOK_PRECISION_MXFP8 if mx else mok.MOK_PRECISION_BF16, tile_sched=args.tile_sched)
    line = {
        "metric": METRIC, "value": main_rec["tokens_per_s"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "mean_ms_per_step": mean_ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "mxfp8 routed experts (fp32 accumulate), bf16 elsewhere" if mx else "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "T": cfg.T, "H": cfg.H, "E": cfg.E, "k": cfg.k, "I": cfg.I,
                   "I_shared": cfg.I_s, "routing": cfg.bias, "parallelism": f"token-sharded replicas x{world}",
                   "h_ring_tiles": args.h_ring, "workspace_bytes": int(ws_bytes),
                   "l2": "inputs larger than L2 (weights + activations >> 126 MB), no explicit flush",
                   "timing": "ms_per_step = median of the per-step CUDA-event times of one bracketed loop of `steps` "
                             "steps (max over ranks); stage times come from a second loop with per-stage events"},
        "tflops": main_rec["tflops"],
        "tflops_frac_of_burst_peak": main_rec["tflops"] / world / ((2.0 if mx else 1.0) * pk["bf16_tflops"]),
        "ffn_phase": main_rec["ffn_phase"],
        "stage_ms": main_rec["stage_ms"],
        "inputs": fp,
        "roofline": roofline,
        "gpu_launches": args.steps * mok.mok_launch_count(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, conf),
        "clocks": main_rec["clocks"],
        "timed_region_s": region_s,
    }
    if "sustained" in main_rec:
        line["sustained"] = main_rec["sustained"]
    if "counters" in main_rec:
        line["counters"] = main_rec["counters"]
    if "one_launch_ffn" in main_rec:
        line["one_launch_ffn"] = main_rec["one_launch_ffn"]
    for key in ("cuda_graph_replay_ms", "cuda_graph_note"):
        if key in main_rec:
            line[key] = main_rec[key]
    if main_counts is not None:
        line["load"] = {"max_count": int(main_counts.max()), "empty_experts": int((main_counts == 0).sum()),
                        "rows_padded_to_128": int(((main_counts + 127) // 128 * 128).sum()), "rows": int(main_counts.sum())}
    if e2e is not None:
        line["e2e"] = e2e
    if not args.no_cpu_baseline:
        cores = os.cpu_count() or 1
        sample = args.cpu_sample or auto_sample(cfg, cores)
        rate, secs, threads, rep = cpu_oracle_leg(cfg, main_d, sample, gpu_idx, gpu_w)
        line["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": secs,
                                "sample": f"routing of all {cfg.T} tokens (charged pro rata) + fp64 FFN of the first {min(sample, cfg.T)} tokens"}
        line["routing_check"] = rep
    if backward is not None:
        line["backward"] = backward
    if per_config:
        line["per_config"] = per_config
    if sweep:
        line["sweep"] = sweep
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
