"""Benchmark of the MoE layer forward pass (one "step" = the whole hot path over one synthetic batch).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl mok|reference]

Prints ONE JSON line.  Default workload: the Qwen3-30B-A3B-like layer (T=16384, H=2048, E=128, k=8, I=768,
Zipf-skewed routing), synthetic seeded inputs.  With N > 1 (launched by torch.distributed.run) every rank holds a
full copy of the weights and its own batch of T tokens (token-sharded replicas: no data-path collective), the step
time is the max over ranks and `value` is the aggregate tokens/s ("weak" scaling).

`--impl reference` times the CPU oracle (the fp64 definition of the layer) on the host cores on a bounded token
sample of the same workload; it is a deliberately slow baseline, not a target.
"""
import argparse
import json
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "moe_layer_fwd_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram bytes (read + write) of one launch of the dominant kernel from the committed ncu capture, keyed by config
# (None until a capture exists for that workload; see profiles/).
NCU_TRAFFIC_BYTES = {"qwen3_30b_a3b": 1.420e9}   # profiles/gemm_kernels_qwen3_30b_a3b.md: 1.189 GB read + 0.231 GB written


def parse():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=300)
    p.add_argument("--warmup", type=int, default=20)
    p.add_argument("--config", default="qwen3_30b_a3b")
    p.add_argument("--impl", default="mok", choices=["mok", "reference"])
    p.add_argument("--tokens", type=int, default=0, help="override T (small-T sweeps)")
    p.add_argument("--cpu-sample", type=int, default=0, help="tokens of the CPU-oracle sample (0 = auto)")
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--gather-mode", type=int, default=0, help="0 auto, 1 fused into the GEMM, 2 separate kernel")
    p.add_argument("--cta-group", type=int, default=0, help="0 default, 1 single CTAs, 2 CTA pairs")
    p.add_argument("--gemm", type=int, default=0, help="0 tcgen05 (tokens on M), 2 tcgen05 (tokens on N), 1 SIMT")
    p.add_argument("--tile-sched", type=int, default=0, help="routed GEMMs: 0 persistent grid, 1 tiles stolen through cluster launch control")
    p.add_argument("--host-chunks", type=int, default=0, help="token chunks of the host-buffer call (0 = auto)")
    p.add_argument("--precision", default="bf16", choices=["bf16", "mxfp8"],
                   help="routed experts in bf16 (the headline workload) or MXFP8 with pre-quantised weights")
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
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.06)
        self.proc.terminate()
        out, _ = self.proc.communicate(timeout=10)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [v.strip() for v in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def cpu_oracle_rate(cfg, d, sample):
    """tokens/s of the oracle as it stands on the host cores: routing of all T tokens (its per-token share is
    charged to the sample) plus the per-token FFN of `sample` tokens."""
    import numpy as np
    from oracle import mok_ref
    t0 = time.perf_counter()
    idx, w, gap, lg = mok_ref.route(d["x"], d["W_r"], d["bias"], cfg.k)
    t_route = time.perf_counter() - t0
    tokens = np.arange(min(sample, cfg.T), dtype=np.int32)
    t0 = time.perf_counter()
    mok_ref.ffn_tokens(d["x"], d["W_gate_up"], d["W_down"], d["W_sgu"], d["W_sd"], idx, w, tokens)
    t_ffn = time.perf_counter() - t0
    t = t_ffn + t_route * len(tokens) / cfg.T
    return len(tokens) / t, t_ffn + t_route, mok_ref.num_threads()


def fingerprints(d, limit=1 << 31):
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


def auto_sample(cfg, cores):
    # aim at ~15 s of CPU work; the scalar oracle sustains about 4 fp64 GFLOP/s per core on the GPU hosts
    per_token = 6.0 * cfg.H * (cfg.k * cfg.I + cfg.I_s)
    n = int(15.0 * 4.0e9 * cores / per_token)
    return max(16, min(cfg.T, n))


def run_reference(args, cfg, rank):
    """The CPU oracle as the reference arm.  Rank 0 only."""
    if rank != 0:
        return
    from paper_2609_36070_b200 import inputs
    d = inputs.make_inputs(cfg)
    cores = os.cpu_count() or 1
    steps = max(1, min(args.steps, 3))
    sample = args.cpu_sample or max(16, auto_sample(cfg, cores) // (steps + min(args.warmup, 1)))
    for _ in range(min(args.warmup, 1)):
        cpu_oracle_rate(cfg, d, sample)
    rates = []
    t_total = 0.0
    for _ in range(steps):
        r, t, threads = cpu_oracle_rate(cfg, d, sample)
        rates.append(r)
        t_total += t
    value = sum(rates) / len(rates)
    line = {"metric": METRIC, "value": value, "unit": UNIT, "impl": "reference", "n_gpus": args.gpus, "steps": steps,
            "warmup": min(args.warmup, 1), "ms_per_step": 1e3 * t_total / steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "T": cfg.T, "H": cfg.H, "E": cfg.E, "k": cfg.k, "I": cfg.I, "I_shared": cfg.I_s},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": f"routing of all {cfg.T} tokens (charged pro rata) + fp64 FFN of the first {sample} tokens per step"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gflops": value * 6.0 * cfg.H * (cfg.k * cfg.I + cfg.I_s) / 1e9}
    print(json.dumps(line), flush=True)


def run_backward(args, cfg):
    """Times mok_moe_backward (activation recomputation, dx, router-weight and weight gradients) on one GPU.  FLOPs
    are counted as twice the forward pass's (dgrad + wgrad), as in the paper's Section 4.1; the recomputed gate/up
    product and the transposes are extra work that is not counted."""
    import numpy as np
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
    idx, w = st["topk_idx"], st["topk_w"]
    rng = np.random.default_rng(1)
    dout = mok.to_device_bf16(inputs.f32_to_bf16_bits(rng.standard_normal((cfg.T, cfg.H), dtype=np.float32)), dev)
    res = mok.mok_moe_backward(g["x"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], idx, w, dout)
    bws = res["workspace"]
    conf = mok._config(cta_group=args.cta_group)

    def step():
        mok.mok_moe_backward(g["x"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], idx, w, dout, workspace=bws,
                             config=conf)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = ev0.elapsed_time(ev1) / args.steps
    assert mok.mok_read_status(bws) == 0
    flops = 2.0 * cfg.ffn_flops()
    print(json.dumps({"metric": "moe_layer_bwd_tokens_per_s", "value": cfg.T / (ms * 1e-3), "unit": UNIT, "n_gpus": 1,
                      "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
                      "dtype": "bf16", "data": "synthetic", "tflops": flops / (ms * 1e-3) / 1e12,
                      "config": {"workload": cfg.name, "T": cfg.T, "H": cfg.H, "E": cfg.E, "k": cfg.k, "I": cfg.I,
                                 "I_shared": cfg.I_s, "pass": "backward (recompute + dgrad + wgrad)"},
                      "clocks": clocks}), flush=True)


def main():
    args = parse()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    from paper_2609_36070_b200 import inputs
    cfg = inputs.CONFIGS[args.config]
    if args.tokens:
        cfg = cfg.with_tokens(args.tokens)
    if args.impl == "reference":
        run_reference(args, cfg, rank)
        return
    if args.which == "backward":
        if rank == 0:
            run_backward(args, cfg)
        return

    import numpy as np
    import torch
    from paper_2609_36070_b200 import mok
    assert args.warmup >= 3, "timing rules: at least 3 warm-up steps"
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    # every rank: same weights, its own batch (seed offset by rank)
    from paper_2609_36070_b200 import sharding
    d = inputs.make_inputs(cfg)
    if rank > 0:
        d["x"] = sharding.rank_tokens(cfg, rank)
    g = {k: (None if d[k] is None else mok.to_device_bf16(d[k], dev)) for k in ("x", "W_gate_up", "W_down", "W_sgu", "W_sd")}
    W_r = torch.from_numpy(d["W_r"]).to(dev)
    bias = None if d["bias"] is None else torch.from_numpy(d["bias"]).to(dev)
    mx = args.precision == "mxfp8"
    prec = mok.MOK_PRECISION_MXFP8 if mx else mok.MOK_PRECISION_BF16
    mxw = mok.MxWeights(g["W_gate_up"], g["W_down"]) if mx else None    # weights are quantised ahead of time
    ws = mok.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, device=dev, host_staging=2, mx=mx)
    out = torch.empty_like(g["x"])
    conf = mok._config(impl=args.gemm, profile=1, gather_mode=args.gather_mode, cta_group=args.cta_group, precision=prec,
                       tile_sched=args.tile_sched)

    def step():
        mok.mok_moe_forward_ex(g["x"], W_r, bias, g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k, ws,
                               out=out, config=conf, mx_weights=mxw)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    status = mok.mok_read_status(ws)
    assert status == 0, mok.mok_status_string(status)

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    mok.mok_profile_begin(args.steps)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    barrier()
    total_ms = ev0.elapsed_time(ev1)
    stage = mok.mok_profile_end(args.steps)
    clocks = sampler.stop() if rank == 0 else None
    status = mok.mok_read_status(ws)
    assert status == 0, mok.mok_status_string(status)

    total_ms = sharding.max_over_ranks(total_ms, dist, dev)
    ms_per_step = total_ms / args.steps
    value = sharding.aggregate_tokens_per_s(cfg.T, world, ms_per_step)
    flops = cfg.ffn_flops()
    tflops = world * flops / (ms_per_step * 1e-3) / 1e12

    # End to end through the host-buffer entry points: pinned host x -> device, layer, result -> pinned host, every step.
    # Throughput (`e2e.value`): a stream of batches through the asynchronous call, whose two staging slots let the upload
    # of step i+1 and the download of step i-1 overlap the layer of step i; the timed region ends when the last result
    # has arrived in host memory.  Latency of ONE isolated batch (`e2e.single_call_ms`): the blocking call, which cuts
    # the batch into token chunks to overlap its own copies.
    xh = g["x"].cpu().pin_memory()
    oh = [torch.empty_like(xh).pin_memory() for _ in range(2)]
    conf0 = mok._config(impl=args.gemm, gather_mode=args.gather_mode, cta_group=args.cta_group, host_chunks=args.host_chunks,
                        precision=prec)

    def e2e_submit(i):
        mok.mok_moe_forward_host_async(xh, oh[i & 1], W_r, bias, g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k,
                                       ws, config=conf0, mx_weights=mxw)

    def single_call():
        mok.mok_moe_forward_host(xh, oh[0], W_r, bias, g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k, ws,
                                 config=conf0, mx_weights=mxw)

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
    e2e_ms = ev0.elapsed_time(ev1) / e2e_steps
    e2e_ms = sharding.max_over_ranks(e2e_ms, dist, dev)
    for _ in range(2):
        single_call()
    barrier()
    ev0.record()
    for _ in range(5):
        single_call()
    ev1.record()
    barrier()
    single_ms = sharding.max_over_ranks(ev0.elapsed_time(ev1) / 5, dist, dev)
    act_bytes = 2 * cfg.T * cfg.H

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    pk = peaks()
    mean = {s: float(np.mean([c[s] for c in stage])) for s in mok.STAGES}
    # dominant kernel: the routed gate/up grouped GEMM with the SwiGLU epilogue (one launch per step)
    g1_flops = 4.0 * cfg.T * cfg.k * cfg.H * cfg.I
    g1_tflops = g1_flops / (mean["gemm1"] * 1e-3) / 1e12
    peak_tf = pk.get("bf16_tflops_sustained", pk["bf16_tflops"])
    if mx:   # fp8 tensor peak = the measured bf16 peak x the nominal 2:1 ratio (4.5 vs 2.25 PFLOP/s dense)
        peak_tf *= 2.0
    per_step = sorted(sum(c[s] for s in mok.STAGES) for c in stage)
    ffn_ms = mean["gemm1"] + mean["gemm2"] + mean["shared_gemm1"] + mean["shared_gemm2"]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "mxfp8 routed experts (fp32 accumulate), bf16 elsewhere" if mx else "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "T": cfg.T, "H": cfg.H, "E": cfg.E, "k": cfg.k, "I": cfg.I,
                   "I_shared": cfg.I_s, "routing": cfg.bias, "parallelism": f"token-sharded replicas x{world}",
                   "l2": "inputs larger than L2 (weights + activations >> 126 MB), no explicit flush"},
        "tflops": tflops,
        "tflops_frac_of_peak": tflops / world / pk["bf16_tflops"],
        "ffn_phase": {"ms": ffn_ms, "tflops": flops / (ffn_ms * 1e-3) / 1e12,
                      "frac_of_bf16_peak": flops / (ffn_ms * 1e-3) / 1e12 / pk["bf16_tflops"],
                      "frac_of_bf16_sustained": flops / (ffn_ms * 1e-3) / 1e12 / peak_tf},
        "stage_ms": mean,
        "median_step_ms_from_stage_events": per_step[len(per_step) // 2],
        "inputs": fingerprints(d),
        "roofline": {"kernel": ("routed gate/up grouped GEMM on MXFP8 operands + SwiGLU + activation quantisation, token gather fused "
                                "(gemm_mx_kernel<EPI_SWIGLU, GATHER>)") if mx else
                               "routed gate/up grouped GEMM + SwiGLU, token gather fused (gemm_m2_kernel<EPI_SWIGLU, GATHER>)",
                     "bound": "tensor",
                     "achieved": g1_tflops, "peak": peak_tf, "unit": "TFLOP/s", "frac": g1_tflops / peak_tf,
                     "peak_source": f"{pk['source']} bf16_tflops_sustained" + (" x 2 (nominal fp8 : bf16 ratio)" if mx else ""),
                     "traffic": None if mx else NCU_TRAFFIC_BYTES.get(cfg.name)},
        "e2e": {"value": world * cfg.T / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": act_bytes, "d2h_bytes_per_step": act_bytes,
                "mode": "stream of batches through mok_moe_forward_host_async (two staging slots), timed until the last "
                        "result is in host memory",
                "single_call_ms": single_ms},
        "gpu_launches": args.steps * mok.mok_launch_count(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, conf),
        "clocks": clocks,
    }
    if not args.no_cpu_baseline:
        cores = os.cpu_count() or 1
        sample = args.cpu_sample or auto_sample(cfg, cores)
        rate, secs, threads = cpu_oracle_rate(cfg, d, sample)
        line["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": secs,
                                "sample": f"routing of all {cfg.T} tokens (charged pro rata) + fp64 FFN of the first {min(sample, cfg.T)} tokens"}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
