"""Expert parallelism on one GPU with emulated ranks: the device-side Algorithm 1 for R source ranks against the
oracle's statement-by-statement version (bit-exact), and the whole expert-parallel layer (local routing, gathered
routes, schedule, pull dispatch into the grouped GEMMs, owner-side combine) against the oracle's per-token
definition and against the one-rank layer on the concatenated batch.  Every rank's buffers live on the same GPU, so a
local pointer stands in for a peer pointer; kernels and schedules are exactly those of the multi-GPU path."""
import numpy as np
import pytest
import torch

from oracle import mok_ref
from paper_2609_36070_b200 import inputs
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def mok():
    from paper_2609_36070_b200 import mok as m
    return m


def skewed_routes(rng, R, T_local, E, k, skew):
    """Distinct experts per token; expert popularity ~ 1/(e+1)^skew, shifted per source rank so that ranks differ."""
    idx = np.empty((R, T_local, k), np.int32)
    base = 1.0 / np.arange(1, E + 1) ** skew
    for r in range(R):
        p = np.roll(base, 3 * r)
        p = p / p.sum()
        for t in range(T_local):
            idx[r, t] = rng.choice(E, size=k, replace=False, p=p)
    return idx.reshape(R, T_local * k)


# (R, T_local, E, k, skew): ragged block tails, several blocks per rank, empty experts, one expert per rank, R = 1
ALG1_CASES = [(2, 64, 8, 2, 0.0), (4, 300, 16, 4, 1.2), (8, 129, 64, 8, 1.1), (3, 1500, 12, 3, 2.0),
              (2, 2100, 4, 2, 0.5), (8, 64, 8, 1, 0.0), (1, 777, 16, 4, 1.0), (16, 40, 32, 2, 3.0)]


@pytest.mark.parametrize("R,T_local,E,k,skew", ALG1_CASES)
def test_device_algorithm1_matches_oracle(R, T_local, E, k, skew):
    m = mok()
    rng = np.random.default_rng(1000 * R + T_local)
    A = skewed_routes(rng, R, T_local, E, k, skew)
    L = E // R
    n = T_local * k
    idx_all = torch.from_numpy(A).cuda()
    ws = torch.empty(m.mok_ep_workspace_bytes(R, T_local, 64, 64, 0, E, k) + 256, dtype=torch.uint8, device="cuda")
    for c in range(R):
        pos = torch.full((R * n,), -7, dtype=torch.int32, device="cuda")
        t = m.mok_ep_expert_ffn(c, None, idx_all, None, None, None, None, E, k, None, pos, None, ws, 64,
                                schedule_only=True, outputs=True)
        assert m.mok_read_status(ws) == 0
        S, pr, pi = mok_ref.alg1(A, L, c)
        total = int(S[L])
        assert np.array_equal(t["S"].cpu().numpy(), S)
        assert np.array_equal(t["phi_rank"].cpu().numpy()[:total], pr)
        assert np.array_equal(t["phi_index"].cpu().numpy()[:total], pi)
        # M is a plain count: routes of rank r to local expert l
        M = np.stack([np.bincount(A[r][(A[r] >= c * L) & (A[r] < (c + 1) * L)] - c * L, minlength=L) for r in range(R)])
        assert np.array_equal(t["M"].cpu().numpy(), M)
        # pos: the row of y of every served route = its schedule position moved into the 128-row-padded space
        counts = np.diff(S)
        pad_off = np.concatenate([[0], np.cumsum((counts + 127) // 128 * 128)])
        want = np.full(R * n, -7, np.int64)
        for l in range(L):
            p = np.arange(S[l], S[l + 1])
            want[pr[p].astype(np.int64) * n + pi[p]] = pad_off[l] + (p - S[l])
        assert np.array_equal(pos.cpu().numpy().astype(np.int64), want)


def ep_case(cfg, R, config=None):
    m = mok()
    from paper_2609_36070_b200 import ep
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    T_local = cfg.T // R
    xs = [g["x"][r * T_local:(r + 1) * T_local].contiguous() for r in range(R)]
    outs = ep.forward_emulated(xs, g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k,
                               config=config)
    out = torch.cat(outs)
    # the one-rank layer on the concatenated batch: same routing, same per-row arithmetic, same combine order
    one, st = pu.run_gpu(cfg, g)
    idx, w, rep = pu.check_routing_and_schedule(cfg, d, st)
    rep.update(pu.check_output(cfg, d, out, idx, w, np.arange(cfg.T, dtype=np.int32)))
    rep["bitwise_equal_to_one_rank"] = bool(torch.equal(out.view(torch.int16), one.view(torch.int16)))
    return rep


@pytest.mark.parametrize("R", [1, 2, 4, 8])
def test_expert_parallel_layer_tiny(R):
    rep = ep_case(inputs.CONFIGS["tiny"], R)
    assert rep["bitwise_equal_to_one_rank"], rep


EP_SHAPES = [
    # name, T, H, E, k, I, I_s, bias, R
    ("skewed_4_ranks", 1024, 512, 32, 4, 384, 0, "zipf", 4),
    ("shared_expert_2_ranks", 768, 256, 16, 2, 256, 256, "none", 2),
    ("one_expert_per_rank", 512, 256, 8, 2, 512, 0, "none", 8),
    ("ragged_sizes_3_ranks", 3 * 150, 264, 12, 3, 200, 72, "normal", 3),
]


@pytest.mark.parametrize("name,T,H,E,k,I,I_s,bias,R", EP_SHAPES)
def test_expert_parallel_layer_shapes(name, T, H, E, k, I, I_s, bias, R):
    cfg = inputs.MoEConfig(name, T, H, E, k, I, I_s, bias=bias, seed=11)
    rep = ep_case(cfg, R)
    assert rep["bitwise_equal_to_one_rank"], rep


@pytest.mark.parametrize("R", [1, 2, 4])
@pytest.mark.parametrize("kw", [{"fused_ffn": 2}, {"fused_ffn": 2, "tile_sched": 2, "gang_sync": 2},
                                {"fused_ffn": 2, "fused_window": -1, "grid": 7}, {"comm_ctas": 6},
                                {"comm_ctas": 12, "tile_sched": 2, "gang_sync": 2}],
                         ids=["dynamic", "static_gang", "no_window", "comm_ctas", "comm_ctas_static"])
def test_expert_parallel_layer_with_the_one_launch_expert_ffn(R, kw):
    """The routed experts of every rank as ONE persistent launch (gate/up tiles pull their rows from the owners'
    buffers, down tiles wait on the completion counters and store into the peer-visible y): every token against the
    oracle and bit for bit the one-rank layer, on a shape with several row tiles per expert and a shared expert.
    With comm_ctas the pulls are made by communication CTAs into staging slots a row tile ahead of their use."""
    m = mok()
    cfg = inputs.MoEConfig("ep_one_launch", 3072, 512, 8, 3, 320, 128, bias="zipf", seed=12)
    rep = ep_case(cfg, R, config=m._config(**kw))
    assert rep["bitwise_equal_to_one_rank"], rep


def test_expert_parallel_is_reproducible_and_independent_of_the_kernel_choice():
    cfg = inputs.MoEConfig("ep_repro", 1024, 512, 16, 4, 512, 0, bias="zipf", seed=5)
    m = mok()
    from paper_2609_36070_b200 import ep
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    xs = [g["x"][r * 256:(r + 1) * 256].contiguous() for r in range(4)]
    runs = []
    for config in (None, None, m._config(cta_group=1), m._config(cta_group=3), m._config(grid=7)):
        outs = ep.forward_emulated(xs, g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], None, None, cfg.k, config=config)
        runs.append(torch.cat(outs).view(torch.int16).clone())
    for r in runs[1:]:
        assert torch.equal(r, runs[0])


def test_expert_parallel_argument_errors():
    m = mok()
    a = m.mok_ep_args()
    a.rank, a.n_ranks, a.T_local, a.H, a.I, a.E, a.k = 0, 3, 64, 64, 64, 8, 2      # E not a multiple of n_ranks
    assert m._lib.mok_ep_expert_ffn(a) == m.MOK_ERR_SHAPE
    a.n_ranks = 17
    assert m._lib.mok_ep_expert_ffn(a) == m.MOK_ERR_SHAPE
    a.n_ranks, a.rank = 2, 2
    assert m._lib.mok_ep_expert_ffn(a) == m.MOK_ERR_SHAPE
    a.rank = 1
    assert m._lib.mok_ep_expert_ffn(a) == m.MOK_ERR_NULL                           # idx_all missing
    assert m._lib.mok_ep_expert_ffn(None) == m.MOK_ERR_NULL
    assert m.mok_ep_workspace_bytes(3, 64, 64, 64, 0, 8, 2) == 0
    assert m.mok_ep_y_rows(2, 64, 8, 2) >= 2 * 64 * 2
    c = m.mok_ep_combine_args()
    c.rank, c.n_ranks, c.T_local, c.H, c.E, c.k = 0, 2, 64, 64, 8, 2
    assert m._lib.mok_ep_combine(c) == m.MOK_ERR_NULL
    c.E = 7
    assert m._lib.mok_ep_combine(c) == m.MOK_ERR_SHAPE


def test_distributed_driver_with_a_world_of_one_rank():
    """The torch.distributed driver (symmetric-memory buffers, route all-gather, barriers) run as its own process with
    one rank: the plumbing of the multi-GPU path on the one GPU available, checked bit for bit against the one-rank
    layer by the module's own self-check."""
    import json
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29547", RANK="0", WORLD_SIZE="1", LOCAL_RANK="0",
               NCCL_NVLS_ENABLE="0", TORCH_SYMM_MEM_DISABLE_MULTICAST="1")
    r = subprocess.run([sys.executable, "-m", "paper_2609_36070_b200.ep", "--config", "tiny", "--steps", "3"],
                       cwd=root, env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
    line = json.loads([l for l in r.stdout.splitlines() if l.startswith("{")][-1])
    assert line["bitwise_equal_to_one_rank_layer"] and line["n_ranks"] == 1


def test_bench_expert_parallel_mode_as_a_world_of_one_rank():
    """`bench.py --parallelism ep` (one process per GPU, symmetric memory, NCCL) run alone: it prints the bench's JSON
    line with the expert-parallel phases, and its host-buffer leg returns the bits of the device-resident leg."""
    import json
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29549", RANK="0", WORLD_SIZE="1", LOCAL_RANK="0",
               NCCL_NVLS_ENABLE="0", TORCH_SYMM_MEM_DISABLE_MULTICAST="1")
    r = subprocess.run([sys.executable, "bench.py", "--parallelism", "ep", "--config", "tiny", "--steps", "5",
                        "--warmup", "3"], cwd=root, env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
    line = json.loads([l for l in r.stdout.splitlines() if l.startswith("{")][-1])
    assert line["config"]["parallelism"] == "ep1" and line["n_gpus"] == 1 and line["value"] > 0
    assert line["bitwise_equal_to_one_rank_layer"] is True
    assert set(line["phase_ms"]) == {"stage_x", "route", "gather_routes", "expert_ffn", "barrier", "combine"}
    assert line["e2e"]["result_bits_equal_device_call"] and line["e2e"]["h2d_bytes_per_step"] > 0
    assert line["gpu_launches"] > 0 and line["roofline"]["frac"] > 0


@pytest.mark.parametrize("world,mx", [(2, False), (4, False), (2, True)], ids=["2_ranks", "4_ranks", "2_ranks_mxfp8"])
def test_ranks_as_separate_processes_on_one_gpu(world, mx):
    """Real cross-process peer pointers: every rank is its own process on GPU 0, maps the other ranks' x / y / pos
    buffers through CUDA IPC, and runs the expert-parallel layer with gloo collectives (routes staged through the
    host).  No kernel waits on another rank's kernel, so sharing one GPU is safe; each rank checks its output bit for
    bit against the one-rank layer and, in bf16 mode, runs the backward pass twice on the same buffers and checks dx and
    dw bit for bit against the one-rank backward pass."""
    from paper_2609_36070_b200 import ep
    assert ep.check_processes_on_one_gpu(world=world, config_name="tiny", port=29561 + world + 10 * int(mx), mx=mx)


@pytest.mark.parametrize("kw,port", [({"fused_ffn": 2}, 29591), ({"comm_ctas": 2}, 29593)], ids=["one_launch", "comm_ctas"])
def test_ranks_as_separate_processes_with_the_one_launch_kernel(kw, port):
    """Two processes on GPU 0, the Qwen3-like shapes with 2048 tokens, the routed experts of each rank as the one-launch
    kernel: its gather warps (or, with comm_ctas, the bulk copies of its communication CTAs) read the other process's
    token rows through a CUDA IPC mapping; each rank's output must equal its slice of the one-rank layer bit for bit,
    and so must dx and dw of the backward pass."""
    from paper_2609_36070_b200 import ep
    assert ep.check_processes_on_one_gpu(world=2, config_name="qwen3_30b_a3b", port=port, tokens=2048, config_kw=kw)


@pytest.mark.parametrize("R", [1, 2, 4])
def test_expert_parallel_mxfp8_equals_the_one_rank_mxfp8_layer(R):
    """The paper's main configuration: expert parallelism with MXFP8 routed experts (Section 3.4).  Every rank quantises
    its own token rows; the serving rank's gather warps pull codes and scales from the owner; the result is bitwise the
    one-rank MXFP8 layer on the concatenated batch (which the MXFP8 tests check against the oracle)."""
    m = mok()
    from paper_2609_36070_b200 import ep
    cfg = inputs.MoEConfig("ep_mx", 1024, 512, 16, 4, 384, 256, bias="zipf", seed=6)
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    T_local = cfg.T // R
    xs = [g["x"][r * T_local:(r + 1) * T_local].contiguous() for r in range(R)]
    out = torch.cat(ep.forward_emulated(xs, g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"],
                                        cfg.k, mx=True))
    one, rep = pu.mx_parity(cfg, d=d, g=g)
    assert torch.equal(out.view(torch.int16), one.view(torch.int16)), rep


EP_BWD = [
    # name, T, H, E, k, I, I_s, bias: ragged segments, empty experts, a shared expert, several row tiles per expert
    ("shared", 512, 256, 8, 2, 512, 256, "none"),
    ("skewed", 1024, 512, 32, 4, 384, 0, "zipf"),
    ("many_rows", 3072, 256, 4, 2, 160, 64, "normal"),
]


@pytest.mark.parametrize("R", [1, 2, 4])
@pytest.mark.parametrize("name,T,H,E,k,I,I_s,bias", EP_BWD)
def test_expert_parallel_backward(name, T, H, E, k, I, I_s, bias, R):
    """The backward pass under expert parallelism (emulated ranks: serving side of every rank, barrier, owner side).
    dx and dw must equal the one-rank backward pass on the concatenated batch bit for bit (every row goes through the
    same products, the owner sums its k rows in slot order); the weight gradients sum an expert's rows in Algorithm 1's
    order, so they are compared with the oracle's fp64 chain rule within the backward tolerances (and, for one rank,
    where that order is the token order, bit for bit with the one-rank pass)."""
    from paper_2609_36070_b200 import ep
    m = mok()
    cfg = inputs.MoEConfig("epbwd_" + name, T, H, E, k, I, I_s, bias=bias, seed=61)
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    out, st = pu.run_gpu(cfg, g)
    idx, w = st["topk_idx"], st["topk_w"]
    rng = np.random.default_rng(cfg.seed + 7)
    dout_bits = inputs.f32_to_bf16_bits(rng.normal(0, 1, (cfg.T, cfg.H)).astype(np.float32))
    dout = m.to_device_bf16(dout_bits)
    one = m.mok_moe_backward(g["x"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], idx, w, dout)
    Tl = T // R
    cut = lambda t: [t[r * Tl:(r + 1) * Tl].contiguous() for r in range(R)]
    res = ep.backward_emulated(cut(g["x"]), cut(dout), cut(idx), cut(w), g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"])
    dx = torch.cat([r["dx"] for r in res])
    dw = torch.cat([r["dw"] for r in res])
    assert torch.equal(dx.view(torch.int16), one["dx"].view(torch.int16))
    assert torch.equal(dw.view(torch.int32), one["dw"].view(torch.int32))
    got = {"dW_gate_up": torch.cat([r["dW_gate_up"] for r in res]).float(),
           "dW_down": torch.cat([r["dW_down"] for r in res]).float()}
    if I_s:     # every rank holds the shared expert and contributes its own tokens' share
        got["dW_sgu"] = sum(r["dW_shared_gate_up"].float() for r in res)
        got["dW_sd"] = sum(r["dW_shared_down"].float() for r in res)
    if R == 1:
        assert torch.equal(res[0]["dW_gate_up"].view(torch.int16), one["dW_gate_up"].view(torch.int16))
        assert torch.equal(res[0]["dW_down"].view(torch.int16), one["dW_down"].view(torch.int16))
    ref = mok_ref.backward(d["x"], d["W_gate_up"], d["W_down"], d["W_sgu"], d["W_sd"], idx.cpu().numpy(),
                           w.cpu().numpy().astype(np.float64), inputs.bf16_bits_to_f32(dout_bits).astype(np.float64),
                           weights=True)
    for name_, t in got.items():
        a, b = t.cpu().numpy().astype(np.float64), ref[name_]
        diff = np.abs(a - b)
        assert np.isfinite(a).all(), name_
        assert diff.max() <= 2e-2 * np.abs(b).max() and diff.mean() <= 1e-2 * np.abs(b).mean(), (name_, R)
