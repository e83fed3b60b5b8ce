"""Backward pass on the GPU against the CPU oracle (the chain rule of the layer definition in fp64) on the same seeded
inputs: activation gradient dx, router-weight gradient dw and the weight gradients, every element, on shapes that span
several tiles, ragged expert segments, empty experts and a shared expert.  Tolerances: the backward chain rounds five
intermediates to bf16 (pre-activations, dL/dh, dg|du, dXg or the transposed operands, the result) where the forward
rounds three, so the bounds are twice the forward pass's: max|gpu - ref| <= 2e-2 max|ref| and
mean|gpu - ref| <= 1e-2 mean|ref| per tensor."""
import numpy as np
import pytest
import torch

from oracle import mok_ref
from paper_2609_36070_b200 import inputs
from tests import parity_util as pu

pytestmark = pytest.mark.gpu

MAX_REL_BWD, MEAN_REL_BWD = 2e-2, 1e-2


def mok():
    from paper_2609_36070_b200 import mok as m
    return m


def run_case(cfg, weight_grads=True, config=None, wscale=None):
    m = mok()
    d = inputs.make_inputs(cfg)
    if wscale:                                                   # larger weights: silu' away from its linear range
        rng = np.random.default_rng(cfg.seed + 100)
        for name in ("W_gate_up", "W_down", "W_sgu", "W_sd"):
            if d[name] is not None:
                d[name] = inputs.f32_to_bf16_bits(rng.normal(0, wscale, d[name].shape).astype(np.float32))
    g = pu.upload(d)
    out, st = pu.run_gpu(cfg, g)
    idx = st["topk_idx"]
    w = st["topk_w"]
    rng = np.random.default_rng(cfg.seed + 7)
    dout_bits = inputs.f32_to_bf16_bits(rng.normal(0, 1, (cfg.T, cfg.H)).astype(np.float32))
    dout = m.to_device_bf16(dout_bits)
    res = m.mok_moe_backward(g["x"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], idx, w, dout,
                             weight_grads=weight_grads, config=config)
    torch.cuda.synchronize()
    assert m.mok_read_status(res["workspace"]) == 0
    ref = mok_ref.backward(d["x"], d["W_gate_up"], d["W_down"], d["W_sgu"], d["W_sd"], idx.cpu().numpy(),
                           w.cpu().numpy().astype(np.float64), inputs.bf16_bits_to_f32(dout_bits).astype(np.float64),
                           weights=weight_grads)
    rep = {}
    names = {"dx": "dx", "dw": "dw", "dW_gate_up": "dW_gate_up", "dW_down": "dW_down", "dW_shared_gate_up": "dW_sgu",
             "dW_shared_down": "dW_sd"}
    for gname, rname in names.items():
        if gname not in res or rname not in ref:
            continue
        got = res[gname].float().cpu().numpy().astype(np.float64)
        want = ref[rname]
        assert np.isfinite(got).all(), gname
        diff = np.abs(got - want)
        rep[gname] = (float(diff.max() / np.abs(want).max()), float(diff.mean() / np.abs(want).mean()))
        assert rep[gname][0] <= MAX_REL_BWD and rep[gname][1] <= MEAN_REL_BWD, (gname, rep[gname])
    return res, rep


SHAPES = [
    # name, T, H, E, k, I, I_s, bias
    ("tiny", 256, 256, 8, 2, 512, 512, "none"),
    ("ragged", 300, 288, 4, 2, 160, 0, "normal"),
    ("skewed_empty_experts", 1024, 512, 32, 4, 384, 0, "zipf"),
    ("shared_wider_than_routed", 200, 128, 4, 2, 64, 256, "none"),
    ("one_route", 130, 64, 2, 1, 32, 0, "none"),
    ("wide_experts_expert_sorted_copies", 200, 64, 3, 2, 2080, 0, "none"),   # I > 2048: rows of x / dout copied once, not pulled
]


@pytest.mark.parametrize("name,T,H,E,k,I,I_s,bias", SHAPES)
def test_activation_and_router_weight_gradients(name, T, H, E, k, I, I_s, bias):
    cfg = inputs.MoEConfig("bwd_" + name, T, H, E, k, I, I_s, bias=bias, seed=51)
    res, rep = run_case(cfg, weight_grads=False)
    print(name, rep)


@pytest.mark.parametrize("name,T,H,E,k,I,I_s,bias", SHAPES)
def test_weight_gradients(name, T, H, E, k, I, I_s, bias):
    cfg = inputs.MoEConfig("bwd_" + name, T, H, E, k, I, I_s, bias=bias, seed=51)
    res, rep = run_case(cfg, weight_grads=True)
    print(name, rep)


def test_gradients_with_large_weights():
    cfg = inputs.MoEConfig("bwd_large_w", 384, 128, 4, 2, 128, 64, seed=52)
    res, rep = run_case(cfg, weight_grads=True, wscale=0.15)
    print(rep)


def test_backward_is_reproducible_and_grid_independent():
    m = mok()
    cfg = inputs.MoEConfig("bwd_repro", 512, 256, 16, 4, 256, 128, bias="zipf", seed=53)
    runs = []
    for conf in (None, None, m._config(grid=3), m._config(cta_group=1), m._config(gather_mode=2)):
        res, _ = run_case(cfg, weight_grads=False, config=conf)
        runs.append((res["dx"].view(torch.int16).clone(), res["dw"].view(torch.int32).clone()))
    for dx, dw in runs[1:]:
        assert torch.equal(dx, runs[0][0]) and torch.equal(dw, runs[0][1])


def test_bench_shape_with_fewer_tokens_all_gradients():
    """The benchmark layer (H = 2048, E = 128, k = 8, I = 768, Zipf routing: hot and empty experts) at T = 2048, where
    the oracle can still evaluate every weight gradient."""
    cfg = inputs.CONFIGS["qwen3_30b_a3b"].with_tokens(2048)
    res, rep = run_case(cfg, weight_grads=True)
    print(rep)


def test_bench_shape_full_size_sampled():
    """Full-size Qwen3-like workload: dx and dw of a token sample and the weight gradients of the experts with few routes
    against the oracle, everything finite, run-to-run bitwise."""
    m = mok()
    cfg = inputs.CONFIGS["qwen3_30b_a3b"]
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    out, st = pu.run_gpu(cfg, g)
    idx, w = st["topk_idx"], st["topk_w"]
    rng = np.random.default_rng(77)
    dout_bits = inputs.f32_to_bf16_bits(rng.normal(0, 1, (cfg.T, cfg.H)).astype(np.float32))
    dout = m.to_device_bf16(dout_bits)
    res = m.mok_moe_backward(g["x"], g["W_gate_up"], g["W_down"], None, None, idx, w, dout)
    torch.cuda.synchronize()
    assert m.mok_read_status(res["workspace"]) == 0
    tokens = inputs.sample_tokens(cfg, idx.cpu().numpy(), 256)
    dx_ref, dw_ref = mok_ref.backward_tokens(d["x"], d["W_gate_up"], d["W_down"], None, None, idx.cpu().numpy(),
                                             w.cpu().numpy().astype(np.float64),
                                             inputs.bf16_bits_to_f32(dout_bits).astype(np.float64), tokens)
    sel = torch.from_numpy(np.asarray(tokens, np.int64)).cuda()
    for got, want, name in ((res["dx"][sel], dx_ref, "dx"), (res["dw"][sel], dw_ref, "dw")):
        got = got.float().cpu().numpy().astype(np.float64)
        diff = np.abs(got - want)
        assert diff.max() <= MAX_REL_BWD * np.abs(want).max() and diff.mean() <= MEAN_REL_BWD * np.abs(want).mean(), name
    for name in ("dW_gate_up", "dW_down"):
        assert torch.isfinite(res[name].float()).all()
    # Weight gradients at full size: an expert's gradient only depends on the tokens routed to it, so for the experts
    # with few routes the oracle evaluates a one-expert layer on exactly those tokens (the route's weight as its only
    # combine weight) -- the same sums, cheap in fp64.  Experts without routes must come out as exact zeros.
    idx_h, w_h = idx.cpu().numpy(), w.cpu().numpy().astype(np.float64)
    counts = np.bincount(idx_h.ravel(), minlength=cfg.E)
    dout64 = inputs.bf16_bits_to_f32(dout_bits).astype(np.float64)
    small = [e for e in np.argsort(counts) if 0 < counts[e] <= 64][:6]
    assert small, "the Zipf routing of this workload has experts with a handful of routes"
    for e in small:
        toks, slots = np.nonzero(idx_h == e)
        sub = mok_ref.backward(np.ascontiguousarray(d["x"][toks]), d["W_gate_up"][e:e + 1], d["W_down"][e:e + 1], None, None,
                               np.zeros((toks.size, 1), np.int32), w_h[toks, slots].reshape(-1, 1),
                               np.ascontiguousarray(dout64[toks]))
        for name in ("dW_gate_up", "dW_down"):
            got = res[name][e].float().cpu().numpy().astype(np.float64)
            want = sub[name][0]
            diff = np.abs(got - want)
            assert diff.max() <= MAX_REL_BWD * np.abs(want).max() and diff.mean() <= MEAN_REL_BWD * np.abs(want).mean(), (name, e)
    for e in np.flatnonzero(counts == 0):
        assert float(res["dW_gate_up"][e].float().abs().max()) == 0.0 and float(res["dW_down"][e].float().abs().max()) == 0.0
    again = m.mok_moe_backward(g["x"], g["W_gate_up"], g["W_down"], None, None, idx, w, dout, workspace=res["workspace"])
    torch.cuda.synchronize()
    for name in ("dx", "dW_gate_up", "dW_down"):
        assert torch.equal(again[name].view(torch.int16), res[name].view(torch.int16)), name
    assert torch.equal(again["dw"].view(torch.int32), res["dw"].view(torch.int32))


def test_backward_argument_errors():
    m = mok()
    assert m._lib.mok_moe_backward(None) == m.MOK_ERR_NULL
    assert m.mok_bwd_workspace_bytes(64, 72, 64, 0, 4, 2) == 0                 # H not a multiple of 32
    assert m.mok_bwd_workspace_bytes(64, 64, 64, 0, 4, 2) > m.mok_workspace_bytes(64, 64, 64, 0, 4, 2)
    a = m.mok_bwd_args()
    a.T, a.H, a.I, a.I_shared, a.E, a.k = 64, 64, 40, 0, 4, 2                  # I not a multiple of 32
    assert m._lib.mok_moe_backward(a) == m.MOK_ERR_SHAPE
    a.I = 64
    assert m._lib.mok_moe_backward(a) == m.MOK_ERR_NULL                        # nothing given
    a.T = 0
    assert m._lib.mok_moe_backward(a) == m.MOK_OK                              # nothing to do
    cfg = inputs.MoEConfig("bwd_err", 64, 64, 4, 2, 64, 0, seed=9)
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    out, st = pu.run_gpu(cfg, g)
    dout = torch.zeros_like(g["x"])
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(m.MokError) as ei:
        m.mok_moe_backward(g["x"], g["W_gate_up"], g["W_down"], None, None, st["topk_idx"], st["topk_w"], dout,
                           workspace=small)
    assert ei.value.status == m.MOK_ERR_WORKSPACE
    with pytest.raises(m.MokError) as ei:                                      # MXFP8 backward is not built
        m.mok_moe_backward(g["x"], g["W_gate_up"], g["W_down"], None, None, st["topk_idx"], st["topk_w"], dout,
                           config=m._config(precision=m.MOK_PRECISION_MXFP8))
    assert ei.value.status == m.MOK_ERR_SHAPE
    res = m.mok_moe_backward(g["x"], g["W_gate_up"], g["W_down"], None, None, st["topk_idx"], st["topk_w"], dout)
    torch.cuda.synchronize()
    assert all(float(res[n].float().abs().max()) == 0.0 for n in ("dx", "dw", "dW_gate_up", "dW_down"))   # dout = 0
