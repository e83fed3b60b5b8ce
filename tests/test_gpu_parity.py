"""GPU parity tests: the CUDA path (through the C-ABI binding) against the CPU oracle, element by element on
small seeded inputs that span several tiles and ragged tails, and on sampled tokens at the full workload sizes."""
import numpy as np
import pytest
import torch

from paper_2609_36070_b200 import inputs
from paper_2609_36070_b200.inputs import MoEConfig

import parity_util as pu
from oracle import mok_ref

pytestmark = pytest.mark.gpu


def mok():
    from paper_2609_36070_b200 import mok as m
    return m


SMALL = [
    # name, T, H, E, k, I, I_s, bias  -- ragged tails everywhere: T, H (not a multiple of 64), I (not of 128)
    MoEConfig("ragged", T=333, H=200, E=6, k=2, I=136, I_s=72, seed=11),
    MoEConfig("k1", T=257, H=128, E=5, k=1, I=128, I_s=0, seed=12),
    MoEConfig("k_eq_E", T=130, H=64, E=4, k=4, I=64, I_s=64, seed=13),
    MoEConfig("one_token", T=1, H=64, E=8, k=2, I=64, I_s=0, seed=14),
    MoEConfig("wide_n", T=300, H=520, E=3, k=2, I=264, I_s=0, seed=15),            # 3 GEMM2 N tiles, 3 GEMM1 N tiles
    MoEConfig("many_experts", T=512, H=256, E=256, k=8, I=128, I_s=0, bias="normal", seed=16),
    MoEConfig("zipf_skew", T=700, H=256, E=64, k=4, I=256, I_s=128, bias="zipf", seed=17),  # empty experts + a hot one
]


@pytest.mark.parametrize("cfg", SMALL, ids=[c.name for c in SMALL])
@pytest.mark.parametrize("impl", ["tcgen05_fused_gather", "tcgen05_separate_gather", "tcgen05_single_cta", "tcgen05_256_row_tiles",
                                  "tcgen05_tokens_as_n", "simt", "tcgen05_one_launch_ffn", "tcgen05_one_launch_ffn_no_window"])
def test_small_shapes_every_token(cfg, impl):
    m = mok()
    conf = {"simt": m._config(impl=m.MOK_IMPL_SIMT),
            "tcgen05_fused_gather": m._config(gather_mode=1),
            "tcgen05_separate_gather": m._config(gather_mode=2),
            "tcgen05_single_cta": m._config(cta_group=1),
            "tcgen05_256_row_tiles": m._config(cta_group=3),
            "tcgen05_one_launch_ffn": m._config(fused_ffn=2),
            "tcgen05_one_launch_ffn_no_window": m._config(fused_ffn=2, fused_window=-1),
            "tcgen05_tokens_as_n": m._config(impl=m.MOK_IMPL_TCGEN05_TN)}[impl]
    out, st, rep = pu.full_parity(cfg, config=conf)
    print(cfg.name, impl, rep)


EDGE = [
    MoEConfig("min_dims", T=70, H=8, E=4, k=2, I=8, I_s=8, seed=41),                      # smallest legal H, I
    MoEConfig("max_experts", T=300, H=64, E=512, k=6, I=64, I_s=0, bias="normal", seed=42),  # E at the limit, most experts empty
    MoEConfig("k28", T=64, H=128, E=64, k=28, I=64, I_s=0, seed=43),                      # largest k of the tensor-core router
    MoEConfig("k32", T=64, H=128, E=40, k=32, I=64, I_s=0, seed=44),                      # k > 28: fp32-FMA router takes over
    MoEConfig("two_halves_exact", T=256, H=192, E=2, k=2, I=192, I_s=0, seed=45),         # every expert owns exactly 256 rows
    MoEConfig("big_shared", T=513, H=128, E=4, k=1, I=64, I_s=640, seed=46),              # shared expert wider than routed
]


@pytest.mark.parametrize("cfg", EDGE, ids=[c.name for c in EDGE])
@pytest.mark.parametrize("cta_group", [0, 3])
def test_edge_shapes_every_token(cfg, cta_group):
    m = mok()
    out, st, rep = pu.full_parity(cfg, config=m._config(cta_group=cta_group))
    print(cfg.name, cta_group, rep)


def test_all_routes_to_one_expert():
    """Degenerate dispatch: a huge bias sends every token's first route to expert 3; other experts get the rest."""
    cfg = MoEConfig("hot", T=400, H=128, E=8, k=2, I=128, I_s=0, seed=21)
    d = inputs.make_inputs(cfg)
    d["bias"] = np.zeros(cfg.E, np.float32)
    d["bias"][3] = 50.0
    out, st, rep = pu.full_parity(cfg, d=d)
    assert st["counts"].cpu().numpy()[3] == cfg.T


ROUTER_SHAPES = [
    # the one-kernel router pads the experts to 32, 64, 96, 128 and 160; ragged token tiles; k up to its limit of 28
    MoEConfig("r_e6", T=333, H=200, E=6, k=2, I=64, I_s=0, seed=71),
    MoEConfig("r_e40", T=129, H=264, E=40, k=28, I=64, I_s=0, bias="normal", seed=72),
    MoEConfig("r_e64", T=700, H=256, E=64, k=4, I=64, I_s=0, bias="zipf", seed=73),
    MoEConfig("r_e96", T=1000, H=512, E=96, k=6, I=64, I_s=0, seed=74),
    MoEConfig("r_e128", T=2100, H=1024, E=128, k=8, I=64, I_s=0, bias="zipf", seed=75),
    MoEConfig("r_e150", T=515, H=320, E=150, k=5, I=64, I_s=0, bias="normal", seed=76),
    MoEConfig("r_e160", T=260, H=2048, E=160, k=8, I=64, I_s=0, seed=77),
    MoEConfig("r_k_eq_e", T=70, H=64, E=4, k=4, I=64, I_s=0, seed=78),
    MoEConfig("r_e161", T=200, H=192, E=161, k=7, I=64, I_s=0, bias="normal", seed=80),   # first size of the three-kernel path
]


@pytest.mark.parametrize("cfg", ROUTER_SHAPES, ids=[c.name for c in ROUTER_SHAPES])
def test_one_kernel_router_against_oracle_and_three_kernel_router(cfg):
    """Projection + top-k in one kernel (the default up to 160 experts): every token against the oracle, and the
    same bits (indices, weights, output) as the three-kernel tensor-core router; grid-size independent."""
    m = mok()
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    out, st, rep = pu.full_parity(cfg, d=d, g=g)
    print(cfg.name, rep)
    out3, st3 = pu.run_gpu(cfg, g, config=m._config(router_impl=2))
    assert torch.equal(st["topk_idx"], st3["topk_idx"])
    assert torch.equal(st["topk_w"].view(torch.int32), st3["topk_w"].view(torch.int32))
    assert torch.equal(out.view(torch.int16), out3.view(torch.int16))
    outg, stg = pu.run_gpu(cfg, g, config=m._config(grid=3))
    assert torch.equal(st["topk_idx"], stg["topk_idx"])
    assert torch.equal(st["topk_w"].view(torch.int32), stg["topk_w"].view(torch.int32))


@pytest.mark.parametrize("name,router_impl", [("r_e128", 0), ("r_e128", 2), ("r_e161", 0), ("r_e6", 0)])
def test_router_weights_prepared_once_give_the_same_bits(name, router_impl):
    """mok_router_prepare splits W_router once; forward calls that are handed the split skip their own split kernel and
    must produce the same routing and output bits, for the one-kernel and the three-kernel layout of the split."""
    m = mok()
    cfg = next(c for c in ROUTER_SHAPES if c.name == name)
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    conf = m._config(router_impl=router_impl)
    out, st = pu.run_gpu(cfg, g, config=conf)
    split = m.mok_router_prepare(g["W_r"], cfg.k, conf)
    ws = m.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k)
    ws.zero_()                                                   # the workspace's own split region stays empty
    out2, st2 = m.mok_moe_forward_ex(g["x"], g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k,
                                     ws, stages=True, config=conf, router_split=split)
    assert m.mok_read_status(ws) == 0
    assert torch.equal(st["topk_idx"], st2["topk_idx"])
    assert torch.equal(st["topk_w"].view(torch.int32), st2["topk_w"].view(torch.int32))
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))
    # a second call with the same prepared split (the near-tie list must start empty each time)
    out3, st3 = m.mok_moe_forward_ex(g["x"], g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k,
                                     ws, stages=True, config=conf, router_split=split)
    assert torch.equal(st["topk_idx"], st3["topk_idx"]) and torch.equal(out.view(torch.int16), out3.view(torch.int16))
    with pytest.raises(m.MokError) as ei:                        # the fp32-FMA router has no split
        m.mok_router_prepare(g["W_r"], cfg.k, m._config(router_impl=1))
    assert ei.value.status == m.MOK_ERR_UNSUPPORTED


@pytest.mark.parametrize("E,router_impl", [(192, 0), (96, 2)])
def test_router_bits_do_not_depend_on_the_batch_a_token_is_in(E, router_impl):
    """The three-kernel tensor-core router cuts its projection into narrower tiles when there are few tokens (more CTAs
    streaming the router weights).  A token's logits are one accumulation over H whatever the tile shape, so its
    experts and weights must have the same bits alone, in a small batch and inside a large one; and they must be the
    oracle's selection."""
    m = mok()
    cfg = MoEConfig("router_only", T=2560, H=1024, E=E, k=6, I=64, I_s=0, bias="normal", seed=95)
    d = inputs.make_inputs(cfg, experts=False)
    x = m.to_device_bf16(d["x"], "cuda")
    W_r = torch.from_numpy(d["W_r"]).cuda()
    bias = None if d["bias"] is None else torch.from_numpy(d["bias"]).cuda()
    conf = m._config(router_impl=router_impl)
    ws = m.alloc_workspace(cfg.T, cfg.H, 64, 0, cfg.E, cfg.k)
    idx_all, w_all = m.mok_route(x, W_r, bias, cfg.k, ws, config=conf)          # 20 row tiles: full-width tiles
    idx_ref, w_ref, gap, lg = mok_ref.route(d["x"], d["W_r"], d["bias"], cfg.k)
    far = gap > 1e-3
    assert np.array_equal(np.sort(idx_all.cpu().numpy()[far], axis=1), np.sort(idx_ref[far], axis=1))
    for T in (1, 64, 130, 900, 1900, 2048):                                     # 1 .. 16 row tiles: narrower tiles
        idx, w = m.mok_route(x[:T].contiguous(), W_r, bias, cfg.k, ws, config=conf)
        assert torch.equal(idx, idx_all[:T]), T
        assert torch.equal(w.view(torch.int32), w_all[:T].view(torch.int32)), T


def test_one_kernel_router_lists_near_ties_for_the_exact_fix_up():
    """Duplicate expert rows give exact ties and rows that differ in the last bit give logits closer than the tensor
    cores' accumulation error: both must come out as the oracle decides them (lowest id first on exact ties)."""
    m = mok()
    cfg = MoEConfig("r_ties", T=300, H=512, E=32, k=4, I=64, I_s=0, seed=79)
    d = inputs.make_inputs(cfg)
    W = d["W_r"].copy()
    W[5] = W[2]                                   # exact tie between experts 2 and 5 for every token
    W[9] = W[7] * np.float32(1 + 2.0 ** -20)      # near-tie between 7 and 9
    d["W_r"] = W
    g = pu.upload(d)
    out, st, rep = pu.full_parity(cfg, d=d, g=g)
    print(rep)
    idx = st["topk_idx"].cpu().numpy()
    both = (idx == 2).any(axis=1) & (idx == 5).any(axis=1)
    assert both.any()
    for t in np.flatnonzero(both):
        assert list(idx[t]).index(2) < list(idx[t]).index(5)
    out3, st3 = pu.run_gpu(cfg, g, config=m._config(router_impl=2))
    assert torch.equal(st["topk_idx"], st3["topk_idx"])
    assert torch.equal(st["topk_w"].view(torch.int32), st3["topk_w"].view(torch.int32))


def test_tiny_config_every_token_and_determinism():
    cfg = inputs.CONFIGS["tiny"]
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    out, st, rep = pu.full_parity(cfg, d=d, g=g)
    print("tiny", rep)
    m = mok()
    out2 = pu.run_gpu(cfg, g, stages=False)
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))            # run-to-run bitwise identity
    for grid in (1, 2, 7, 148):                                                    # bits do not depend on the grid,
        for cta_group in (1, 2, 3):                                                # nor on the tile / CTA arrangement
            o = pu.run_gpu(cfg, g, config=m._config(grid=grid, cta_group=cta_group), stages=False)
            assert torch.equal(out.view(torch.int16), o.view(torch.int16)), (grid, cta_group)
    o = pu.run_gpu(cfg, g, config=m._config(tile_sched=1), stages=False)                # nor on who computes which tile
    assert torch.equal(out.view(torch.int16), o.view(torch.int16))


@pytest.mark.parametrize("cfg", [SMALL[0], SMALL[5], SMALL[6]], ids=lambda c: c.name)
def test_tiles_stolen_through_cluster_launch_control_give_the_same_bits(cfg):
    """config.tile_sched = 1: one CTA per tile, running CTAs cancel pending ones and compute their tiles.  Every token
    against the oracle, and the same bits as the persistent grid."""
    m = mok()
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    out, st, rep = pu.full_parity(cfg, d=d, g=g, config=m._config(tile_sched=1))
    out0 = pu.run_gpu(cfg, g, stages=False)
    assert torch.equal(out.view(torch.int16), out0.view(torch.int16))


def test_fixed_size_macrobatches_need_only_their_own_workspace_and_give_the_same_bits():
    """config.macrobatch_tokens: the batch passes through a workspace sized for one macrobatch (ragged last one
    included); bits equal the single pass; schedule tables cannot be returned."""
    m = mok()
    cfg = SMALL[6]                                                   # T = 700
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    out = pu.run_gpu(cfg, g, stages=False)
    for mb in (256, 300, 699):
        ws = m.alloc_workspace(mb, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k)           # NOT large enough for T tokens
        full = m.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k).numel()
        assert ws.numel() <= full and (mb > 300 or ws.numel() < full)
        o = m.mok_moe_forward_ex(g["x"], g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k, ws,
                                 config=m._config(macrobatch_tokens=mb))
        torch.cuda.synchronize()
        assert m.mok_read_status(ws) == 0
        assert torch.equal(out.view(torch.int16), o.view(torch.int16)), mb
    ws = m.alloc_workspace(256, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k)
    with pytest.raises(m.MokError):                                   # without the knob the small workspace is refused
        m.mok_moe_forward_ex(g["x"], g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k, ws)
    with pytest.raises(m.MokError):                                   # the tables of one schedule do not exist here
        m.mok_moe_forward_ex(g["x"], g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k, ws,
                             stages=True, config=m._config(macrobatch_tokens=256))


def test_fourteen_argument_entry_point_matches_ex():
    m = mok()
    cfg = inputs.CONFIGS["tiny"]
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    out_ex = pu.run_gpu(cfg, g, stages=False)
    out = m.mok_moe_forward(g["x"], g["W_r"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), out_ex.view(torch.int16))
    # a second, larger problem makes the library-owned workspace grow
    cfg2 = SMALL[-1]
    d2 = inputs.make_inputs(cfg2)
    d2["bias"] = None
    g2 = pu.upload(d2)
    out2 = m.mok_moe_forward(g2["x"], g2["W_r"], g2["W_gate_up"], g2["W_down"], g2["W_sgu"], g2["W_sd"], cfg2.k)
    ref2 = pu.run_gpu(cfg2, g2, stages=False)
    torch.cuda.synchronize()
    assert torch.equal(out2.view(torch.int16), ref2.view(torch.int16))


def test_host_buffer_entry_point():
    m = mok()
    cfg = inputs.CONFIGS["tiny"]
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    ref = pu.run_gpu(cfg, g, stages=False)
    ws = m.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, host_staging=True)
    xh = g["x"].cpu().pin_memory()
    oh = torch.empty_like(xh).pin_memory()
    m.mok_moe_forward_host(xh, oh, g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k, ws)
    assert torch.equal(oh.view(torch.int16), ref.cpu().view(torch.int16))


def test_host_buffer_entry_point_chunked_copies_give_the_same_bits():
    """Token chunks (upload / compute / download overlapped) must not change a single bit of the result."""
    m = mok()
    cfg = MoEConfig("chunky", T=1500, H=256, E=16, k=4, I=256, I_s=128, bias="normal", seed=31)
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    ref = pu.run_gpu(cfg, g, stages=False).cpu()
    ws = m.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, host_staging=True)
    xh = g["x"].cpu().pin_memory()
    for chunks in (1, 2, 5):
        oh = torch.zeros_like(xh).pin_memory()
        m.mok_moe_forward_host(xh, oh, g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k,
                               ws, config=m._config(host_chunks=chunks))
        assert torch.equal(oh.view(torch.int16), ref.view(torch.int16)), chunks


def test_asynchronous_host_submissions_overlap_and_match_the_device_call():
    """A stream of batches through mok_moe_forward_host_async: different inputs in flight together (the two staging
    slots alternate), results after mok_host_wait bitwise equal to mok_moe_forward_ex on the same inputs."""
    m = mok()
    cfg = SMALL[-1]
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    ws = m.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, host_staging=2)
    xs = [g["x"], (g["x"].float() * 0.5).to(torch.bfloat16), (g["x"].float() * -1.25).to(torch.bfloat16)]
    want = []
    for x in xs:
        want.append(m.mok_moe_forward_ex(x, g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"],
                                         cfg.k, ws).clone())
    torch.cuda.synchronize()
    xh = [x.cpu().pin_memory() for x in xs]
    n_sub = 7
    oh = [torch.zeros_like(xh[0]).pin_memory() for _ in range(n_sub)]
    for i in range(n_sub):
        m.mok_moe_forward_host_async(xh[i % 3], oh[i], g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], g["W_sgu"],
                                     g["W_sd"], cfg.k, ws)
    m.mok_host_wait()
    assert m.mok_read_status(ws) == 0
    for i in range(n_sub):
        assert torch.equal(oh[i].view(torch.int16), want[i % 3].cpu().view(torch.int16)), i
    # the blocking call still works on the same workspace afterwards, and a workspace without the second slot is refused
    out1 = torch.zeros_like(xh[0]).pin_memory()
    m.mok_moe_forward_host(xh[1], out1, g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k, ws)
    assert torch.equal(out1.view(torch.int16), want[1].cpu().view(torch.int16))
    small = m.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, host_staging=True)
    small = small[:small.numel() - 256]
    with pytest.raises(m.MokError):
        m.mok_moe_forward_host_async(xh[0], oh[0], g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"],
                                     cfg.k, small)
    m.mok_host_wait()


def test_stage_entry_points():
    m = mok()
    cfg = SMALL[-1]
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    ws = m.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k)
    idx, w = m.mok_route(g["x"], g["W_r"], g["bias"], cfg.k, ws)
    counts, offsets, perm, inv = m.mok_schedule(idx, cfg.E, ws)
    st = {"topk_idx": idx, "topk_w": w, "counts": counts, "offsets": offsets, "perm": perm, "inv_perm": inv}
    assert m.mok_read_status(ws) == 0
    pu.check_routing_and_schedule(cfg, d, st)


def test_argument_errors_launch_nothing():
    m = mok()
    cfg = inputs.CONFIGS["tiny"]
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    ws = m.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k)
    args = (g["x"], g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"])
    with pytest.raises(m.MokError) as e:
        m.mok_moe_forward_ex(*args, cfg.E + 1, ws)                                  # k > E
    assert e.value.status == m.MOK_ERR_SHAPE
    with pytest.raises(m.MokError) as e:
        m.mok_moe_forward_ex(*args, cfg.k, torch.empty(1024, dtype=torch.uint8, device="cuda"))
    assert e.value.status == m.MOK_ERR_WORKSPACE
    with pytest.raises(m.MokError) as e:                                             # shared weights without both halves
        m.mok_moe_forward_ex(g["x"], g["W_r"], None, g["W_gate_up"], g["W_down"], g["W_sgu"], None, cfg.k, ws)
    assert e.value.status == m.MOK_ERR_SHAPE
    with pytest.raises(m.MokError) as e:                                             # misaligned activation pointer
        xm = torch.empty(cfg.T * cfg.H + 8, dtype=torch.bfloat16, device="cuda")[1:1 + cfg.T * cfg.H].view(cfg.T, cfg.H)
        m.mok_moe_forward_ex(xm, *args[1:], cfg.k, ws)
    assert e.value.status == m.MOK_ERR_ALIGN
    # T == 0 is a no-op
    x0 = torch.empty((0, cfg.H), dtype=torch.bfloat16, device="cuda")
    out0 = m.mok_moe_forward_ex(x0, *args[1:], cfg.k, ws)
    assert out0.shape == (0, cfg.H)


MID = [
    # several row groups per expert, ragged last tiles, a narrow last gate/up tile (I mod 128 = 64), an empty expert
    MoEConfig("mid_groups", T=3000, H=512, E=6, k=3, I=320, I_s=0, bias="zipf", seed=91),
    MoEConfig("mid_many", T=2048, H=576, E=40, k=4, I=256, I_s=128, bias="normal", seed=92),
]


@pytest.mark.parametrize("cfg", MID, ids=[c.name for c in MID])
def test_one_launch_ffn_gives_the_bits_of_two_launches(cfg):
    """Gate/up + SwiGLU + down in ONE persistent launch (down tiles wait on completion counters of the gate/up tiles):
    every token against the oracle, and bit for bit the output of the two-launch path -- whatever the grid size and
    the distance between a row group's gate/up tiles and its down tiles (none: every down tile has to wait; huge:
    all down tiles at the end of the list)."""
    m = mok()
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    out2, st, rep = pu.full_parity(cfg, d=d, g=g, config=m._config(fused_ffn=1, cta_group=3))
    print(cfg.name, rep)
    for kw in ({}, {"fused_window": -1}, {"fused_window": 1}, {"fused_window": 1 << 20}, {"grid": 1}, {"grid": 7},
               {"grid": 37, "fused_window": -1}, {"tile_sched": 2}, {"tile_sched": 2, "fused_window": -1},
               {"tile_sched": 2, "grid": 5, "fused_window": 40},
               # static stride with synchronised tile starts (what large expert matrices get by default)
               {"gang_sync": 2}, {"gang_sync": 2, "fused_window": -1}, {"gang_sync": 2, "grid": 8},
               {"gang_sync": 2, "grid": 11, "fused_window": 40}, {"gang_sync": 2, "grid": 3},
               {"gang_sync": 2, "tile_sched": 1},
               # the combine at the end of the same launch (the shared expert then runs first)
               {"fused_ffn": 3}, {"fused_ffn": 3, "grid": 1}, {"fused_ffn": 3, "fused_window": -1, "grid": 37},
               {"fused_ffn": 3, "tile_sched": 2, "grid": 5}, {"fused_ffn": 3, "gang_sync": 2},
               {"fused_ffn": 3, "gang_sync": 2, "grid": 11, "fused_window": 40},
               # communication CTAs: some CTAs of the grid stage the token rows, the others load them by TMA
               {"comm_ctas": 4}, {"comm_ctas": 16, "tile_sched": 2, "gang_sync": 2}, {"comm_ctas": 1, "grid": 9},
               {"comm_ctas": 8, "fused_window": -1}, {"comm_ctas": 4, "fused_ffn": 3}, {"comm_ctas": 200},
               {"comm_ctas": 3, "tile_sched": 1, "grid": 5}):
        out1 = pu.run_gpu(cfg, g, config=m._config(**(dict(fused_ffn=2) | kw)), stages=False)
        assert torch.equal(out1.view(torch.int16), out2.view(torch.int16)), kw
    # ... and against the oracle with the stage outputs requested, and under the per-stage profiler (the stages then run
    # in another order than their numbers: every stage time must still be a non-negative interval)
    out3, st3, rep3 = pu.full_parity(cfg, d=d, g=g, config=m._config(fused_ffn=3))
    assert torch.equal(out3.view(torch.int16), out2.view(torch.int16))
    m.mok_profile_begin(2)
    for _ in range(2):
        pu.run_gpu(cfg, g, config=m._config(fused_ffn=3, profile=1), stages=False)
    ms = m.mok_profile_end(2)
    assert len(ms) == 2 and all(v >= 0.0 for call in ms for v in call.values()), ms
    assert all(call["combine"] < 0.05 and call["gemm1"] > 0.0 for call in ms), ms


RING = MID + [
    # about 270 row tiles of 256 rows: a ring of 24 slots is rewritten eleven times
    MoEConfig("ring_long", T=16384, H=512, E=16, k=4, I=256, I_s=0, bias="zipf", seed=93),
]


@pytest.mark.parametrize("cfg", RING, ids=[c.name for c in RING])
def test_gated_activation_in_a_ring_gives_the_same_bits(cfg):
    """config.h_ring_tiles: the gated activation lives in a ring of 256-row slots that the row tiles in flight reuse
    (Section 3.3), in a workspace without the rows beyond the ring.  A gate/up tile stores into its slot only after
    the slot's previous rows were loaded by all their down tiles.  Every token against the oracle, and bit for bit
    the two-launch path, for the smallest ring and larger ones, both hand-outs, several grids and windows, and with
    the combine in the same launch."""
    m = mok()
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    ref = pu.run_gpu(cfg, g, config=m._config(fused_ffn=1, cta_group=3), stages=False)
    full = m.mok_workspace_bytes(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k)
    ring = m.MOK_H_RING_MIN_TILES
    assert 0 < m.mok_workspace_bytes_ring(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, ring) < full
    assert m.mok_workspace_bytes_ring(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, ring - 1) == 0
    ws = m.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, h_ring_tiles=ring)
    out, st, rep = pu.full_parity(cfg, d=d, g=g, config=m._config(h_ring_tiles=ring), ws=ws)
    print(cfg.name, rep)
    assert torch.equal(out.view(torch.int16), ref.view(torch.int16))
    for kw in ({"grid": 1}, {"grid": 7}, {"fused_window": -1}, {"fused_window": 1 << 20}, {"tile_sched": 1},
               {"tile_sched": 2, "grid": 5}, {"gang_sync": 2}, {"gang_sync": 2, "grid": 11}, {"fused_ffn": 3},
               {"fused_ffn": 3, "tile_sched": 2, "gang_sync": 2}):
        out1 = pu.run_gpu(cfg, g, ws=ws, config=m._config(h_ring_tiles=ring, **kw), stages=False)
        assert torch.equal(out1.view(torch.int16), ref.view(torch.int16)), kw
    for r in (32, 100, 1 << 20):      # (a ring with more slots than row tiles is the plain layout)
        wr = m.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, h_ring_tiles=r)
        out1 = pu.run_gpu(cfg, g, ws=wr, config=m._config(h_ring_tiles=r), stages=False)
        assert torch.equal(out1.view(torch.int16), ref.view(torch.int16)), r
    # what cannot run with a ring says so: the two-launch kernels on request, a ring below the minimum
    args = (g["x"], g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k, ws)
    with pytest.raises(m.MokError) as e:
        m.mok_moe_forward_ex(*args, config=m._config(h_ring_tiles=ring, cta_group=1))
    assert e.value.status == m.MOK_ERR_UNSUPPORTED
    with pytest.raises(m.MokError) as e:
        m.mok_moe_forward_ex(*args, config=m._config(h_ring_tiles=ring - 1))
    assert e.value.status == m.MOK_ERR_SHAPE


@pytest.mark.parametrize("cfg", MID + [SMALL[0], SMALL[6]], ids=[c.name for c in MID + [SMALL[0], SMALL[6]]])
def test_synchronised_tile_starts_give_the_same_bits(cfg):
    """The 256-row kernel can make the row tiles that share a weight tile start together (config.gang_sync; chosen
    automatically for large expert matrices).  Forced on here: every token against the oracle, the same bits as without
    it, for the smallest grid that allows it, a ragged one and the full one; a grid below eight CTAs falls back to
    unsynchronised starts instead of deadlocking."""
    m = mok()
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    out0, st, rep = pu.full_parity(cfg, d=d, g=g, config=m._config(cta_group=3, gang_sync=2))
    print(cfg.name, rep)
    ref = pu.run_gpu(cfg, g, config=m._config(cta_group=3, gang_sync=1), stages=False)
    assert torch.equal(out0.view(torch.int16), ref.view(torch.int16))
    for grid in (3, 8, 11, 148):
        out = pu.run_gpu(cfg, g, config=m._config(cta_group=3, gang_sync=2, grid=grid), stages=False)
        assert torch.equal(out.view(torch.int16), ref.view(torch.int16)), grid


@pytest.mark.parametrize("fused,sched,gang,ring", [(1, 0, 0, 0), (2, 0, 0, 0), (2, 2, 0, 0), (2, 0, 2, 0), (1, 0, 2, 0),
                                                  (3, 0, 0, 0), (3, 2, 0, 0), (2, 0, 0, 24), (2, 2, 0, 24)])
def test_bounded_waits_report_a_timeout_and_leave_the_context_usable(fused, sched, gang, ring):
    """Failure detection without a fault: the test hook silences the gate/up GEMM's TMA producer, so its MMA issuer
    waits for operands that never come.  Every wait is bounded (2 ms here), the kernel records MOK_ERR_TIMEOUT, frees
    its tensor memory and returns; the next call on the same context must be correct again.  fused = 2: the same on
    the one-launch expert FFN, where the down tiles' producers additionally wait for gate/up tiles that never finish."""
    m = mok()
    cfg = inputs.CONFIGS["tiny"]
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    ws = m.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k)
    good = pu.run_gpu(cfg, g, ws=ws, stages=False).clone()
    m.mok_moe_forward_ex(g["x"], g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k, ws,
                         config=m._config(debug=m.MOK_DEBUG_STARVE, fused_ffn=fused, tile_sched=sched, gang_sync=gang,
                                          cta_group=3 if fused == 1 else 0, h_ring_tiles=ring))
    assert m.mok_read_status(ws) == m.MOK_ERR_TIMEOUT
    again = pu.run_gpu(cfg, g, ws=ws, stages=False)
    assert torch.equal(good.view(torch.int16), again.view(torch.int16))


@pytest.mark.parametrize("kw", [{"h_ring_tiles": 24}, {"h_ring_tiles": 24, "tile_sched": 1}, {"fused_ffn": 3},
                                {"fused_ffn": 3, "tile_sched": 2}, {"comm_ctas": 2}, {"comm_ctas": 2, "tile_sched": 2}],
                         ids=["ring", "ring_dynamic", "combine", "combine_static", "comm", "comm_static"])
def test_completion_counter_waits_of_the_one_launch_kernel_run_out_cleanly(kw):
    """The waits on the one-launch kernel's own completion counters -- a ring slot's previous rows consumed, all
    epilogue warps done before the in-launch combine, a staging slot released for the communication CTAs -- are bounded too: with the test hook that suppresses every
    arrival on those counters (and a 2 ms limit) the call ends with MOK_ERR_TIMEOUT, nothing faults, and the next call
    on the same context and workspace gives the normal bits."""
    m = mok()
    cfg = MID[0]                                     # about 40 row tiles: a ring of 24 slots wraps
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    ws = m.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k)
    good = pu.run_gpu(cfg, g, ws=ws, config=m._config(**kw), stages=False).clone()
    m.mok_moe_forward_ex(g["x"], g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k, ws,
                         config=m._config(debug=m.MOK_DEBUG_NO_ARRIVALS, **kw))
    assert m.mok_read_status(ws) == m.MOK_ERR_TIMEOUT
    again = pu.run_gpu(cfg, g, ws=ws, config=m._config(**kw), stages=False)
    assert torch.equal(good.view(torch.int16), again.view(torch.int16))


@pytest.mark.parametrize("cfg", [inputs.CONFIGS["tiny"], MID[1]], ids=["tiny", "mid_many"])
def test_shared_expert_beside_the_routed_experts_gives_the_same_bits(cfg):
    """config.shared_overlap: the shared expert's GEMMs on a library-owned second stream, forked from and joined to the
    caller's stream by events (the default for small layers), against the same GEMMs in line: every token against the
    oracle, the same bits with either order, with the one-launch expert FFN, small grids, and several calls in a row on
    one workspace (the fork of a call waits for the previous call's combine)."""
    m = mok()
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    inline, st, rep = pu.full_parity(cfg, d=d, g=g, config=m._config(shared_overlap=1))
    print(cfg.name, rep)
    ws = m.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k)
    for kw in ({}, {"shared_overlap": 2}, {"shared_overlap": 2, "fused_ffn": 2}, {"shared_overlap": 2, "grid": 3},
               {"shared_overlap": 2, "cta_group": 1}, {"shared_overlap": 2, "cta_group": 3, "gang_sync": 2}):
        for _ in range(3):
            out = pu.run_gpu(cfg, g, ws=ws, config=m._config(**kw), stages=False)
            assert torch.equal(out.view(torch.int16), inline.view(torch.int16)), kw


GRAPH_CASES = [
    ("tiny", {}),                                                     # two streams: the shared expert beside the routed ones
    ("mid_many", {"fused_ffn": 2}),                                   # the one-launch kernel, dynamic draw
    ("mid_many", {"fused_ffn": 2, "tile_sched": 2, "gang_sync": 2}),  # ... as a cooperative launch
    ("mid_many", {"comm_ctas": 4}),
    ("mid_many", {"fused_ffn": 3}),
    ("mid_many", {"h_ring_tiles": 24}),
]


@pytest.mark.parametrize("name,kw", GRAPH_CASES, ids=[f"{n}-{'-'.join(k) or 'default'}" for n, k in GRAPH_CASES])
def test_forward_can_be_captured_in_a_cuda_graph_and_replayed(name, kw):
    """The layer makes no host synchronisation and no allocation after its first call for a shape, so a whole
    forward can be recorded once into a CUDA graph and replayed (launch-bound small batches): same bits.  That holds
    for the call with a second stream inside, for the cooperative launches and for the one-launch kernel's options."""
    m = mok()
    cfg = inputs.CONFIGS["tiny"] if name == "tiny" else MID[1]
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    ws = m.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k)
    out = torch.empty_like(g["x"])
    conf = m._config(**kw)
    args = (g["x"], g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k, ws)
    m.mok_moe_forward_ex(*args, out=out, config=conf)          # first call: one-time kernel attribute set-up
    torch.cuda.synchronize()
    want = out.clone()
    graph = torch.cuda.CUDAGraph()
    out.zero_()
    with torch.cuda.graph(graph):
        m.mok_moe_forward_ex(*args, out=out, config=conf)
    for _ in range(3):
        out.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int16), want.view(torch.int16))
    assert m.mok_read_status(ws) == 0
