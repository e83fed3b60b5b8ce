"""MXFP8 mode of the routed experts on the GPU against the CPU oracle: the quantisation kernels bit for bit (codes and
scales are decided exactly on both sides), and the whole layer against the oracle's fp64 evaluation of the same
quantised definition within the layer's tolerances (the gated activation is quantised from fp32 sums on the device
and from fp64 sums in the oracle, so its codes may differ where a value sits on a rounding boundary)."""
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


def atoms_from_row_major(scales, rows_per_group):
    """Oracle scales [groups*rows, K/32] -> the 512-byte atom layout, padded with 127."""
    total, nblk = scales.shape
    groups = total // rows_per_group
    NB, KG = (rows_per_group + 127) // 128, (nblk + 3) // 4
    out = np.full((groups, NB, KG, 512), 127, np.uint8)
    s = scales.reshape(groups, rows_per_group, nblk)
    for r in range(rows_per_group):
        for kb in range(nblk):
            out[:, r // 128, kb // 4, (r % 32) * 16 + ((r % 128) // 32) * 4 + kb % 4] = s[:, r, kb]
    return out.reshape(-1)


@pytest.mark.parametrize("groups,rows,K", [(1, 128, 128), (3, 200, 96), (4, 64, 288), (2, 300, 2880)])
def test_weight_quantiser_matches_oracle(groups, rows, K):
    m = mok()
    rng = np.random.default_rng(groups * 1000 + rows)
    w = (rng.normal(0, 0.02, (groups, rows, K)) * 10.0 ** rng.uniform(-2, 2, (groups, rows, 1))).astype(np.float32)
    w[0, 0, :32] = 0.0                                                       # an all-zero block
    w[0, 1, 5] = 3.0e38                                                      # a huge value
    bits = inputs.f32_to_bf16_bits(w)
    wide = inputs.bf16_bits_to_f32(bits).astype(np.float64)
    codes_ref, scales_ref = mok_ref.mx_quantize(wide.reshape(-1, K))
    codes, scales = m.mok_mx_quantize_weights(m.to_device_bf16(bits))
    assert np.array_equal(codes.cpu().numpy().reshape(-1, K), codes_ref)
    assert np.array_equal(scales.cpu().numpy(), atoms_from_row_major(scales_ref, rows))


@pytest.mark.parametrize("rows,K", [(1, 32), (77, 256), (300, 2880), (1024, 2048)])
def test_row_quantiser_matches_oracle(rows, K):
    m = mok()
    rng = np.random.default_rng(rows + K)
    x = rng.normal(0, 1, (rows, K)).astype(np.float32)
    x[rows // 2] = 0.0
    bits = inputs.f32_to_bf16_bits(x)
    codes_ref, scales_ref = mok_ref.mx_quantize(inputs.bf16_bits_to_f32(bits).astype(np.float64))
    codes, scales = m.mok_mx_quantize_rows(m.to_device_bf16(bits))
    assert np.array_equal(codes.cpu().numpy(), codes_ref)
    got = scales.cpu().numpy()
    assert np.array_equal(got[:, :K // 32], scales_ref)
    assert (got[:, K // 32:] == 127).all()


def mx_case(cfg, config_kw=None):
    return pu.mx_parity(cfg, config_kw=config_kw)


MX_SHAPES = [
    # name, T, H, E, k, I, I_s, bias
    ("tiny", 256, 256, 8, 2, 512, 512, "none"),
    ("one_tile", 64, 128, 2, 1, 128, 0, "none"),
    ("ragged_k_and_n", 300, 288, 4, 2, 160, 0, "normal"),          # K tails of 32 and 64 elements, N tails
    ("skewed", 1024, 512, 32, 4, 384, 0, "zipf"),
    ("gpt_oss_like_dims", 512, 2880 // 5, 8, 2, 2880 // 5, 0, "none"),   # 576: multiple of 32, not of 128
    ("minimal", 1, 32, 1, 1, 32, 0, "none"),
]


@pytest.mark.parametrize("cta_group", [1, 2], ids=["single_cta", "cta_pairs"])
@pytest.mark.parametrize("name,T,H,E,k,I,I_s,bias", MX_SHAPES)
def test_mx_layer_parity(name, T, H, E, k, I, I_s, bias, cta_group):
    cfg = inputs.MoEConfig("mx_" + name, T, H, E, k, I, I_s, bias=bias, seed=31)
    out, rep = mx_case(cfg, {"cta_group": cta_group})
    print(name, cta_group, rep)


def test_mx_layer_is_reproducible_and_grid_independent():
    cfg = inputs.MoEConfig("mx_repro", 768, 256, 16, 4, 256, 0, bias="zipf", seed=32)
    runs = [mx_case(cfg, kw)[0].view(torch.int16).clone()
            for kw in (None, None, {"grid": 1}, {"grid": 7}, {"cta_group": 2}, {"cta_group": 2, "grid": 6})]
    for r in runs[1:]:
        assert torch.equal(r, runs[0])


def test_mx_argument_errors():
    m = mok()
    cfg = inputs.CONFIGS["tiny"]
    d = inputs.make_inputs(cfg)
    g = pu.upload(d)
    ws = m.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, mx=True)
    conf = m._config(precision=m.MOK_PRECISION_MXFP8)
    with pytest.raises(m.MokError) as ei:                                    # pre-quantised weights missing
        m.mok_moe_forward_ex(g["x"], g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k, ws,
                             config=conf)
    assert ei.value.status == m.MOK_ERR_NULL
    small = m.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k)    # bf16-sized workspace
    mxw = m.MxWeights(g["W_gate_up"], g["W_down"])
    with pytest.raises(m.MokError) as ei:
        m.mok_moe_forward_ex(g["x"], g["W_r"], g["bias"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k,
                             small, config=conf, mx_weights=mxw)
    assert ei.value.status == m.MOK_ERR_WORKSPACE
    assert m.mok_mx_workspace_bytes(64, 72, 64, 0, 4, 2) == 0                # H not a multiple of 32
    assert m._lib.mok_mx_scale_bytes(1, 128, 100) == 0
