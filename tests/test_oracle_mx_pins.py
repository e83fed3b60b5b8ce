"""Pins of the MXFP8 part of the CPU oracle (oracle/mok_ref_mx.c; Section 3.4 "MXFP8 Support" and the microscaling
format it cites): the E4M3 grid and its rounding against the closed form and against PyTorch's float8_e4m3fn
conversion, the shared-scale rule, round-trip properties, and the MXFP8 layer against an independent vectorised
evaluation and against exact special cases.  CPU only."""
import numpy as np
import pytest
import torch

from oracle import mok_ref
from paper_2609_36070_b200 import inputs

ALL = np.arange(256, dtype=np.uint8)
FINITE = ALL[(ALL & 0x7F) != 0x7F]


def closed_form(c):
    s, e, m = c >> 7, (c >> 3) & 15, c & 7
    v = (m / 8.0) * 2.0 ** -6 if e == 0 else (1 + m / 8.0) * 2.0 ** (e - 7)
    return -v if s else v


def test_e4m3_grid_is_the_closed_form_and_round_trips():
    dec = mok_ref.e4m3_decode(ALL)
    assert np.isnan(dec[0x7F]) and np.isnan(dec[0xFF])
    for c in FINITE:
        assert dec[c] == closed_form(int(c))
    assert dec[0x7E] == 448.0 and dec[0x01] == 2.0 ** -9 and dec[0x08] == 2.0 ** -6
    assert np.array_equal(mok_ref.e4m3_encode(dec[FINITE]), FINITE)          # includes -0 -> 0x80


def test_e4m3_rounding_matches_the_library_conversion():
    rng = np.random.default_rng(3)
    v = np.concatenate([rng.uniform(-448, 448, 4000), rng.normal(0, 1, 4000), rng.normal(0, 0.01, 4000),
                        rng.uniform(-2.0 ** -6, 2.0 ** -6, 2000)]).astype(np.float32)
    want = torch.from_numpy(v).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = mok_ref.e4m3_encode(v.astype(np.float64))
    assert np.array_equal(got, want)


def test_e4m3_ties_go_to_the_even_code_and_large_values_clamp():
    pos = np.arange(0, 0x7E, dtype=np.uint8)                                   # consecutive positive codes c, c+1
    lo, hi = mok_ref.e4m3_decode(pos), mok_ref.e4m3_decode(pos + 1)
    mid = (lo + hi) / 2
    got = mok_ref.e4m3_encode(mid)
    assert np.array_equal(got, np.where(pos % 2 == 0, pos, pos + 1))
    assert np.array_equal(mok_ref.e4m3_encode(-mid), np.where(pos % 2 == 0, pos, pos + 1) | 0x80)
    assert np.array_equal(mok_ref.e4m3_encode(np.nextafter(mid, np.inf)), pos + 1)
    assert np.array_equal(mok_ref.e4m3_encode(np.nextafter(mid, -np.inf)), pos)
    assert np.array_equal(mok_ref.e4m3_encode([448.0, 449.0, 464.0, 480.0, 1e30, -1e30]),
                          [0x7E, 0x7E, 0x7E, 0x7E, 0x7E, 0xFE])


def test_shared_scale_rule():
    rng = np.random.default_rng(5)
    for n in (-20, -3, 0, 1, 9, 30):
        blk = rng.uniform(-1, 1, (1, 32)) * 2.0 ** n * 0.99
        blk[0, 7] = 2.0 ** n                                                   # amax exactly a power of two
        _, sc = mok_ref.mx_quantize(blk)
        assert sc[0, 0] == n - 8 + 127
        blk[0, 7] = -np.nextafter(2.0 ** (n + 1), 0)                           # just below the next power of two
        codes, sc = mok_ref.mx_quantize(blk)
        assert sc[0, 0] == n - 8 + 127
        assert codes[0, 7] == 0xFE                                             # (448, 512) * X clamps to 448
    v = rng.normal(0, 3, (64, 96))
    codes, sc = mok_ref.mx_quantize(v)
    amax = np.abs(v.reshape(64, 3, 32)).max(axis=2)
    ratio = amax / 2.0 ** (sc.astype(np.int64) - 127)
    assert ((ratio >= 256) & (ratio < 512)).all()
    z = np.zeros((2, 32))
    codes, sc = mok_ref.mx_quantize(z)
    assert (sc == 0).all() and (codes == 0).all()


def test_quantise_dequantise_properties():
    rng = np.random.default_rng(7)
    # values already on an MXFP8 grid come back exactly
    scale = rng.integers(100, 150, (40, 4))
    codes = rng.choice(mok_ref.e4m3_encode(rng.uniform(-255, 255, 500)), (40, 128))
    codes[:, ::32] = 0x78                                                      # 256 in every block: fixes the scale
    grid = mok_ref.mx_dequantize(codes.astype(np.uint8), scale.astype(np.uint8))
    c2, s2 = mok_ref.mx_quantize(grid)
    assert np.array_equal(s2, scale) and np.array_equal(mok_ref.mx_dequantize(c2, s2), grid)
    # error bound: half a grid step of the element's own binade (elements above 448 X clamp)
    v = rng.normal(0, 1, (50, 64)) * 10.0 ** rng.uniform(-3, 3, (50, 1))
    c, s = mok_ref.mx_quantize(v)
    dq = mok_ref.mx_dequantize(c, s)
    X = np.repeat(2.0 ** (s.astype(np.int64) - 127), 32, axis=1)
    a = np.abs(v) / X
    step = np.where(a < 2.0 ** -6, 2.0 ** -9, 2.0 ** (np.floor(np.log2(np.maximum(a, 1e-300))) - 3))
    ok = a <= 448
    assert (np.abs(v - dq)[ok] <= (step * X / 2)[ok] * (1 + 1e-12)).all()
    assert (np.abs(dq[~ok]) == (448 * X)[~ok]).all()
    assert (np.sign(dq) * np.sign(v) >= 0).all()
    # a power-of-two factor commutes with the quantiser
    c4, s4 = mok_ref.mx_quantize(v * 16.0)
    assert np.array_equal(c4, c) and np.array_equal(s4.astype(int), s.astype(int) + 4)
    # bf16 inputs: the fp32 round trip equals quantise + dequantise of the widened values
    bits = inputs.f32_to_bf16_bits(rng.normal(0, 0.02, (8, 64)).astype(np.float32))
    wide = inputs.bf16_bits_to_f32(bits).astype(np.float64)
    assert np.array_equal(mok_ref.mx_roundtrip_bf16(bits).astype(np.float64), mok_ref.mx_dequantize(*mok_ref.mx_quantize(wide)))


def library_quantise(v):
    """An independent route to the same definition: power-of-two scale from frexp, elements through PyTorch's
    float8_e4m3fn conversion after clamping to +-448."""
    v = np.asarray(v, np.float64)
    blk = v.reshape(v.shape[0], -1, 32)
    amax = np.abs(blk).max(axis=2, keepdims=True)
    _, ex = np.frexp(amax)
    X = np.where(amax > 0, 2.0 ** (ex - 1 - 8), 2.0 ** -127)
    q = np.clip(blk / X, -448, 448)
    dq = torch.from_numpy(q).to(torch.float32).to(torch.float8_e4m3fn).to(torch.float64).numpy() * X
    return dq.reshape(v.shape)


def test_mx_layer_against_an_independent_vectorised_evaluation():
    cfg = inputs.MoEConfig("mx_pin", 24, 64, 4, 2, 96, 32, seed=21)
    d = inputs.make_inputs(cfg)
    idx, w, _, _ = mok_ref.route(d["x"], d["W_r"], d["bias"], cfg.k)
    Wgu_q, Wd_q = mok_ref.mx_roundtrip_bf16(d["W_gate_up"]), mok_ref.mx_roundtrip_bf16(d["W_down"])
    got = mok_ref.ffn_tokens_mx(d["x"], Wgu_q, Wd_q, d["W_sgu"], d["W_sd"], idx, w, np.arange(cfg.T))
    f = lambda b: inputs.bf16_bits_to_f32(b).astype(np.float64)
    x = f(d["x"])
    xq = library_quantise(x)
    Wgu = library_quantise(f(d["W_gate_up"]).reshape(-1, cfg.H)).reshape(cfg.E, 2 * cfg.I, cfg.H)
    Wd = library_quantise(f(d["W_down"]).reshape(-1, cfg.I)).reshape(cfg.E, cfg.H, cfg.I)
    silu = lambda z: z / (1 + np.exp(-z))
    gs = f(d["W_sgu"]) @ x.T                                                   # shared expert: bf16 operands
    want = (f(d["W_sd"]) @ (silu(gs[:cfg.I_s]) * gs[cfg.I_s:])).T
    for t in range(cfg.T):
        for s in range(cfg.k):
            e = idx[t, s]
            gu = Wgu[e] @ xq[t]
            h = library_quantise((silu(gu[:cfg.I]) * gu[cfg.I:])[None, :])[0]
            want[t] += w[t, s] * (Wd[e] @ h)
    assert np.abs(got - want).max() <= 1e-12 * np.abs(want).max()


def test_mx_layer_special_cases():
    cfg = inputs.MoEConfig("mx_pin2", 16, 64, 4, 2, 64, 32, seed=22)
    d = inputs.make_inputs(cfg)
    idx, w, _, _ = mok_ref.route(d["x"], d["W_r"], d["bias"], cfg.k)
    Wgu_q, Wd_q = mok_ref.mx_roundtrip_bf16(d["W_gate_up"]), mok_ref.mx_roundtrip_bf16(d["W_down"])
    tok = np.arange(cfg.T)
    base = mok_ref.ffn_tokens_mx(d["x"], Wgu_q, Wd_q, d["W_sgu"], d["W_sd"], idx, w, tok)
    # routed W_down = 0: only the (bf16) shared expert is left, which is the plain oracle's shared term
    shared = mok_ref.ffn_tokens_mx(d["x"], Wgu_q, np.zeros_like(Wd_q), d["W_sgu"], d["W_sd"], idx, w, tok)
    zero_down = np.zeros_like(d["W_down"])
    want = mok_ref.ffn_tokens(d["x"], d["W_gate_up"], zero_down, d["W_sgu"], d["W_sd"], idx, w, tok)
    assert np.abs(shared - want).max() <= 1e-13 * np.abs(want).max()
    # W_down scaled by a power of two: the routed part scales by exactly that factor
    scaled = mok_ref.ffn_tokens_mx(d["x"], Wgu_q, Wd_q * 8.0, d["W_sgu"], d["W_sd"], idx, w, tok)
    assert np.abs((scaled - shared) - 8.0 * (base - shared)).max() <= 1e-12 * np.abs(base).max()
    # the quantised layer stays close to the unquantised one (a few per cent), and is not identical to it
    plain = mok_ref.ffn_tokens(d["x"], d["W_gate_up"], d["W_down"], d["W_sgu"], d["W_sd"], idx, w, tok)
    rel = np.abs(base - plain).mean() / np.abs(plain).mean()
    assert 1e-4 < rel < 0.1, rel
