"""Pins of the backward-pass oracle (oracle/mok_ref_bwd.c): its analytic gradients against central finite differences
of an independent fp64 forward (numpy matmuls written from the Section 2.1 definition), against the forward oracle
where the two meet (dw = <dout, f_e(x)>), and exact special cases.  CPU only."""
import numpy as np

from oracle import mok_ref
from paper_2609_36070_b200 import inputs

f64 = lambda bits: inputs.bf16_bits_to_f32(bits).astype(np.float64)


def forward_np(x, Wgu, Wd, Wsgu, Wsd, idx, w):
    """The layer on real-valued fp64 arrays (no bf16 anywhere): library matmuls, per token."""
    silu = lambda z: z / (1 + np.exp(-z))
    T, H = x.shape
    I = Wgu.shape[1] // 2
    out = np.zeros((T, H))
    for t in range(T):
        if Wsgu is not None:
            gu = Wsgu @ x[t]
            Is = Wsgu.shape[0] // 2
            out[t] += Wsd @ (silu(gu[:Is]) * gu[Is:])
        for s in range(idx.shape[1]):
            e = idx[t, s]
            gu = Wgu[e] @ x[t]
            out[t] += w[t, s] * (Wd[e] @ (silu(gu[:I]) * gu[I:]))
    return out


def case(seed, T=5, H=8, E=3, k=2, I=16, I_s=8):
    cfg = inputs.MoEConfig("bwd_pin", T, H, E, k, I, I_s, seed=seed)
    d = inputs.make_inputs(cfg)
    # larger weights than the workloads': the derivative of silu must matter for the pin to bite
    rng = np.random.default_rng(seed)
    for name in ("W_gate_up", "W_down", "W_sgu", "W_sd"):
        if d[name] is not None:
            d[name] = inputs.f32_to_bf16_bits(rng.normal(0, 0.5, d[name].shape).astype(np.float32))
    idx, w, _, _ = mok_ref.route(d["x"], d["W_r"], d["bias"], k)
    dout = rng.normal(0, 1, (T, H))
    return cfg, d, idx, w, dout


def numeric_grad(fun, a, eps=1e-6):
    g = np.zeros_like(a)
    it = np.nditer(a, flags=["multi_index"])
    for _ in it:
        i = it.multi_index
        old = a[i]
        a[i] = old + eps
        fp = fun()
        a[i] = old - eps
        fm = fun()
        a[i] = old
        g[i] = (fp - fm) / (2 * eps)
    return g


def test_gradients_match_central_finite_differences():
    cfg, d, idx, w, dout = case(3)
    got = mok_ref.backward(d["x"], d["W_gate_up"], d["W_down"], d["W_sgu"], d["W_sd"], idx, w, dout)
    x, Wgu, Wd, Wsgu, Wsd = f64(d["x"]), f64(d["W_gate_up"]), f64(d["W_down"]), f64(d["W_sgu"]), f64(d["W_sd"])
    wv = w.copy()
    loss = lambda: float((forward_np(x, Wgu, Wd, Wsgu, Wsd, idx, wv) * dout).sum())
    for name, arr in (("dx", x), ("dw", wv), ("dW_gate_up", Wgu), ("dW_down", Wd), ("dW_sgu", Wsgu), ("dW_sd", Wsd)):
        num = numeric_grad(loss, arr)
        err = np.abs(got[name] - num).max()
        assert err <= 2e-7 * max(1.0, np.abs(num).max()), (name, err)
        assert np.abs(num).max() > 1e-3, name                      # the pin is not vacuous


def test_router_weight_gradient_is_the_expert_output_dotted_with_dout():
    cfg, d, idx, w, dout = case(4, T=7, k=3, E=5)
    got = mok_ref.backward(d["x"], d["W_gate_up"], d["W_down"], d["W_sgu"], d["W_sd"], idx, w, dout, weights=False)
    tok = np.arange(cfg.T)
    for s in range(cfg.k):
        onehot = np.zeros_like(w)
        onehot[:, s] = 1.0
        # forward oracle with weight 1 on slot s only and no shared expert = f_{idx[t,s]}(x[t])
        y = mok_ref.ffn_tokens(d["x"], d["W_gate_up"], d["W_down"], None, None, idx, onehot, tok)
        want = (y * dout).sum(axis=1)
        assert np.abs(got["dw"][:, s] - want).max() <= 1e-12 * max(1.0, np.abs(want).max())


def test_special_cases():
    cfg, d, idx, w, dout = case(5)
    base = mok_ref.backward(d["x"], d["W_gate_up"], d["W_down"], d["W_sgu"], d["W_sd"], idx, w, dout)
    # linear in dout
    twice = mok_ref.backward(d["x"], d["W_gate_up"], d["W_down"], d["W_sgu"], d["W_sd"], idx, w, 2.0 * dout)
    for name in base:
        assert np.allclose(twice[name], 2.0 * base[name], rtol=1e-13, atol=0)
    # dout = 0 => every gradient is zero
    zero = mok_ref.backward(d["x"], d["W_gate_up"], d["W_down"], d["W_sgu"], d["W_sd"], idx, w, 0.0 * dout)
    assert all((v == 0).all() for v in zero.values())
    # routed W_down = 0: dx comes from the shared expert only, routed dW_gate_up vanishes, dw = 0
    zd = np.zeros_like(d["W_down"])
    g0 = mok_ref.backward(d["x"], d["W_gate_up"], zd, d["W_sgu"], d["W_sd"], idx, w, dout)
    assert (g0["dW_gate_up"] == 0).all() and (g0["dw"] == 0).all()
    only_shared = mok_ref.backward(d["x"], d["W_gate_up"], zd, d["W_sgu"], d["W_sd"], idx, 0.0 * w, dout)
    assert np.array_equal(g0["dx"], only_shared["dx"])
    assert np.array_equal(g0["dW_sgu"], base["dW_sgu"]) and np.array_equal(g0["dW_sd"], base["dW_sd"])
    # an expert nobody selected gets a zero weight gradient
    unused = sorted(set(range(cfg.E)) - set(idx.ravel().tolist()))
    for e in unused:
        assert (base["dW_gate_up"][e] == 0).all() and (base["dW_down"][e] == 0).all()
    # dW_down of expert e is the sum over its routes of (w dout) h^T: total over experts equals one big outer sum
    x = f64(d["x"])
    silu = lambda z: z / (1 + np.exp(-z))
    acc = np.zeros_like(base["dW_down"])
    for t in range(cfg.T):
        for s in range(cfg.k):
            e = idx[t, s]
            gu = f64(d["W_gate_up"])[e] @ x[t]
            acc[e] += np.outer(w[t, s] * dout[t], silu(gu[:cfg.I]) * gu[cfg.I:])
    assert np.abs(acc - base["dW_down"]).max() <= 1e-12 * np.abs(acc).max()


def test_token_subset_equals_the_full_backward():
    cfg, d, idx, w, dout = case(6, T=9)
    full = mok_ref.backward(d["x"], d["W_gate_up"], d["W_down"], d["W_sgu"], d["W_sd"], idx, w, dout, weights=False)
    tok = np.array([7, 0, 3], np.int32)
    dx, dw = mok_ref.backward_tokens(d["x"], d["W_gate_up"], d["W_down"], d["W_sgu"], d["W_sd"], idx, w, dout, tok)
    assert np.array_equal(dx, full["dx"][tok]) and np.array_equal(dw, full["dw"][tok])
