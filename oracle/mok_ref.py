"""ctypes/numpy front end of the CPU oracle (oracle/mok_ref.c).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's cpu-baseline leg may import this module; it
imports nothing from the CUDA package.  bf16 tensors are numpy uint16 arrays of bit patterns.
Every function cites the passage of the paper it follows in oracle/mok_ref.c.
"""
import ctypes

import numpy as np

from . import build as _build

_lib = None

_u16p = np.ctypeslib.ndpointer(np.uint16, flags="C_CONTIGUOUS")
_f32p = np.ctypeslib.ndpointer(np.float32, flags="C_CONTIGUOUS")
_f64p = np.ctypeslib.ndpointer(np.float64, flags="C_CONTIGUOUS")
_i32p = np.ctypeslib.ndpointer(np.int32, flags="C_CONTIGUOUS")


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(_build.build())
        _lib.mok_ref_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().mok_ref_num_threads())


def _ptr(a, dtype):
    """Optional array -> void pointer (None -> NULL)."""
    if a is None:
        return None
    assert a.dtype == dtype and a.flags["C_CONTIGUOUS"], (a.dtype, dtype)
    return a.ctypes.data_as(ctypes.c_void_p)


def _check(rc, what):
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")


def logits(x, W_r, bias=None):
    """Router projection (Section 2.1): fp64 logits[T,E] from bf16-bit x[T,H], fp32 W_r[E,H], fp32 bias[E]."""
    T, H = x.shape
    E = W_r.shape[0]
    out = np.empty((T, E), np.float64)
    rc = lib().mok_ref_logits(_ptr(x, np.uint16), _ptr(W_r, np.float32), _ptr(bias, np.float32),
                              T, H, E, _ptr(out, np.float64))
    _check(rc, "logits")
    return out


def topk(lg, k):
    """Top-k by (logit desc, expert id asc) (Section 2.1).  Returns idx[T,k] int32, gap[T] fp64."""
    T, E = lg.shape
    idx = np.empty((T, k), np.int32)
    gap = np.empty((T,), np.float64)
    _check(lib().mok_ref_topk(_ptr(lg, np.float64), T, E, k, _ptr(idx, np.int32), _ptr(gap, np.float64)), "topk")
    return idx, gap


def weights(lg, idx):
    """Normalised router weights s_i / sum_j s_j with s = softmax over all E (Section 2.1 equation)."""
    T, E = lg.shape
    k = idx.shape[1]
    w = np.empty((T, k), np.float64)
    _check(lib().mok_ref_weights(_ptr(lg, np.float64), _ptr(np.ascontiguousarray(idx, np.int32), np.int32),
                                 T, E, k, _ptr(w, np.float64)), "weights")
    return w


def route(x, W_r, bias, k):
    """logits -> (idx, w, gap, logits)."""
    lg = logits(x, W_r, bias)
    idx, gap = topk(lg, k)
    return idx, weights(lg, idx), gap, lg


def schedule(a, E):
    """Algorithm 1 for one rank.  a = flattened routes (token-major).  Returns counts, offsets, perm, inv."""
    a = np.ascontiguousarray(a, np.int32).ravel()
    n = a.size
    counts = np.empty((E,), np.int32)
    offsets = np.empty((E + 1,), np.int32)
    perm = np.empty((max(n, 1),), np.int32)
    inv = np.empty((max(n, 1),), np.int32)
    _check(lib().mok_ref_schedule(_ptr(a, np.int32), n, E, _ptr(counts, np.int32), _ptr(offsets, np.int32),
                                  _ptr(perm, np.int32), _ptr(inv, np.int32)), "schedule")
    return counts, offsets, perm[:n], inv[:n]


def alg1(A, L, c):
    """The pull schedule Algorithm 1 defines for destination rank c and R source ranks (Section 3.1), built as a sort by
    (local expert, ordinal, source rank).  A[R,NK] global expert per route.  Returns S[L+1], phi_rank, phi_idx
    (length S[L])."""
    A = np.ascontiguousarray(A, np.int32)
    R, NK = A.shape
    S = np.empty((L + 1,), np.int32)
    pr = np.full((max(R * NK, 1),), -1, np.int32)
    pi = np.full((max(R * NK, 1),), -1, np.int32)
    _check(lib().mok_ref_alg1(_ptr(A, np.int32), R, NK, L, c, _ptr(S, np.int32), _ptr(pr, np.int32),
                              _ptr(pi, np.int32)), "alg1")
    n = int(S[L])
    return S, pr[:n], pi[:n]


def ffn_tokens(x, W_gate_up, W_down, W_sgu, W_sd, idx, w, tokens, mimic_bf16=False):
    """MoE equation of Section 2.1 evaluated per token from the definition, for the listed tokens.  out[n,H] fp64."""
    T, H = x.shape
    k = idx.shape[1]
    if W_gate_up is not None:
        E, twoI, _ = W_gate_up.shape
        I = twoI // 2
    else:
        E, I = 0, 0
    I_s = 0 if W_sgu is None else W_sgu.shape[0] // 2
    tokens = np.ascontiguousarray(tokens, np.int32)
    out = np.empty((tokens.size, H), np.float64)
    rc = lib().mok_ref_ffn_tokens(_ptr(x, np.uint16), _ptr(W_gate_up, np.uint16), _ptr(W_down, np.uint16),
                                  _ptr(W_sgu, np.uint16), _ptr(W_sd, np.uint16),
                                  H, I, I_s, E, k,
                                  _ptr(np.ascontiguousarray(idx, np.int32), np.int32),
                                  _ptr(np.ascontiguousarray(w, np.float64), np.float64),
                                  _ptr(tokens, np.int32), int(tokens.size), int(bool(mimic_bf16)),
                                  _ptr(out, np.float64))
    _check(rc, "ffn_tokens")
    return out


def forward(x, W_r, bias, W_gate_up, W_down, W_sgu, W_sd, k):
    """Whole layer for every token.  Returns out[T,H] fp64, idx[T,k], w[T,k]."""
    T, H = x.shape
    E = W_r.shape[0]
    I = W_gate_up.shape[1] // 2
    I_s = 0 if W_sgu is None else W_sgu.shape[0] // 2
    out = np.zeros((T, H), np.float64)
    idx = np.empty((T, k), np.int32)
    w = np.empty((T, k), np.float64)
    rc = lib().mok_ref_forward(_ptr(x, np.uint16), _ptr(W_r, np.float32), _ptr(bias, np.float32),
                               _ptr(W_gate_up, np.uint16), _ptr(W_down, np.uint16),
                               _ptr(W_sgu, np.uint16), _ptr(W_sd, np.uint16),
                               T, H, I, I_s, E, k, _ptr(out, np.float64), _ptr(idx, np.int32), _ptr(w, np.float64))
    _check(rc, "forward")
    return out, idx, w


# ---- MXFP8 mode of the routed experts (Section 3.4 "MXFP8 Support"; oracle/mok_ref_mx.c) ----

def e4m3_decode(codes):
    """The real number of every E4M3 code (uint8 array) as fp64; NaN codes decode to NaN."""
    lib().mok_ref_e4m3_decode.restype = ctypes.c_double
    lib().mok_ref_e4m3_decode.argtypes = [ctypes.c_uint8]
    c = np.asarray(codes, np.uint8)
    return np.array([lib().mok_ref_e4m3_decode(int(v)) for v in c.ravel()], np.float64).reshape(c.shape)


def e4m3_encode(values):
    """Nearest E4M3 code of every finite fp64 value (ties to even, clamped to +-448)."""
    lib().mok_ref_e4m3_encode.restype = ctypes.c_uint8
    lib().mok_ref_e4m3_encode.argtypes = [ctypes.c_double]
    v = np.asarray(values, np.float64)
    return np.array([lib().mok_ref_e4m3_encode(float(a)) for a in v.ravel()], np.uint8).reshape(v.shape)


def mx_quantize(values):
    """fp64 [rows, cols] (cols % 32 == 0) -> (codes uint8 [rows, cols], scales uint8 [rows, cols/32])."""
    v = np.ascontiguousarray(values, np.float64)
    rows, cols = v.shape
    codes = np.empty((rows, cols), np.uint8)
    scales = np.empty((rows, cols // 32), np.uint8)
    _check(lib().mok_ref_mx_quantize(_ptr(v, np.float64), ctypes.c_longlong(rows), cols, _ptr(codes, np.uint8),
                                     _ptr(scales, np.uint8)), "mx_quantize")
    return codes, scales


def mx_dequantize(codes, scales):
    rows, cols = codes.shape
    out = np.empty((rows, cols), np.float64)
    _check(lib().mok_ref_mx_dequantize(_ptr(np.ascontiguousarray(codes), np.uint8),
                                       _ptr(np.ascontiguousarray(scales), np.uint8), ctypes.c_longlong(rows), cols,
                                       _ptr(out, np.float64)), "mx_dequantize")
    return out


def mx_roundtrip_bf16(bits):
    """bf16 bit patterns [..., cols] -> fp32 array of the numbers their MXFP8 quantisation (blocks along the last
    index) stands for."""
    b = np.ascontiguousarray(bits, np.uint16)
    cols = b.shape[-1]
    rows = b.size // cols
    out = np.empty(b.shape, np.float32)
    _check(lib().mok_ref_mx_roundtrip_bf16(_ptr(b, np.uint16), ctypes.c_longlong(rows), cols, _ptr(out, np.float32)),
           "mx_roundtrip_bf16")
    return out


def ffn_tokens_mx(x, Wgu_q, Wd_q, W_sgu, W_sd, idx, w, tokens):
    """MoE equation with MXFP8 routed experts and a bf16 shared expert, per token from the definition.
    Wgu_q / Wd_q: mx_roundtrip_bf16 of W_gate_up / W_down.  out[n,H] fp64."""
    T, H = x.shape
    k = idx.shape[1]
    E, twoI, _ = Wgu_q.shape
    I = twoI // 2
    I_s = 0 if W_sgu is None else W_sgu.shape[0] // 2
    tokens = np.ascontiguousarray(tokens, np.int32)
    out = np.empty((tokens.size, H), np.float64)
    rc = lib().mok_ref_ffn_tokens_mx(_ptr(x, np.uint16), _ptr(np.ascontiguousarray(Wgu_q, np.float32), np.float32),
                                     _ptr(np.ascontiguousarray(Wd_q, np.float32), np.float32),
                                     _ptr(W_sgu, np.uint16), _ptr(W_sd, np.uint16), H, I, I_s, E, k,
                                     _ptr(np.ascontiguousarray(idx, np.int32), np.int32),
                                     _ptr(np.ascontiguousarray(w, np.float64), np.float64),
                                     _ptr(tokens, np.int32), int(tokens.size), _ptr(out, np.float64))
    _check(rc, "ffn_tokens_mx")
    return out


# ---- backward pass (oracle/mok_ref_bwd.c): the derivative of the Section 2.1 definition ----

def backward(x, W_gate_up, W_down, W_sgu, W_sd, idx, w, dout, weights=True):
    """dout fp64 [T,H] -> dict(dx [T,H], dw [T,k], and with weights=True dW_gate_up [E,2I,H], dW_down [E,H,I],
    dW_sgu, dW_sd), all fp64.  The router weights w are inputs of the layer; dw is their gradient."""
    T, H = x.shape
    k = idx.shape[1]
    E, twoI, _ = W_gate_up.shape
    I = twoI // 2
    I_s = 0 if W_sgu is None else W_sgu.shape[0] // 2
    out = {"dx": np.empty((T, H), np.float64), "dw": np.empty((T, k), np.float64)}
    if weights:
        out["dW_gate_up"] = np.empty((E, 2 * I, H), np.float64)
        out["dW_down"] = np.empty((E, H, I), np.float64)
        if I_s:
            out["dW_sgu"] = np.empty((2 * I_s, H), np.float64)
            out["dW_sd"] = np.empty((H, I_s), np.float64)
    g = lambda name: _ptr(out[name], np.float64) if name in out else None
    rc = lib().mok_ref_backward(_ptr(x, np.uint16), _ptr(W_gate_up, np.uint16), _ptr(W_down, np.uint16),
                                _ptr(W_sgu, np.uint16), _ptr(W_sd, np.uint16), T, H, I, I_s, E, k,
                                _ptr(np.ascontiguousarray(idx, np.int32), np.int32),
                                _ptr(np.ascontiguousarray(w, np.float64), np.float64),
                                _ptr(np.ascontiguousarray(dout, np.float64), np.float64),
                                g("dx"), g("dw"), g("dW_gate_up"), g("dW_down"), g("dW_sgu"), g("dW_sd"))
    _check(rc, "backward")
    return out


def backward_tokens(x, W_gate_up, W_down, W_sgu, W_sd, idx, w, dout, tokens):
    """dx [n,H] and dw [n,k] of the listed tokens only (full-size checks); same chain rule as backward()."""
    T, H = x.shape
    k = idx.shape[1]
    E, twoI, _ = W_gate_up.shape
    I = twoI // 2
    I_s = 0 if W_sgu is None else W_sgu.shape[0] // 2
    tokens = np.ascontiguousarray(tokens, np.int32)
    dx = np.empty((tokens.size, H), np.float64)
    dw = np.empty((tokens.size, k), np.float64)
    rc = lib().mok_ref_backward_tokens(_ptr(x, np.uint16), _ptr(W_gate_up, np.uint16), _ptr(W_down, np.uint16),
                                       _ptr(W_sgu, np.uint16), _ptr(W_sd, np.uint16), H, I, I_s, E, k,
                                       _ptr(np.ascontiguousarray(idx, np.int32), np.int32),
                                       _ptr(np.ascontiguousarray(w, np.float64), np.float64),
                                       _ptr(np.ascontiguousarray(dout, np.float64), np.float64),
                                       _ptr(tokens, np.int32), int(tokens.size), _ptr(dx, np.float64), _ptr(dw, np.float64))
    _check(rc, "backward_tokens")
    return dx, dw
