"""Thin Python binding over the C-ABI library libmok.so (see include/mok.h).

Argument marshalling only: every step of the layer runs in the library's CUDA kernels.  PyTorch is used for
device memory and streams.  Importing this module fails loudly if the library has not been built
(`python -m paper_2609_36070_b200.build`); there is no CPU or PyTorch fallback.
"""
import ctypes
import os

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libmok.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2609_36070_b200.build`")
_lib = ctypes.CDLL(_LIB_PATH)

MOK_OK = 0
MOK_ERR_NULL, MOK_ERR_SHAPE, MOK_ERR_ALIGN, MOK_ERR_WORKSPACE = -1, -2, -3, -4
MOK_ERR_CUDA, MOK_ERR_TIMEOUT, MOK_ERR_SCHEDULE, MOK_ERR_UNSUPPORTED = -5, -6, -7, -8
MOK_IMPL_TCGEN05, MOK_IMPL_SIMT, MOK_IMPL_TCGEN05_TN = 0, 1, 2

EXPORTS = ["mok_moe_forward", "mok_workspace_bytes", "mok_workspace_bytes_ring", "mok_moe_forward_ex", "mok_moe_forward_host",
           "mok_moe_forward_host_async", "mok_host_wait", "mok_route",
           "mok_schedule", "mok_read_status", "mok_launch_count", "mok_last_cuda_error", "mok_status_string",
           "mok_version", "mok_profile_begin", "mok_profile_end", "mok_schedule_noalloc", "mok_debug_counters",
           "mok_ep_workspace_bytes", "mok_ep_y_rows", "mok_ep_expert_ffn", "mok_ep_combine",
           "mok_mx_scale_bytes", "mok_mx_quantize_weights", "mok_mx_quantize_rows", "mok_mx_workspace_bytes",
           "mok_ep_mx_workspace_bytes", "mok_bwd_workspace_bytes", "mok_moe_backward", "mok_ep_bwd_workspace_bytes",
           "mok_ep_expert_bwd", "mok_ep_bwd_combine", "mok_selftest_per_device",
           "mok_router_prepared_bytes", "mok_router_prepare"]
MOK_PRECISION_BF16, MOK_PRECISION_MXFP8 = 0, 1
MOK_H_RING_MIN_TILES = 24
MOK_MAX_RANKS = 16
MOK_NOALLOC_MAX_ROUTES = 32768
MOK_DEBUG_STARVE = 2
MOK_DEBUG_NO_ARRIVALS = 3
STAGES = ["router", "schedule", "gather", "gemm1", "gemm2", "shared_gemm1", "shared_gemm2", "combine"]


class mok_config(ctypes.Structure):
    _fields_ = [("impl", ctypes.c_int32), ("grid", ctypes.c_int32), ("router_impl", ctypes.c_int32),
                ("profile", ctypes.c_int32), ("gather_mode", ctypes.c_int32), ("cta_group", ctypes.c_int32),
                ("debug", ctypes.c_int32), ("host_chunks", ctypes.c_int32), ("precision", ctypes.c_int32),
                ("tile_sched", ctypes.c_int32), ("macrobatch_tokens", ctypes.c_int32),
                ("fused_ffn", ctypes.c_int32), ("fused_window", ctypes.c_int32), ("gang_sync", ctypes.c_int32),
                ("serial_launches", ctypes.c_int32), ("h_ring_tiles", ctypes.c_int32),
                ("shared_overlap", ctypes.c_int32), ("comm_ctas", ctypes.c_int32)]


class mok_args(ctypes.Structure):
    _fields_ = [("x", ctypes.c_void_p), ("W_router", ctypes.c_void_p), ("router_bias", ctypes.c_void_p),
                ("W_gate_up", ctypes.c_void_p), ("W_down", ctypes.c_void_p),
                ("W_shared_gate_up", ctypes.c_void_p), ("W_shared_down", ctypes.c_void_p),
                ("T", ctypes.c_int32), ("H", ctypes.c_int32), ("I", ctypes.c_int32), ("I_shared", ctypes.c_int32),
                ("E", ctypes.c_int32), ("k", ctypes.c_int32),
                ("out", ctypes.c_void_p), ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
                ("topk_idx", ctypes.c_void_p), ("topk_w", ctypes.c_void_p), ("counts", ctypes.c_void_p),
                ("offsets", ctypes.c_void_p), ("perm", ctypes.c_void_p), ("inv_perm", ctypes.c_void_p),
                ("config", ctypes.POINTER(mok_config)), ("stream", ctypes.c_void_p),
                ("W_gate_up_codes", ctypes.c_void_p), ("W_gate_up_scales", ctypes.c_void_p),
                ("W_down_codes", ctypes.c_void_p), ("W_down_scales", ctypes.c_void_p),
                ("W_router_split", ctypes.c_void_p)]


class mok_ep_args(ctypes.Structure):
    _fields_ = [("rank", ctypes.c_int32), ("n_ranks", ctypes.c_int32),
                ("T_local", ctypes.c_int32), ("H", ctypes.c_int32), ("I", ctypes.c_int32), ("I_shared", ctypes.c_int32),
                ("E", ctypes.c_int32), ("k", ctypes.c_int32),
                ("x_peers", ctypes.c_void_p * MOK_MAX_RANKS), ("idx_all", ctypes.c_void_p),
                ("W_gate_up", ctypes.c_void_p), ("W_down", ctypes.c_void_p),
                ("W_shared_gate_up", ctypes.c_void_p), ("W_shared_down", ctypes.c_void_p),
                ("y", ctypes.c_void_p), ("y_rows", ctypes.c_int64), ("pos", ctypes.c_void_p),
                ("y_shared", ctypes.c_void_p),
                ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
                ("M", ctypes.c_void_p), ("S", ctypes.c_void_p), ("phi_rank", ctypes.c_void_p),
                ("phi_index", ctypes.c_void_p), ("schedule_only", ctypes.c_int32),
                ("config", ctypes.POINTER(mok_config)), ("stream", ctypes.c_void_p),
                ("x_codes_peers", ctypes.c_void_p * MOK_MAX_RANKS), ("x_scales_peers", ctypes.c_void_p * MOK_MAX_RANKS),
                ("W_gate_up_codes", ctypes.c_void_p), ("W_gate_up_scales", ctypes.c_void_p),
                ("W_down_codes", ctypes.c_void_p), ("W_down_scales", ctypes.c_void_p)]


class mok_ep_combine_args(ctypes.Structure):
    _fields_ = [("rank", ctypes.c_int32), ("n_ranks", ctypes.c_int32),
                ("T_local", ctypes.c_int32), ("H", ctypes.c_int32), ("E", ctypes.c_int32), ("k", ctypes.c_int32),
                ("topk_idx", ctypes.c_void_p), ("topk_w", ctypes.c_void_p),
                ("y_peers", ctypes.c_void_p * MOK_MAX_RANKS), ("pos_peers", ctypes.c_void_p * MOK_MAX_RANKS),
                ("y_shared", ctypes.c_void_p), ("out", ctypes.c_void_p), ("stream", ctypes.c_void_p)]


class mok_ep_bwd_args(ctypes.Structure):
    _fields_ = [("rank", ctypes.c_int32), ("n_ranks", ctypes.c_int32),
                ("T_local", ctypes.c_int32), ("H", ctypes.c_int32), ("I", ctypes.c_int32), ("I_shared", ctypes.c_int32),
                ("E", ctypes.c_int32), ("k", ctypes.c_int32),
                ("x_peers", ctypes.c_void_p * MOK_MAX_RANKS), ("dout_peers", ctypes.c_void_p * MOK_MAX_RANKS),
                ("idx_all", ctypes.c_void_p), ("w_all", ctypes.c_void_p),
                ("W_gate_up", ctypes.c_void_p), ("W_down", ctypes.c_void_p),
                ("W_shared_gate_up", ctypes.c_void_p), ("W_shared_down", ctypes.c_void_p),
                ("dxg", ctypes.c_void_p), ("dxg_rows", ctypes.c_longlong), ("pos", ctypes.c_void_p),
                ("dw_routes", ctypes.c_void_p), ("dx_shared", ctypes.c_void_p),
                ("dW_gate_up", ctypes.c_void_p), ("dW_down", ctypes.c_void_p),
                ("dW_shared_gate_up", ctypes.c_void_p), ("dW_shared_down", ctypes.c_void_p),
                ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
                ("config", ctypes.POINTER(mok_config)), ("stream", ctypes.c_void_p)]


class mok_ep_bwd_combine_args(ctypes.Structure):
    _fields_ = [("rank", ctypes.c_int32), ("n_ranks", ctypes.c_int32),
                ("T_local", ctypes.c_int32), ("H", ctypes.c_int32), ("E", ctypes.c_int32), ("k", ctypes.c_int32),
                ("topk_idx", ctypes.c_void_p),
                ("dxg_peers", ctypes.c_void_p * MOK_MAX_RANKS), ("pos_peers", ctypes.c_void_p * MOK_MAX_RANKS),
                ("dw_peers", ctypes.c_void_p * MOK_MAX_RANKS),
                ("dx_shared", ctypes.c_void_p), ("dx", ctypes.c_void_p), ("dw", ctypes.c_void_p),
                ("stream", ctypes.c_void_p)]


class mok_bwd_args(ctypes.Structure):
    _fields_ = [("x", ctypes.c_void_p), ("W_gate_up", ctypes.c_void_p), ("W_down", ctypes.c_void_p),
                ("W_shared_gate_up", ctypes.c_void_p), ("W_shared_down", ctypes.c_void_p),
                ("T", ctypes.c_int32), ("H", ctypes.c_int32), ("I", ctypes.c_int32), ("I_shared", ctypes.c_int32),
                ("E", ctypes.c_int32), ("k", ctypes.c_int32),
                ("topk_idx", ctypes.c_void_p), ("topk_w", ctypes.c_void_p), ("dout", ctypes.c_void_p),
                ("dx", ctypes.c_void_p), ("dw", ctypes.c_void_p), ("dW_gate_up", ctypes.c_void_p),
                ("dW_down", ctypes.c_void_p), ("dW_shared_gate_up", ctypes.c_void_p), ("dW_shared_down", ctypes.c_void_p),
                ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
                ("config", ctypes.POINTER(mok_config)), ("stream", ctypes.c_void_p)]


_lib.mok_bwd_workspace_bytes.restype = ctypes.c_size_t
_lib.mok_bwd_workspace_bytes.argtypes = [ctypes.c_int] * 6
_lib.mok_moe_backward.restype = ctypes.c_int
_lib.mok_moe_backward.argtypes = [ctypes.POINTER(mok_bwd_args)]
_lib.mok_ep_workspace_bytes.restype = ctypes.c_size_t
_lib.mok_ep_workspace_bytes.argtypes = [ctypes.c_int] * 7
_lib.mok_ep_mx_workspace_bytes.restype = ctypes.c_size_t
_lib.mok_ep_mx_workspace_bytes.argtypes = [ctypes.c_int] * 7
_lib.mok_ep_y_rows.restype = ctypes.c_longlong
_lib.mok_ep_y_rows.argtypes = [ctypes.c_int] * 4
_lib.mok_ep_expert_ffn.restype = ctypes.c_int
_lib.mok_ep_expert_ffn.argtypes = [ctypes.POINTER(mok_ep_args)]
_lib.mok_ep_combine.restype = ctypes.c_int
_lib.mok_ep_combine.argtypes = [ctypes.POINTER(mok_ep_combine_args)]
_lib.mok_workspace_bytes.restype = ctypes.c_size_t
_lib.mok_workspace_bytes.argtypes = [ctypes.c_int] * 6
_lib.mok_ep_bwd_workspace_bytes.restype = ctypes.c_size_t
_lib.mok_ep_bwd_workspace_bytes.argtypes = [ctypes.c_int] * 7
_lib.mok_workspace_bytes_ring.restype = ctypes.c_size_t
_lib.mok_workspace_bytes_ring.argtypes = [ctypes.c_int] * 7
_lib.mok_mx_workspace_bytes.restype = ctypes.c_size_t
_lib.mok_mx_workspace_bytes.argtypes = [ctypes.c_int] * 6
_lib.mok_mx_scale_bytes.restype = ctypes.c_size_t
_lib.mok_mx_scale_bytes.argtypes = [ctypes.c_int] * 3
_lib.mok_mx_quantize_weights.restype = ctypes.c_int
_lib.mok_mx_quantize_weights.argtypes = [ctypes.c_void_p] + [ctypes.c_int] * 3 + [ctypes.c_void_p] * 3
_lib.mok_mx_quantize_rows.restype = ctypes.c_int
_lib.mok_mx_quantize_rows.argtypes = [ctypes.c_void_p] + [ctypes.c_int] * 2 + [ctypes.c_void_p] * 3
_lib.mok_moe_forward.restype = ctypes.c_int
_lib.mok_moe_forward.argtypes = [ctypes.c_void_p] * 6 + [ctypes.c_int] * 6 + [ctypes.c_void_p] * 2
_lib.mok_moe_forward_ex.restype = ctypes.c_int
_lib.mok_moe_forward_ex.argtypes = [ctypes.POINTER(mok_args)]
_lib.mok_moe_forward_host.restype = ctypes.c_int
_lib.mok_moe_forward_host.argtypes = [ctypes.POINTER(mok_args), ctypes.c_void_p, ctypes.c_void_p]
_lib.mok_moe_forward_host_async.restype = ctypes.c_int
_lib.mok_moe_forward_host_async.argtypes = [ctypes.POINTER(mok_args), ctypes.c_void_p, ctypes.c_void_p]
_lib.mok_host_wait.restype = ctypes.c_int
_lib.mok_host_wait.argtypes = []
_lib.mok_route.restype = ctypes.c_int
_lib.mok_route.argtypes = ([ctypes.c_void_p] * 3 + [ctypes.c_int] * 4 + [ctypes.c_void_p] * 3 +
                           [ctypes.c_size_t, ctypes.POINTER(mok_config), ctypes.c_void_p])
_lib.mok_schedule.restype = ctypes.c_int
_lib.mok_schedule.argtypes = ([ctypes.c_void_p] + [ctypes.c_int] * 3 + [ctypes.c_void_p] * 5 +
                              [ctypes.c_size_t, ctypes.c_void_p])
_lib.mok_schedule_noalloc.restype = ctypes.c_int
_lib.mok_schedule_noalloc.argtypes = [ctypes.c_void_p] + [ctypes.c_int] * 3 + [ctypes.c_void_p] * 5
_lib.mok_debug_counters.restype = ctypes.c_int
_lib.mok_debug_counters.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
_lib.mok_read_status.restype = ctypes.c_int
_lib.mok_read_status.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
_lib.mok_launch_count.restype = ctypes.c_int
_lib.mok_launch_count.argtypes = [ctypes.c_int] * 6 + [ctypes.POINTER(mok_config)]
_lib.mok_last_cuda_error.restype = ctypes.c_int
_lib.mok_status_string.restype = ctypes.c_char_p
_lib.mok_status_string.argtypes = [ctypes.c_int]
_lib.mok_version.restype = ctypes.c_int
_lib.mok_router_prepared_bytes.restype = ctypes.c_size_t
_lib.mok_router_prepared_bytes.argtypes = [ctypes.c_int] * 2
_lib.mok_router_prepare.restype = ctypes.c_int
_lib.mok_router_prepare.argtypes = ([ctypes.c_void_p] + [ctypes.c_int] * 3 + [ctypes.POINTER(mok_config), ctypes.c_void_p,
                                    ctypes.c_size_t, ctypes.c_void_p])
_lib.mok_selftest_per_device.restype = ctypes.c_int
_lib.mok_selftest_per_device.argtypes = []
_lib.mok_profile_begin.restype = ctypes.c_int
_lib.mok_profile_begin.argtypes = [ctypes.c_int]
_lib.mok_profile_end.restype = ctypes.c_int
_lib.mok_profile_end.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(ctypes.c_int)]


class MokError(RuntimeError):
    def __init__(self, status):
        self.status = status
        msg = _lib.mok_status_string(status).decode()
        if status == MOK_ERR_CUDA:
            msg += f" (cudaError {_lib.mok_last_cuda_error()})"
        super().__init__(f"libmok: {msg} [{status}]")


def _check(status):
    if status != MOK_OK:
        raise MokError(status)


def _p(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _config(impl=0, grid=0, router_impl=0, profile=0, gather_mode=0, cta_group=0, debug=0, host_chunks=0,
            precision=0, tile_sched=0, macrobatch_tokens=0, fused_ffn=0, fused_window=0, gang_sync=0, serial_launches=0,
            h_ring_tiles=0, shared_overlap=0, comm_ctas=0):
    c = mok_config()
    c.comm_ctas = comm_ctas
    c.shared_overlap = shared_overlap
    c.serial_launches = serial_launches
    c.h_ring_tiles = h_ring_tiles
    c.gang_sync = gang_sync
    c.fused_ffn, c.fused_window = fused_ffn, fused_window
    c.precision = precision
    c.tile_sched = tile_sched
    c.macrobatch_tokens = macrobatch_tokens
    c.impl, c.grid, c.router_impl, c.profile, c.gather_mode = impl, grid, router_impl, profile, gather_mode
    c.cta_group = cta_group
    c.debug = debug
    c.host_chunks = host_chunks
    return c


def mok_profile_begin(max_calls):
    _check(_lib.mok_profile_begin(max_calls))


def mok_profile_end(max_calls):
    """Returns a list of per-call dicts {stage name: milliseconds} for the calls recorded since mok_profile_begin."""
    buf = (ctypes.c_float * (max_calls * len(STAGES)))()
    n = ctypes.c_int(0)
    _check(_lib.mok_profile_end(buf, max_calls, ctypes.byref(n)))
    return [{s: buf[c * len(STAGES) + i] for i, s in enumerate(STAGES)} for c in range(n.value)]


def mok_version():
    return int(_lib.mok_version())


def mok_selftest_per_device():
    """0 if the library's per-device launch-state cache behaves (host-only check, no CUDA call)."""
    return int(_lib.mok_selftest_per_device())


def mok_status_string(status):
    return _lib.mok_status_string(status).decode()


def mok_workspace_bytes(T, H, I, I_shared, E, k):
    return int(_lib.mok_workspace_bytes(T, H, I, I_shared, E, k))


def mok_workspace_bytes_ring(T, H, I, I_shared, E, k, h_ring_tiles):
    return int(_lib.mok_workspace_bytes_ring(T, H, I, I_shared, E, k, h_ring_tiles))


def mok_launch_count(T, H, I, I_shared, E, k, config=None):
    return int(_lib.mok_launch_count(T, H, I, I_shared, E, k, None if config is None else ctypes.pointer(config)))


def mok_mx_workspace_bytes(T, H, I, I_shared, E, k):
    return int(_lib.mok_mx_workspace_bytes(T, H, I, I_shared, E, k))


class MxWeights:
    """The routed weights pre-quantised to MXFP8 by the library's quantisation kernel (Section 3.4)."""

    def __init__(self, W_gate_up, W_down, stream=None):
        E, twoI, H = W_gate_up.shape
        I = twoI // 2
        self.gate_up_codes, self.gate_up_scales = mok_mx_quantize_weights(W_gate_up.view(2 * E, I, H), stream)
        self.down_codes, self.down_scales = mok_mx_quantize_weights(W_down, stream)


def mok_mx_quantize_weights(W, stream=None):
    """W bf16 [groups, rows, K] -> (codes uint8 [groups, rows, K], scales uint8 in the MMA's atom layout)."""
    groups, rows, K = W.shape
    n = int(_lib.mok_mx_scale_bytes(groups, rows, K))
    if n == 0:
        raise MokError(MOK_ERR_SHAPE)
    codes = torch.empty((groups, rows, K), dtype=torch.uint8, device=W.device)
    scales = torch.empty((n,), dtype=torch.uint8, device=W.device)
    _check(_lib.mok_mx_quantize_weights(_p(W), groups, rows, K, _p(codes), _p(scales), _stream(stream)))
    return codes, scales


def mok_mx_quantize_rows(x, stream=None):
    """x bf16 [rows, K] -> (codes uint8 [rows, K], scales uint8 [rows, 4 * ceil(K / 128)])."""
    rows, K = x.shape
    codes = torch.empty((rows, K), dtype=torch.uint8, device=x.device)
    scales = torch.empty((rows, (K + 127) // 128 * 4), dtype=torch.uint8, device=x.device)
    _check(_lib.mok_mx_quantize_rows(_p(x), rows, K, _p(codes), _p(scales), _stream(stream)))
    return codes, scales


def alloc_workspace(T, H, I, I_shared, E, k, device="cuda", host_staging=False, mx=False, h_ring_tiles=0):
    """A torch uint8 buffer large enough for mok_moe_forward_ex (plus the x/out staging copies of the host variant;
    mx=True: plus the MXFP8 mode's quantised activations; h_ring_tiles > 0: the smaller workspace of calls whose config
    has that h_ring_tiles)."""
    if h_ring_tiles:
        n = mok_workspace_bytes_ring(T, H, I, I_shared, E, k, h_ring_tiles)
    else:
        n = (mok_mx_workspace_bytes if mx else mok_workspace_bytes)(T, H, I, I_shared, E, k)
    if n == 0:
        raise MokError(MOK_ERR_SHAPE)
    if host_staging:    # True / 1: the blocking host call; 2: the two slots of the asynchronous one
        n += (4 if host_staging == 2 else 2) * ((2 * T * H + 255) // 256 * 256)
    return torch.empty(n + 256, dtype=torch.uint8, device=device)


def _aligned_ws(ws):
    off = (-ws.data_ptr()) % 256
    return ws.data_ptr() + off, ws.numel() - off


def _shapes(x_shape, W_router, W_gate_up, W_shared_gate_up, k):
    T, H = x_shape
    E = W_router.shape[0]
    I = W_gate_up.shape[1] // 2
    I_s = 0 if W_shared_gate_up is None else W_shared_gate_up.shape[0] // 2
    return T, H, I, I_s, E, k


def mok_moe_forward(x, W_router, W_gate_up, W_down, W_shared_gate_up, W_shared_down, k, out=None, stream=None):
    """The 14-argument entry point (library-owned workspace, no router bias).  Returns out (bf16 [T,H])."""
    T, H, I, I_s, E, k = _shapes(x.shape, W_router, W_gate_up, W_shared_gate_up, k)
    if out is None:
        out = torch.empty_like(x)
    _check(_lib.mok_moe_forward(_p(x), _p(W_router), _p(W_gate_up), _p(W_down), _p(W_shared_gate_up),
                                _p(W_shared_down), T, H, I, I_s, E, k, _p(out), _stream(stream)))
    return out


def _fill_args(x_shape, W_router, router_bias, W_gate_up, W_down, W_shared_gate_up, W_shared_down, k, workspace,
               stages, config, stream, device):
    T, H, I, I_s, E, k = _shapes(x_shape, W_router, W_gate_up, W_shared_gate_up, k)
    a = mok_args()
    a.W_router = W_router.data_ptr()
    a.router_bias = None if router_bias is None else router_bias.data_ptr()
    a.W_gate_up, a.W_down = W_gate_up.data_ptr(), W_down.data_ptr()
    a.W_shared_gate_up = None if W_shared_gate_up is None else W_shared_gate_up.data_ptr()
    a.W_shared_down = None if W_shared_down is None else W_shared_down.data_ptr()
    a.T, a.H, a.I, a.I_shared, a.E, a.k = T, H, I, I_s, E, k
    a.workspace, a.workspace_bytes = _aligned_ws(workspace)
    res = {}
    if stages:
        R = T * k
        res = {"topk_idx": torch.empty((T, k), dtype=torch.int32, device=device),
               "topk_w": torch.empty((T, k), dtype=torch.float32, device=device),
               "counts": torch.empty((E,), dtype=torch.int32, device=device),
               "offsets": torch.empty((E + 1,), dtype=torch.int32, device=device),
               "perm": torch.empty((R,), dtype=torch.int32, device=device),
               "inv_perm": torch.empty((R,), dtype=torch.int32, device=device)}
        for name, t in res.items():
            setattr(a, name, t.data_ptr())
    if config is not None:
        a.config = ctypes.pointer(config)
    a.stream = _stream(stream).value
    return a, res


def mok_router_prepare(W_router, k, config=None, stream=None):
    """The exact three-way bf16 split of W_router, made once; pass the result as router_split= to the forward calls."""
    E, H = W_router.shape
    n = int(_lib.mok_router_prepared_bytes(E, H))
    if n == 0:
        raise MokError(MOK_ERR_SHAPE)
    out = torch.empty(n, dtype=torch.uint8, device=W_router.device)
    _check(_lib.mok_router_prepare(_p(W_router), E, H, k, None if config is None else ctypes.pointer(config), _p(out), n,
                                   _stream(stream)))
    return out


def mok_moe_forward_ex(x, W_router, router_bias, W_gate_up, W_down, W_shared_gate_up, W_shared_down, k, workspace,
                       out=None, stages=False, config=None, stream=None, mx_weights=None, router_split=None):
    """The layer with router bias, caller-owned workspace, optional stage outputs and knobs.

    Returns out, or (out, dict of stage tensors) when stages=True.
    """
    if out is None:
        out = torch.empty_like(x)
    a, res = _fill_args(x.shape, W_router, router_bias, W_gate_up, W_down, W_shared_gate_up, W_shared_down, k,
                        workspace, stages, config, stream, x.device)
    a.x, a.out = x.data_ptr(), out.data_ptr()
    if router_split is not None:
        a.W_router_split = router_split.data_ptr()
    if mx_weights is not None:
        a.W_gate_up_codes, a.W_gate_up_scales = mx_weights.gate_up_codes.data_ptr(), mx_weights.gate_up_scales.data_ptr()
        a.W_down_codes, a.W_down_scales = mx_weights.down_codes.data_ptr(), mx_weights.down_scales.data_ptr()
    _check(_lib.mok_moe_forward_ex(ctypes.byref(a)))
    return (out, res) if stages else out


def mok_moe_forward_host(x_host, out_host, W_router, router_bias, W_gate_up, W_down, W_shared_gate_up, W_shared_down,
                         k, workspace, config=None, stream=None, mx_weights=None):
    """Host-buffer variant: x_host / out_host are CPU (ideally pinned) bf16 tensors; blocks until out_host is filled."""
    assert not x_host.is_cuda and not out_host.is_cuda
    a, _ = _fill_args(x_host.shape, W_router, router_bias, W_gate_up, W_down, W_shared_gate_up, W_shared_down, k,
                      workspace, False, config, stream, W_router.device)
    if mx_weights is not None:
        a.W_gate_up_codes, a.W_gate_up_scales = mx_weights.gate_up_codes.data_ptr(), mx_weights.gate_up_scales.data_ptr()
        a.W_down_codes, a.W_down_scales = mx_weights.down_codes.data_ptr(), mx_weights.down_scales.data_ptr()
    _check(_lib.mok_moe_forward_host(ctypes.byref(a), ctypes.c_void_p(x_host.data_ptr()),
                                     ctypes.c_void_p(out_host.data_ptr())))
    return out_host


def mok_moe_forward_host_async(x_host, out_host, W_router, router_bias, W_gate_up, W_down, W_shared_gate_up,
                               W_shared_down, k, workspace, config=None, stream=None, mx_weights=None):
    """Submission without waiting (workspace from alloc_workspace(..., host_staging=2)); out_host is valid after
    mok_host_wait()."""
    assert not x_host.is_cuda and not out_host.is_cuda
    a, _ = _fill_args(x_host.shape, W_router, router_bias, W_gate_up, W_down, W_shared_gate_up, W_shared_down, k,
                      workspace, False, config, stream, W_router.device)
    if mx_weights is not None:
        a.W_gate_up_codes, a.W_gate_up_scales = mx_weights.gate_up_codes.data_ptr(), mx_weights.gate_up_scales.data_ptr()
        a.W_down_codes, a.W_down_scales = mx_weights.down_codes.data_ptr(), mx_weights.down_scales.data_ptr()
    _check(_lib.mok_moe_forward_host_async(ctypes.byref(a), ctypes.c_void_p(x_host.data_ptr()),
                                           ctypes.c_void_p(out_host.data_ptr())))


def mok_host_wait():
    _check(_lib.mok_host_wait())


def mok_route(x, W_router, router_bias, k, workspace, config=None, stream=None):
    T, H = x.shape
    E = W_router.shape[0]
    idx = torch.empty((T, k), dtype=torch.int32, device=x.device)
    w = torch.empty((T, k), dtype=torch.float32, device=x.device)
    wp, wn = _aligned_ws(workspace)
    _check(_lib.mok_route(_p(x), _p(W_router), _p(router_bias), T, H, E, k, _p(idx), _p(w), wp, wn,
                          None if config is None else ctypes.pointer(config), _stream(stream)))
    return idx, w


def mok_schedule(topk_idx, E, workspace, stream=None):
    T, k = topk_idx.shape
    dev = topk_idx.device
    counts = torch.empty((E,), dtype=torch.int32, device=dev)
    offsets = torch.empty((E + 1,), dtype=torch.int32, device=dev)
    perm = torch.empty((T * k,), dtype=torch.int32, device=dev)
    inv = torch.empty((T * k,), dtype=torch.int32, device=dev)
    wp, wn = _aligned_ws(workspace)
    _check(_lib.mok_schedule(_p(topk_idx), T, E, k, _p(counts), _p(offsets), _p(perm), _p(inv), wp, wn,
                             _stream(stream)))
    return counts, offsets, perm, inv


def mok_schedule_noalloc(topk_idx, E, stream=None):
    """mok_schedule for callers that cannot allocate device memory: the scratch is a fixed array inside the library
    (T*k <= MOK_NOALLOC_MAX_ROUTES).  The four result tensors are the caller's outputs, allocated here by torch only
    because this is the Python convenience wrapper; the C entry point itself allocates nothing."""
    T, k = topk_idx.shape
    dev = topk_idx.device
    counts = torch.empty((E,), dtype=torch.int32, device=dev)
    offsets = torch.empty((E + 1,), dtype=torch.int32, device=dev)
    perm = torch.empty((T * k,), dtype=torch.int32, device=dev)
    inv = torch.empty((T * k,), dtype=torch.int32, device=dev)
    _check(_lib.mok_schedule_noalloc(_p(topk_idx), T, E, k, _p(counts), _p(offsets), _p(perm), _p(inv),
                                     _stream(stream)))
    return counts, offsets, perm, inv


def mok_ep_workspace_bytes(n_ranks, T_local, H, I, I_shared, E, k):
    return int(_lib.mok_ep_workspace_bytes(n_ranks, T_local, H, I, I_shared, E, k))


def mok_ep_mx_workspace_bytes(n_ranks, T_local, H, I, I_shared, E, k):
    return int(_lib.mok_ep_mx_workspace_bytes(n_ranks, T_local, H, I, I_shared, E, k))


def mok_ep_y_rows(n_ranks, T_local, E, k):
    return int(_lib.mok_ep_y_rows(n_ranks, T_local, E, k))


def mok_ep_expert_ffn(rank, x_peer_ptrs, idx_all, W_gate_up, W_down, W_shared_gate_up, W_shared_down, E, k, y, pos,
                      y_shared, workspace, H, schedule_only=False, outputs=False, config=None, stream=None,
                      mx_weights=None, x_codes_ptrs=None, x_scales_ptrs=None):
    """Algorithm 1 for `rank` from the gathered routes idx_all [n_ranks, T_local*k], then this rank's expert FFNs with
    the rows pulled from x_peer_ptrs (device addresses, one per rank).  Fills y, pos (and y_shared).  With
    outputs=True also returns Algorithm 1's tables {M, S, phi_rank, phi_index}."""
    n_ranks, n = idx_all.shape
    T_local = n // k
    a = mok_ep_args()
    a.rank, a.n_ranks, a.T_local, a.H, a.E, a.k = rank, n_ranks, T_local, H, E, k
    a.I = 8 if W_gate_up is None else W_gate_up.shape[1] // 2
    a.I_shared = 0 if W_shared_gate_up is None else W_shared_gate_up.shape[0] // 2
    for r, ptr in enumerate(x_peer_ptrs or []):
        a.x_peers[r] = ptr
    a.idx_all = idx_all.data_ptr()
    for name, t in (("W_gate_up", W_gate_up), ("W_down", W_down), ("W_shared_gate_up", W_shared_gate_up),
                    ("W_shared_down", W_shared_down), ("y", y), ("pos", pos), ("y_shared", y_shared)):
        setattr(a, name, None if t is None else t.data_ptr())
    a.y_rows = 0 if y is None else y.shape[0]
    a.workspace, a.workspace_bytes = _aligned_ws(workspace)
    res = {}
    if outputs:
        L = E // n_ranks
        dev = idx_all.device
        res = {"M": torch.empty((n_ranks, L), dtype=torch.int32, device=dev),
               "S": torch.empty((L + 1,), dtype=torch.int32, device=dev),
               "phi_rank": torch.full((n_ranks * n,), -1, dtype=torch.int32, device=dev),
               "phi_index": torch.full((n_ranks * n,), -1, dtype=torch.int32, device=dev)}
        for name, t in res.items():
            setattr(a, name, t.data_ptr())
    a.schedule_only = int(schedule_only)
    if config is not None:
        a.config = ctypes.pointer(config)
    if mx_weights is not None:      # MXFP8 mode: this rank's pre-quantised experts and every rank's quantised token rows
        a.I = mx_weights.gate_up_codes.shape[1]
        a.W_gate_up_codes, a.W_gate_up_scales = mx_weights.gate_up_codes.data_ptr(), mx_weights.gate_up_scales.data_ptr()
        a.W_down_codes, a.W_down_scales = mx_weights.down_codes.data_ptr(), mx_weights.down_scales.data_ptr()
        for r in range(n_ranks):
            a.x_codes_peers[r] = x_codes_ptrs[r]
            a.x_scales_peers[r] = x_scales_ptrs[r]
    a.stream = _stream(stream).value
    _check(_lib.mok_ep_expert_ffn(ctypes.byref(a)))
    return res


def mok_ep_combine(rank, n_ranks, topk_idx, topk_w, y_peer_ptrs, pos_peer_ptrs, y_shared, E, out, stream=None):
    """Owner-side deterministic combine: out[t] = y_shared[t] + sum_s w[t,s] * (row of the serving rank's y)."""
    a = mok_ep_combine_args()
    a.rank, a.n_ranks = rank, n_ranks
    a.T_local, a.k = topk_idx.shape
    a.H, a.E = out.shape[1], E
    a.topk_idx, a.topk_w = topk_idx.data_ptr(), topk_w.data_ptr()
    for r in range(n_ranks):
        a.y_peers[r] = y_peer_ptrs[r]
        a.pos_peers[r] = pos_peer_ptrs[r]
    a.y_shared = None if y_shared is None else y_shared.data_ptr()
    a.out = out.data_ptr()
    a.stream = _stream(stream).value
    _check(_lib.mok_ep_combine(ctypes.byref(a)))
    return out


def mok_ep_bwd_workspace_bytes(n_ranks, T_local, H, I, I_shared, E, k):
    return int(_lib.mok_ep_bwd_workspace_bytes(n_ranks, T_local, H, I, I_shared, E, k))


def mok_ep_expert_bwd(rank, x_peer_ptrs, dout_peer_ptrs, idx_all, w_all, W_gate_up, W_down, W_shared_gate_up,
                      W_shared_down, E, k, H, dxg, pos, dw_routes, dx_shared, workspace, weight_grads=True, config=None,
                      stream=None):
    """Backward chain of one expert-parallel rank on the rows it serves (see include/mok.h).  idx_all / w_all:
    [n_ranks, T_local*k] all-gathered routes and router weights.  Fills dxg, pos, dw_routes (and dx_shared); returns
    the local weight gradients {dW_gate_up, dW_down (, dW_shared_gate_up, dW_shared_down)} when weight_grads."""
    n_ranks, n = idx_all.shape
    a = mok_ep_bwd_args()
    a.rank, a.n_ranks, a.T_local, a.H, a.E, a.k = rank, n_ranks, n // k, H, E, k
    a.I = W_gate_up.shape[1] // 2
    a.I_shared = 0 if W_shared_gate_up is None else W_shared_gate_up.shape[0] // 2
    for r in range(n_ranks):
        a.x_peers[r] = x_peer_ptrs[r]
        a.dout_peers[r] = dout_peer_ptrs[r]
    a.idx_all, a.w_all = idx_all.data_ptr(), w_all.data_ptr()
    a.W_gate_up, a.W_down = W_gate_up.data_ptr(), W_down.data_ptr()
    a.W_shared_gate_up = None if W_shared_gate_up is None else W_shared_gate_up.data_ptr()
    a.W_shared_down = None if W_shared_down is None else W_shared_down.data_ptr()
    a.dxg, a.dxg_rows, a.pos, a.dw_routes = dxg.data_ptr(), dxg.shape[0], pos.data_ptr(), dw_routes.data_ptr()
    a.dx_shared = None if dx_shared is None else dx_shared.data_ptr()
    res = {}
    if weight_grads:
        res["dW_gate_up"] = torch.empty_like(W_gate_up)
        res["dW_down"] = torch.empty_like(W_down)
        if a.I_shared:
            res["dW_shared_gate_up"] = torch.empty_like(W_shared_gate_up)
            res["dW_shared_down"] = torch.empty_like(W_shared_down)
    for name, t in res.items():
        setattr(a, name, t.data_ptr())
    a.workspace, a.workspace_bytes = _aligned_ws(workspace)
    if config is not None:
        a.config = ctypes.pointer(config)
    a.stream = _stream(stream).value
    _check(_lib.mok_ep_expert_bwd(ctypes.byref(a)))
    return res


def mok_ep_bwd_combine(rank, n_ranks, topk_idx, dxg_peer_ptrs, pos_peer_ptrs, dw_peer_ptrs, dx_shared, E, dx, dw=None,
                       stream=None):
    """Owner side of the expert-parallel backward: dx[t] = dx_shared[t] + sum_s (row of the serving rank's dxg), and dw."""
    a = mok_ep_bwd_combine_args()
    a.rank, a.n_ranks = rank, n_ranks
    a.T_local, a.k = topk_idx.shape
    a.H, a.E = dx.shape[1], E
    a.topk_idx = topk_idx.data_ptr()
    for r in range(n_ranks):
        a.dxg_peers[r] = dxg_peer_ptrs[r]
        a.pos_peers[r] = pos_peer_ptrs[r]
        a.dw_peers[r] = None if dw_peer_ptrs is None else dw_peer_ptrs[r]
    a.dx_shared = None if dx_shared is None else dx_shared.data_ptr()
    a.dx = dx.data_ptr()
    a.dw = None if dw is None else dw.data_ptr()
    a.stream = _stream(stream).value
    _check(_lib.mok_ep_bwd_combine(ctypes.byref(a)))
    return dx, dw


def mok_bwd_workspace_bytes(T, H, I, I_shared, E, k):
    return int(_lib.mok_bwd_workspace_bytes(T, H, I, I_shared, E, k))


def mok_moe_backward(x, W_gate_up, W_down, W_shared_gate_up, W_shared_down, topk_idx, topk_w, dout, workspace=None,
                     weight_grads=True, config=None, stream=None):
    """Backward pass from the forward inputs, its routing and dout.  Returns a dict: dx (bf16 [T,H]), dw (fp32 [T,k])
    and, with weight_grads, dW_gate_up, dW_down (and dW_shared_gate_up, dW_shared_down) in bf16."""
    T, H = x.shape
    E, twoI, _ = W_gate_up.shape
    I = twoI // 2
    I_s = 0 if W_shared_gate_up is None else W_shared_gate_up.shape[0] // 2
    k = topk_idx.shape[1]
    if workspace is None:
        n = mok_bwd_workspace_bytes(T, H, I, I_s, E, k)
        if n == 0:
            raise MokError(MOK_ERR_SHAPE)
        workspace = torch.empty(n + 256, dtype=torch.uint8, device=x.device)
    a = mok_bwd_args()
    a.x, a.W_gate_up, a.W_down = x.data_ptr(), W_gate_up.data_ptr(), W_down.data_ptr()
    a.W_shared_gate_up = None if W_shared_gate_up is None else W_shared_gate_up.data_ptr()
    a.W_shared_down = None if W_shared_down is None else W_shared_down.data_ptr()
    a.T, a.H, a.I, a.I_shared, a.E, a.k = T, H, I, I_s, E, k
    a.topk_idx, a.topk_w, a.dout = topk_idx.data_ptr(), topk_w.data_ptr(), dout.data_ptr()
    res = {"dx": torch.empty_like(x), "dw": torch.empty((T, k), dtype=torch.float32, device=x.device)}
    if weight_grads:
        res["dW_gate_up"] = torch.empty_like(W_gate_up)
        res["dW_down"] = torch.empty_like(W_down)
        if I_s:
            res["dW_shared_gate_up"] = torch.empty_like(W_shared_gate_up)
            res["dW_shared_down"] = torch.empty_like(W_shared_down)
    for name, t in res.items():
        setattr(a, name, t.data_ptr())
    a.workspace, a.workspace_bytes = _aligned_ws(workspace)
    if config is not None:
        a.config = ctypes.pointer(config)
    a.stream = _stream(stream).value
    _check(_lib.mok_moe_backward(ctypes.byref(a)))
    res["workspace"] = workspace
    return res


DEBUG_COUNTERS = ["mma_wait_operands", "mma_wait_peer_operands", "mma_wait_accumulator", "mma_total", "k_blocks",
                  "producer_wait_stage", "epilogue_wait_accumulator", "epilogue_total", "mma_total_max_cta",
                  "mma_total_ns", "valid_rows_x_k_blocks", "ctas"]


def mok_debug_counters(workspace, stream=None):
    """{slot: {counter: cycles}} of the last forward call that ran with config.debug != 0."""
    n = len(DEBUG_COUNTERS)
    buf = (ctypes.c_ulonglong * (4 * n))()
    wp, _ = _aligned_ws(workspace)
    _check(_lib.mok_debug_counters(wp, _stream(stream), buf))
    names = {0: "fused", 1: "gemm1", 2: "gemm2", 3: "shared"}
    return {names[s]: {c: int(buf[s * n + i]) for i, c in enumerate(DEBUG_COUNTERS)} for s in names}


def mok_read_status(workspace, stream=None):
    wp, _ = _aligned_ws(workspace)
    return int(_lib.mok_read_status(wp, _stream(stream)))


def to_device_bf16(bits, device="cuda"):
    """numpy uint16 bf16 bit patterns -> torch bf16 tensor on the device (a byte copy, no arithmetic)."""
    import numpy as np
    return torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)
