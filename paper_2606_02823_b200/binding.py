"""ctypes binding of libqift.so: the same entry points as include/qift.h, taking torch CUDA tensors.

Argument marshalling only -- every step of the layer runs in the library's CUDA kernels.  torch is
used for device memory and the current stream.  There is no CPU fallback: if the shared library is
missing, loading raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libqift.so")

# enums of qift.h
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED_SHAPE, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_TOO_LARGE = range(8)
MNZ, POT, SYM, INT4, INT3 = 0, 1, 2, 3, 4
SCALE_GIVEN, SCALE_ABSMAX, SCALE_MSE = 0, 1, 2
F32, BF16 = 0, 1
ROUTE_AUTO, ROUTE_GENERIC, ROUTE_DECODE, ROUTE_PREFILL, ROUTE_PREFILL_SCRATCH, ROUTE_PREFILL_PAIR = 0, 1, 2, 3, 4, 5
ROUTE_PREFILL_FUSED_PAIR = 6
ROUTE_DECODE_ROWS = 7

EXPORTS = [
    "qift_status_string", "qift_packed_bytes", "qift_workspace_bytes", "qift_workspace_bytes_route", "qift_pack_weights",
    "qift_unpack_codes", "qift_rotate", "qift_quantize_act", "qift_w2a4_linear", "qift_w4a4_linear",
    "qift_w3a4_linear", "qift_linear_route", "qift_device_status", "qift_forward_scratch_bytes", "qift_forward", "qift_forward_host",
    "qift_group_plan_bytes", "qift_group_plan", "qift_group_quantize_act", "qift_group_linear", "qift_group_forward",
    "qift_group_forward_host", "qift_static_scratch_bytes", "qift_w2a4_linear_static",
    "qift_kv4_quantize", "qift_kv4_attention_workspace_bytes", "qift_kv4_attention_decode",
    "qift_expand_weights", "qift_expanded_linear",
    "qift_diag_grid_quantize", "qift_diag_bucket_stats", "qift_diag_ratio_scan_workspace_bytes", "qift_diag_ratio_scan",
    "qift_selftest_wait_timeout", "qift_levels_bytes", "qift_forward_multi_scratch_bytes", "qift_forward_multi",
    "qift_linear_multi_workspace_bytes", "qift_linear_multi", "qift_calib_hbm_read", "qift_calib_mma_i8",
]

_lib = None


class QiftError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (qift_status {status})")


def lib() -> ctypes.CDLL:
    """Loads libqift.so; raises if it has not been built (python -m paper_2606_02823_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2606_02823_b200.build` "
                "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, ci, cf, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
        L.qift_status_string.restype = ctypes.c_char_p
        L.qift_status_string.argtypes = [ci]
        L.qift_packed_bytes.restype = sz
        L.qift_packed_bytes.argtypes = [ci, ci, ci]
        L.qift_workspace_bytes.restype = sz
        L.qift_workspace_bytes.argtypes = [ci, ci, ci, ci]
        L.qift_workspace_bytes_route.restype = sz
        L.qift_workspace_bytes_route.argtypes = [ci, ci, ci, ci, ci]
        L.qift_pack_weights.argtypes = [vp, ci, ci, ci, ci, vp, vp, vp]
        L.qift_unpack_codes.argtypes = [vp, ci, ci, ci, vp, vp]
        L.qift_rotate.argtypes = [vp, ci, ci, ci, vp, vp]
        L.qift_quantize_act.argtypes = [vp, ci, ci, ci, ci, cf, vp, vp, vp]
        L.qift_w2a4_linear.argtypes = [vp, vp, ci, vp, vp, ci, ci, ci, vp, ci, vp, vp, sz, vp]
        L.qift_w4a4_linear.argtypes = [vp, vp, vp, vp, ci, ci, ci, vp, ci, vp, vp, sz, vp]
        L.qift_w3a4_linear.argtypes = [vp, vp, vp, vp, ci, ci, ci, vp, ci, vp, vp, sz, vp]
        L.qift_linear_route.argtypes = [vp, vp, ci, vp, vp, ci, ci, ci, vp, ci, vp, vp, sz, ci, vp]
        L.qift_device_status.argtypes = [vp, vp]
        L.qift_forward_scratch_bytes.restype = sz
        L.qift_forward_scratch_bytes.argtypes = [ci, ci, ci, ci, ci, ci]
        fwd = [vp, ci, ci, ci, ci, cf, vp, vp, ci, ci, vp, ci, vp, sz, vp]
        L.qift_forward.argtypes = fwd
        L.qift_forward_host.argtypes = fwd
        L.qift_group_plan_bytes.restype = sz
        L.qift_group_plan_bytes.argtypes = [ci]
        L.qift_group_plan.argtypes = [vp, ci, ci, ci, ci, ci, cf, vp, vp, sz, vp]
        for name in ("qift_group_quantize_act", "qift_group_linear", "qift_group_forward"):
            getattr(L, name).argtypes = [vp, vp, vp]
        L.qift_group_forward_host.argtypes = [vp, vp, vp, vp, sz, vp, vp, sz, vp]
        L.qift_static_scratch_bytes.restype = sz
        L.qift_static_scratch_bytes.argtypes = []
        L.qift_w2a4_linear_static.argtypes = [vp, vp, ci, vp, vp, ci, ci, ci, vp, ci, vp, vp]
        L.qift_expand_weights.argtypes = [vp, ci, ci, ci, vp, vp]
        L.qift_expanded_linear.argtypes = [vp, vp, vp, vp, ci, ci, ci, vp, ci, vp, vp]
        L.qift_kv4_quantize.argtypes = [vp, ci, ci, ci, ci, ci, cf, ci, ci, ci, vp, vp, vp, vp]
        L.qift_kv4_attention_workspace_bytes.restype = sz
        L.qift_kv4_attention_workspace_bytes.argtypes = [ci, ci, ci]
        L.qift_kv4_attention_decode.argtypes = [vp, vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, vp, vp, sz, vp]
        L.qift_diag_grid_quantize.argtypes = [vp, ci, ci, vp, ci, vp, vp, vp]
        L.qift_diag_bucket_stats.argtypes = [vp, vp, ci, ci, vp, vp, ci, vp, vp, vp]
        L.qift_diag_ratio_scan_workspace_bytes.restype = sz
        L.qift_diag_ratio_scan_workspace_bytes.argtypes = [ctypes.c_longlong, ci]
        L.qift_diag_ratio_scan.argtypes = [vp, ctypes.c_longlong, vp, ci, vp, vp, vp, sz, vp]
        L.qift_selftest_wait_timeout.argtypes = [ci, ctypes.c_uint, vp]
        L.qift_levels_bytes.restype = sz
        L.qift_levels_bytes.argtypes = [ci, vp, ci]
        L.qift_forward_multi_scratch_bytes.restype = sz
        L.qift_forward_multi_scratch_bytes.argtypes = [ci, ci, ci, vp, ci]
        L.qift_forward_multi.argtypes = [vp, ci, ci, ci, ci, cf, ci, vp, ci, ci, vp, sz, vp, sz, ci, vp, vp]
        L.qift_linear_multi_workspace_bytes.restype = sz
        L.qift_linear_multi_workspace_bytes.argtypes = [ci, ci, ci, vp, ci]
        L.qift_linear_multi.argtypes = [vp, vp, ci, ci, ci, vp, ci, ci, vp, sz, vp, sz, ci, vp, vp]
        L.qift_calib_hbm_read.argtypes = [vp, sz, vp, vp]
        L.qift_calib_mma_i8.argtypes = [ci, vp, vp]
        for name in EXPORTS:
            if name not in ("qift_diag_ratio_scan_workspace_bytes", "qift_status_string", "qift_packed_bytes", "qift_workspace_bytes",
                            "qift_forward_scratch_bytes", "qift_group_plan_bytes", "qift_static_scratch_bytes",
                            "qift_workspace_bytes_route", "qift_kv4_attention_workspace_bytes", "qift_levels_bytes",
                            "qift_forward_multi_scratch_bytes", "qift_linear_multi_workspace_bytes"):
                getattr(L, name).restype = ci
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().qift_status_string(int(status)).decode()


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(rc: int, where: str):
    if rc != OK:
        raise QiftError(rc, where)


def _dev(t, dtype=None):
    assert t.is_cuda and t.is_contiguous(), "expected a contiguous CUDA tensor"
    if dtype is not None:
        assert t.dtype == dtype, f"expected {dtype}, got {t.dtype}"
    return t


def qift_packed_bytes(N: int, K: int, levels: int) -> int:
    return int(lib().qift_packed_bytes(N, K, levels))


def qift_workspace_bytes(M: int, N: int, K: int, levels: int, route: int = ROUTE_AUTO) -> int:
    return int(lib().qift_workspace_bytes_route(M, N, K, levels, route))


def qift_pack_weights(W, levels: int, scale_mode: int, s_n=None, packed=None):
    """W fp32 [N,K] (already rotated) -> (packed: flat int32 buffer of qift_packed_bytes(N,K) bytes in
    the tiled storage order, s_n fp32 [N])."""
    _dev(W, torch.float32)
    N, K = W.shape
    if s_n is None:
        s_n = torch.empty(N, dtype=torch.float32, device=W.device)
    if packed is None:
        packed = torch.empty((max(qift_packed_bytes(N, K, levels) // 4, 1),), dtype=torch.int32, device=W.device)
    _check(lib().qift_pack_weights(_ptr(W), N, K, levels, scale_mode, _ptr(_dev(s_n, torch.float32)),
                                   _ptr(_dev(packed)), _stream()), "qift_pack_weights")
    return packed, s_n


def qift_unpack_codes(packed, N: int, K: int, levels: int):
    _dev(packed)
    codes = torch.empty((N, K), dtype=torch.uint8, device=packed.device)
    _check(lib().qift_unpack_codes(_ptr(packed), N, K, levels, _ptr(codes), _stream()), "qift_unpack_codes")
    return codes


def qift_rotate(X, had_block: int, out=None):
    _dev(X, torch.float32)
    M, K = X.shape
    if out is None:
        out = torch.empty_like(X)
    _check(lib().qift_rotate(_ptr(X), M, K, had_block, _ptr(_dev(out, torch.float32)), _stream()), "qift_rotate")
    return out


def qift_quantize_act(X, had_block: int, clip_ratio: float = 0.9, q_a=None, s_a=None):
    """X fp32 or bf16 [M,K] -> (q_a int8 [M,K], s_a fp32 [M])."""
    _dev(X)
    assert X.dtype in (torch.float32, torch.bfloat16)
    M, K = X.shape
    if q_a is None:
        q_a = torch.empty((M, K), dtype=torch.int8, device=X.device)
    if s_a is None:
        s_a = torch.empty((M,), dtype=torch.float32, device=X.device)
    _check(lib().qift_quantize_act(_ptr(X), F32 if X.dtype == torch.float32 else BF16, M, K, had_block,
                                   clip_ratio, _ptr(_dev(q_a, torch.int8)), _ptr(_dev(s_a, torch.float32)),
                                   _stream()), "qift_quantize_act")
    return q_a, s_a


def _linear(fn_name, packed, s_n, levels, q_a, s_a, N, out_dtype, want_acc, workspace, route, out):
    _dev(packed), _dev(s_n, torch.float32), _dev(q_a, torch.int8), _dev(s_a, torch.float32)
    M, K = q_a.shape
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=q_a.device)
    assert out.dtype in (torch.float32, torch.bfloat16)
    acc = torch.empty((M, N), dtype=torch.int32, device=q_a.device) if want_acc else None
    need = qift_workspace_bytes(M, N, K, levels, route)
    if workspace is None and need:
        workspace = torch.empty(need, dtype=torch.uint8, device=q_a.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    ydt = F32 if out.dtype == torch.float32 else BF16
    L = lib()
    if fn_name == "qift_linear_route":
        rc = L.qift_linear_route(_ptr(packed), _ptr(s_n), levels, _ptr(q_a), _ptr(s_a), M, N, K, _ptr(out), ydt,
                                 _ptr(acc), _ptr(workspace), ws_bytes, route, _stream())
    elif fn_name in ("qift_w4a4_linear", "qift_w3a4_linear"):
        rc = getattr(L, fn_name)(_ptr(packed), _ptr(s_n), _ptr(q_a), _ptr(s_a), M, N, K, _ptr(out), ydt, _ptr(acc),
                                 _ptr(workspace), ws_bytes, _stream())
    else:
        rc = L.qift_w2a4_linear(_ptr(packed), _ptr(s_n), levels, _ptr(q_a), _ptr(s_a), M, N, K, _ptr(out), ydt,
                                _ptr(acc), _ptr(workspace), ws_bytes, _stream())
    _check(rc, fn_name)
    return (out, acc) if want_acc else out


def qift_w2a4_linear(packed, s_n, levels, q_a, s_a, out_dtype=torch.float32, want_acc=False, workspace=None, out=None):
    """N is the length of s_n."""
    return _linear("qift_w2a4_linear", packed, s_n, levels, q_a, s_a, s_n.shape[0], out_dtype, want_acc,
                   workspace, ROUTE_AUTO, out)


def qift_w4a4_linear(packed, s_n, q_a, s_a, out_dtype=torch.float32, want_acc=False, workspace=None, out=None):
    return _linear("qift_w4a4_linear", packed, s_n, INT4, q_a, s_a, s_n.shape[0], out_dtype, want_acc,
                   workspace, ROUTE_AUTO, out)


def qift_w3a4_linear(packed, s_n, q_a, s_a, out_dtype=torch.float32, want_acc=False, workspace=None, out=None):
    return _linear("qift_w3a4_linear", packed, s_n, INT3, q_a, s_a, s_n.shape[0], out_dtype, want_acc,
                   workspace, ROUTE_AUTO, out)


def qift_linear_route(packed, s_n, levels, q_a, s_a, route, out_dtype=torch.float32, want_acc=False, workspace=None,
                      out=None):
    return _linear("qift_linear_route", packed, s_n, levels, q_a, s_a, s_n.shape[0], out_dtype, want_acc,
                   workspace, route, out)


def qift_device_status():
    """Synchronizes the current stream; returns (status, detail word)."""
    detail = ctypes.c_uint32(0)
    rc = lib().qift_device_status(_stream(), ctypes.byref(detail))
    return rc, detail.value


def qift_selftest_wait_timeout(which: int, limit_us: int):
    """Enqueues a kernel whose bounded wait runs out after limit_us (0: a lone waiting CTA; 1: the CTA-pair
    prefill GEMM starved of its loads); qift_device_status() then reports ERR_TIMEOUT once."""
    _check(lib().qift_selftest_wait_timeout(which, limit_us, _stream()), "qift_selftest_wait_timeout")


def _dt(t):
    assert t.dtype in (torch.float32, torch.bfloat16)
    return F32 if t.dtype == torch.float32 else BF16


def qift_forward_scratch_bytes(M: int, N: int, K: int, levels: int, x_dtype: int = F32, y_dtype: int = F32) -> int:
    return int(lib().qift_forward_scratch_bytes(M, N, K, levels, x_dtype, y_dtype))


def _forward(fn, X, had_block, clip_ratio, packed, s_n, levels, out, scratch):
    M, K = X.shape
    N = s_n.shape[0]
    need = qift_forward_scratch_bytes(M, N, K, levels, _dt(X), _dt(out))
    if scratch is None:
        scratch = torch.empty(need, dtype=torch.uint8, device=packed.device)
    _check(fn(_ptr(X), _dt(X), M, K, had_block, clip_ratio, _ptr(_dev(packed)), _ptr(_dev(s_n, torch.float32)), levels, N,
              _ptr(out), _dt(out), _ptr(_dev(scratch)), scratch.numel(), _stream()), "qift_forward")
    return out


def qift_forward(X, had_block, packed, s_n, levels, clip_ratio: float = 0.9, out_dtype=torch.float32, out=None,
                 scratch=None):
    """Whole layer on device tensors: rotate + quantize X [M,K], multiply, scale -> Y [M,N]."""
    _dev(X)
    if out is None:
        out = torch.empty((X.shape[0], s_n.shape[0]), dtype=out_dtype, device=X.device)
    return _forward(lib().qift_forward, X, had_block, clip_ratio, packed, s_n, levels, out, scratch)


def qift_forward_host(X_host, had_block, packed, s_n, levels, out_host, clip_ratio: float = 0.9, scratch=None):
    """Whole layer with X and Y in (pinned) host tensors; Y is valid after the stream is synchronized."""
    assert not X_host.is_cuda and not out_host.is_cuda and X_host.is_contiguous() and out_host.is_contiguous()
    return _forward(lib().qift_forward_host, X_host, had_block, clip_ratio, packed, s_n, levels, out_host, scratch)


class LinearOutput(ctypes.Structure):
    """Mirror of qift_linear_output."""
    _fields_ = [("packed", ctypes.c_void_p), ("s_n", ctypes.c_void_p), ("Y", ctypes.c_void_p), ("acc_debug", ctypes.c_void_p),
                ("N", ctypes.c_int), ("reserved", ctypes.c_int)]


class DecodeAhead(ctypes.Structure):
    """Mirror of qift_decode_ahead."""
    _fields_ = [("outputs", ctypes.c_void_p), ("count", ctypes.c_int), ("K", ctypes.c_int), ("levels", ctypes.c_int),
                ("reserved", ctypes.c_int), ("levels_buf", ctypes.c_void_p), ("levels_bytes", ctypes.c_size_t),
                ("next", ctypes.c_void_p)]


def _ahead_chain(ahead):
    """ahead: one (weights, K, levels, levels_buf) tuple or a list of them -> (address of the first descriptor or None,
    objects to keep alive)."""
    if ahead is None:
        return None, None
    items = ahead if isinstance(ahead, list) else [ahead]
    keep, nxt = [], None
    for nw, nK, nlv, nbuf in reversed(items):
        arr = _outputs_array(nw)
        d = DecodeAhead(ctypes.addressof(arr), len(nw), nK, nlv, 0, _dev(nbuf).data_ptr(), nbuf.numel(), nxt)
        keep += [arr, d]
        nxt = ctypes.addressof(d)
    return nxt, keep


def _outputs_array(weights, ys=None, accs=None):
    """weights: list of (packed, s_n) -> ctypes array of qift_linear_output (Y / acc filled when given)."""
    arr = (LinearOutput * len(weights))()
    for i, (packed, s_n) in enumerate(weights):
        arr[i] = LinearOutput(_dev(packed).data_ptr(), _dev(s_n, torch.float32).data_ptr(),
                              None if ys is None else ys[i].data_ptr(),
                              None if accs is None or accs[i] is None else accs[i].data_ptr(), s_n.shape[0], 0)
    return arr


def qift_levels_bytes(K: int, weights) -> int:
    """Bytes of the int8 levels buffer for a list of (packed, s_n) weights sharing K."""
    arr = _outputs_array(weights)
    return int(lib().qift_levels_bytes(K, ctypes.addressof(arr), len(weights)))


def qift_forward_multi(X, had_block: int, weights, levels: int, clip_ratio: float = 0.9, out_dtype=torch.float32,
                       want_acc: bool = False, scratch=None, levels_buf=None, levels_ready: bool = False, ahead=None, outs=None):
    """One activation X [M,K], several products: weights = [(packed, s_n), ...] (1..4) -> ([Y_i [M,N_i]], [acc_i or None]).
    levels_buf: uint8 tensor of qift_levels_bytes(K, weights) bytes (allocated when omitted; needed for M > 128);
    levels_ready: it already holds these weights' decoded levels (written through a previous call's `ahead`);
    ahead = (next_weights, next_K, next_levels, next_levels_buf), or a list of such tuples: decode later calls' codes
    during this one."""
    _dev(X)
    M, K = X.shape
    ys = outs if outs is not None else [torch.empty((M, s_n.shape[0]), dtype=out_dtype, device=X.device) for _, s_n in weights]
    accs = [torch.empty((M, s_n.shape[0]), dtype=torch.int32, device=X.device) if want_acc else None for _, s_n in weights]
    arr = _outputs_array(weights, ys, accs)
    L = lib()
    need = int(L.qift_forward_multi_scratch_bytes(M, K, levels, ctypes.addressof(arr), len(weights)))
    if scratch is None:
        scratch = torch.empty(max(need, 256), dtype=torch.uint8, device=X.device)
    if levels_buf is None:
        assert not levels_ready
        levels_buf = torch.empty(max(qift_levels_bytes(K, weights), 256), dtype=torch.uint8, device=X.device)
    ah, keep = _ahead_chain(ahead)
    _check(L.qift_forward_multi(_ptr(X), _dt(X), M, K, had_block, clip_ratio, levels, ctypes.addressof(arr), len(weights),
                                _dt(ys[0]), _ptr(_dev(scratch)), scratch.numel(), _ptr(_dev(levels_buf)), levels_buf.numel(),
                                1 if levels_ready else 0, ah, _stream()),
           "qift_forward_multi")
    return ys, accs


def qift_linear_multi(q_a, s_a, weights, levels: int, out_dtype=torch.float32, want_acc: bool = False, levels_buf=None,
                      levels_ready: bool = False, ahead=None):
    """The product part of qift_forward_multi on an activation that is already quantized -> ([Y_i], [acc_i or None])."""
    _dev(q_a, torch.int8), _dev(s_a, torch.float32)
    M, K = q_a.shape
    ys = [torch.empty((M, s_n.shape[0]), dtype=out_dtype, device=q_a.device) for _, s_n in weights]
    accs = [torch.empty((M, s_n.shape[0]), dtype=torch.int32, device=q_a.device) if want_acc else None for _, s_n in weights]
    arr = _outputs_array(weights, ys, accs)
    L = lib()
    need = int(L.qift_linear_multi_workspace_bytes(M, K, levels, ctypes.addressof(arr), len(weights)))
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device=q_a.device)
    if levels_buf is None:
        assert not levels_ready
        levels_buf = torch.empty(max(qift_levels_bytes(K, weights), 256), dtype=torch.uint8, device=q_a.device)
    ah, keep = _ahead_chain(ahead)
    _check(L.qift_linear_multi(_ptr(q_a), _ptr(s_a), M, K, levels, ctypes.addressof(arr), len(weights), _dt(ys[0]), _ptr(ws),
                               ws.numel(), _ptr(_dev(levels_buf)), levels_buf.numel(), 1 if levels_ready else 0,
                               ah, _stream()), "qift_linear_multi")
    return ys, accs


class GroupProblem(ctypes.Structure):
    """Mirror of qift_group_problem."""
    _fields_ = [("X", ctypes.c_void_p), ("packed", ctypes.c_void_p), ("s_n", ctypes.c_void_p), ("q_a", ctypes.c_void_p),
                ("s_a", ctypes.c_void_p), ("Y", ctypes.c_void_p), ("acc_debug", ctypes.c_void_p), ("N", ctypes.c_int),
                ("K", ctypes.c_int), ("had_block", ctypes.c_int), ("reserved", ctypes.c_int)]


class GroupPlan:
    """A validated problem list: host and device copies of the plan plus references that keep every
    tensor named in it alive.  `outputs[i]` / `accs[i]` are the results of problem i; `inputs[i]` is
    its activation tensor (a view into the X arena when the plan owns the inputs)."""

    def __init__(self, host, dev, keep, inputs, outputs, accs, x_arena=None, y_arena=None):
        self.host, self.dev, self.keep, self.inputs, self.outputs, self.accs = host, dev, keep, inputs, outputs, accs
        self.x_arena, self.y_arena = x_arena, y_arena
        self.x_host = self.y_host = None


def qift_group_plan_bytes(count: int) -> int:
    return int(lib().qift_group_plan_bytes(count))


def _align(n, a=256):
    return (n + a - 1) // a * a


def qift_group_plan(problems, levels: int, clip_ratio: float = 0.9, out_dtype=torch.float32, want_acc: bool = False,
                    arenas: bool = False, share: bool = True):
    """problems: list of (X [M,K], packed, s_n, had_block) sharing M and the dtype of X.  Allocates
    q_a / s_a / Y (and the accumulators when asked) and returns a GroupPlan.  Problems that name the same X tensor
    (and rotation) get the same q_a / s_a, which the library then quantizes once (share=False: one each).  With arenas=True the
    activations are copied into one contiguous device arena and the outputs live in another, each
    with a pinned host mirror (plan.x_host / plan.y_host), for qift_group_forward_host."""
    assert problems
    M = problems[0][0].shape[0]
    xdt = _dt(problems[0][0])
    device = problems[0][0].device
    arr = (GroupProblem * len(problems))()
    keep, ins, outs, accs = [], [], [], []
    shared = {}
    x_arena = y_arena = None
    if arenas:
        xe = problems[0][0].element_size()
        ye = torch.empty(0, dtype=out_dtype).element_size()
        xo, yo, x_off, y_off = 0, 0, [], []
        for (X, packed, s_n, had_block) in problems:
            x_off.append(xo), y_off.append(yo)
            xo += _align(M * X.shape[1] * xe)
            yo += _align(M * s_n.shape[0] * ye)
        x_arena = torch.zeros(xo, dtype=torch.uint8, device=device)
        y_arena = torch.zeros(yo, dtype=torch.uint8, device=device)
    for i, (X, packed, s_n, had_block) in enumerate(problems):
        _dev(X), _dev(packed), _dev(s_n, torch.float32)
        assert X.shape[0] == M and _dt(X) == xdt
        K, N = X.shape[1], s_n.shape[0]
        if arenas:
            xv = x_arena[x_off[i]:x_off[i] + M * K * xe].view(X.dtype).view(M, K)
            xv.copy_(X)
            X = xv
            Y = y_arena[y_off[i]:y_off[i] + M * N * ye].view(out_dtype).view(M, N)
        else:
            Y = torch.empty((M, N), dtype=out_dtype, device=device)
        key = (X.data_ptr(), K, had_block)
        if share and not arenas and key in shared:      # modules reading one activation share its quantization
            q_a, s_a = shared[key]
        else:
            q_a = torch.empty((M, K), dtype=torch.int8, device=device)
            s_a = torch.empty((max(M, 4),), dtype=torch.float32, device=device)
            shared[key] = (q_a, s_a)
        acc = torch.empty((M, N), dtype=torch.int32, device=device) if want_acc else None
        arr[i] = GroupProblem(X.data_ptr(), packed.data_ptr(), s_n.data_ptr(), q_a.data_ptr(), s_a.data_ptr(), Y.data_ptr(),
                              acc.data_ptr() if want_acc else None, N, K, had_block, 0)
        keep += [X, packed, s_n, q_a, s_a]
        ins.append(X)
        outs.append(Y)
        accs.append(acc)
    nbytes = qift_group_plan_bytes(len(problems))
    host = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
    dev = torch.empty(nbytes, dtype=torch.uint8, device=device)
    ydt = F32 if out_dtype == torch.float32 else BF16
    _check(lib().qift_group_plan(ctypes.addressof(arr), len(problems), M, levels, xdt, ydt, clip_ratio, host.data_ptr(),
                                 dev.data_ptr(), nbytes, _stream()), "qift_group_plan")
    plan = GroupPlan(host, dev, keep, ins, outs, accs, x_arena, y_arena)
    if arenas:
        plan.x_host = x_arena.cpu().pin_memory()
        plan.y_host = torch.empty(y_arena.shape, dtype=torch.uint8).pin_memory()
    return plan


def qift_group_quantize_act(plan: GroupPlan):
    _check(lib().qift_group_quantize_act(plan.host.data_ptr(), plan.dev.data_ptr(), _stream()), "qift_group_quantize_act")


def qift_group_linear(plan: GroupPlan):
    _check(lib().qift_group_linear(plan.host.data_ptr(), plan.dev.data_ptr(), _stream()), "qift_group_linear")


def qift_group_forward(plan: GroupPlan):
    _check(lib().qift_group_forward(plan.host.data_ptr(), plan.dev.data_ptr(), _stream()), "qift_group_forward")
    return plan.outputs


def qift_static_scratch_bytes() -> int:
    return int(lib().qift_static_scratch_bytes())


def qift_w2a4_linear_static(packed, s_n, levels, q_a, s_a, out, acc=None):
    """The W2A4 product for callers that cannot allocate: the int8 scratch of the prefill route comes
    from an array built into the library, and the caller passes every output buffer (`out` [M,N]
    fp32 or bf16, optionally `acc` int32 [M,N]).  This wrapper allocates nothing either.  Calls that
    may overlap on the GPU share the scratch and must be serialized; make the first call on a device
    outside stream capture."""
    _dev(packed), _dev(s_n, torch.float32), _dev(q_a, torch.int8), _dev(s_a, torch.float32), _dev(out)
    M, K = q_a.shape
    N = s_n.shape[0]
    assert tuple(out.shape) == (M, N)
    _check(lib().qift_w2a4_linear_static(_ptr(packed), _ptr(s_n), levels, _ptr(q_a), _ptr(s_a), M, N, K, _ptr(out),
                                         _dt(out), _ptr(acc), _stream()), "qift_w2a4_linear_static")
    return out


def qift_group_forward_host(plan: GroupPlan):
    """The grouped layer with activations read from plan.x_host and results written to plan.y_host
    (pinned host arenas laid out like the device arenas); valid after the stream is synchronized."""
    assert plan.x_arena is not None, "build the plan with arenas=True"
    _check(lib().qift_group_forward_host(plan.host.data_ptr(), plan.dev.data_ptr(), plan.x_host.data_ptr(),
                                         plan.x_arena.data_ptr(), plan.x_arena.numel(), plan.y_arena.data_ptr(),
                                         plan.y_host.data_ptr(), plan.y_arena.numel(), _stream()), "qift_group_forward_host")
    return plan.y_host


# ---------------------------------------------------------------------------------------- KV4
KV_KEYS, KV_VALUES = 0, 1


class Kv4Cache:
    """Device buffers of a 4-bit cache for keys (codes uint8 [H, T_cap, D/2], two dimensions per byte) or values
    (codes uint8 [H, T_cap/2, D], two tokens per byte); scale / zero fp32 [H, T_cap].  T_cap even."""

    def __init__(self, H: int, T_cap: int, layout: int = KV_KEYS, D: int = 128, device="cuda"):
        assert T_cap % 2 == 0
        self.H, self.T_cap, self.D, self.layout = H, T_cap, D, layout
        shape = (H, T_cap, D // 2) if layout == KV_KEYS else (H, T_cap // 2, D)
        self.codes = torch.zeros(shape, dtype=torch.uint8, device=device)
        self.scale = torch.zeros((H, T_cap), dtype=torch.float32, device=device)
        self.zero = torch.zeros((H, T_cap), dtype=torch.float32, device=device)


def qift_kv4_quantize(X, cache: Kv4Cache, t0: int = 0, had_block: int = 0, clip_ratio: float = 0.95):
    """X fp32 or bf16 [T, H, D] -> written into cache slots t0 .. t0+T-1."""
    _dev(X)
    assert X.dtype in (torch.float32, torch.bfloat16)
    T, H, D = X.shape
    _check(lib().qift_kv4_quantize(_ptr(X), F32 if X.dtype == torch.float32 else BF16, T, H, D, had_block, clip_ratio, t0,
                                   cache.T_cap, cache.layout, _ptr(cache.codes), _ptr(cache.scale), _ptr(cache.zero), _stream()),
           "qift_kv4_quantize")
    return cache


def qift_kv4_attention_workspace_bytes(T: int, Hq: int, Hkv: int) -> int:
    return int(lib().qift_kv4_attention_workspace_bytes(T, Hq, Hkv))


def qift_kv4_attention_decode(q, K: Kv4Cache, V: Kv4Cache, T: int, out=None, workspace=None):
    """q fp32 [Hq, D] -> out fp32 [Hq, D]: softmax(q K^T / sqrt(D)) V over the first T cached tokens."""
    _dev(q, torch.float32)
    Hq, D = q.shape
    if out is None:
        out = torch.empty((Hq, D), dtype=torch.float32, device=q.device)
    need = qift_kv4_attention_workspace_bytes(T, Hq, K.H)
    if workspace is None:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=q.device)
    _check(lib().qift_kv4_attention_decode(_ptr(q), _ptr(K.codes), _ptr(K.scale), _ptr(K.zero), _ptr(V.codes), _ptr(V.scale),
                                           _ptr(V.zero), T, K.T_cap, Hq, K.H, D, _ptr(_dev(out, torch.float32)),
                                           _ptr(workspace), workspace.numel(), _stream()), "qift_kv4_attention_decode")
    return out


# ---------------------------------------------------------------------------------------- resident decoded weights
def qift_expand_weights(packed, N: int, K: int, levels: int, out=None):
    """packed codes -> int8 levels [N, K] (kept resident for the prefill product)."""
    _dev(packed)
    if out is None:
        out = torch.empty((N, K), dtype=torch.int8, device=packed.device)
    _check(lib().qift_expand_weights(_ptr(packed), N, K, levels, _ptr(_dev(out, torch.int8)), _stream()), "qift_expand_weights")
    return out


def qift_expanded_linear(levels_i8, s_n, q_a, s_a, out_dtype=torch.float32, want_acc: bool = False, out=None):
    """The prefill product on resident decoded weights -> (Y [M, N], acc int32 [M, N] or None)."""
    _dev(levels_i8, torch.int8), _dev(s_n, torch.float32), _dev(q_a, torch.int8), _dev(s_a, torch.float32)
    N, K = levels_i8.shape
    M = q_a.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=q_a.device)
    acc = torch.empty((M, N), dtype=torch.int32, device=q_a.device) if want_acc else None
    _check(lib().qift_expanded_linear(_ptr(levels_i8), _ptr(s_n), _ptr(q_a), _ptr(s_a), M, N, K, _ptr(out),
                                      F32 if out.dtype == torch.float32 else BF16, _ptr(acc), _stream()), "qift_expanded_linear")
    return out, acc


# ------------------------------------------------------------------------------------------ quantizer diagnostics
def _host_array(values, ctype):
    values = [float(v) for v in values]
    return (ctype * len(values))(*values), len(values)


def qift_diag_grid_quantize(W, grid, scale_mode: int, s_n=None, want_codes: bool = True):
    """Nearest-level quantization onto four float levels -> (s_n fp32 [N], codes uint8 [N, K] or None)."""
    _dev(W, torch.float32)
    N, K = W.shape
    g, n = _host_array(grid, ctypes.c_float)
    if n != 4:
        raise ValueError("a grid has four levels")
    if s_n is None:
        if scale_mode == SCALE_GIVEN:
            raise ValueError("SCALE_GIVEN needs s_n")
        s_n = torch.empty((N,), dtype=torch.float32, device=W.device)
    codes = torch.empty((N, K), dtype=torch.uint8, device=W.device) if want_codes else None
    _check(lib().qift_diag_grid_quantize(_ptr(W), N, K, g, scale_mode, _ptr(_dev(s_n, torch.float32)), _ptr(codes), _stream()),
           "qift_diag_grid_quantize")
    return s_n, codes


def qift_diag_bucket_stats(W, codes, s_n, values):
    """-> (count int64 [L], sqerr fp64 [L]): weights and squared error per assigned level."""
    _dev(W, torch.float32), _dev(codes, torch.uint8), _dev(s_n, torch.float32)
    N, K = W.shape
    v, L = _host_array(values, ctypes.c_float)
    count = torch.empty((L,), dtype=torch.int64, device=W.device)
    sqerr = torch.empty((L,), dtype=torch.float64, device=W.device)
    _check(lib().qift_diag_bucket_stats(_ptr(W), _ptr(codes), N, K, _ptr(s_n), v, L, _ptr(count), _ptr(sqerr), _stream()),
           "qift_diag_bucket_stats")
    return count, sqerr


def qift_diag_ratio_scan_workspace_bytes(n: int, R: int) -> int:
    return int(lib().qift_diag_ratio_scan_workspace_bytes(int(n), int(R)))


def qift_diag_ratio_scan(x, ratios, workspace=None):
    """x fp32 [n] -> (beta fp64 [R], nmse fp64 [R]) for the grids {-1, -r, +r, +1}."""
    _dev(x, torch.float32)
    n = x.numel()
    r, R = _host_array(ratios, ctypes.c_double)
    need = qift_diag_ratio_scan_workspace_bytes(n, R)
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=x.device)
    beta = torch.empty((R,), dtype=torch.float64, device=x.device)
    nmse = torch.empty((R,), dtype=torch.float64, device=x.device)
    _check(lib().qift_diag_ratio_scan(_ptr(x), n, r, R, _ptr(beta), _ptr(nmse), _ptr(workspace), workspace.numel(), _stream()),
           "qift_diag_ratio_scan")
    return beta, nmse
