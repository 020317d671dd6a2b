"""ctypes binding of the C-ABI library (argument marshalling only).

Every function here has the name of the `extern "C"` entry point it forwards to.  Tensors
are torch CUDA tensors used purely as device memory; the current torch stream is passed as
the library's stream.  Nothing in this module computes: if the shared library is missing the
import of any entry point fails loudly, there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# CALIDROP_LIB selects another build of the same library (e.g. an instrumented one).
LIB_PATH = os.environ.get("CALIDROP_LIB") or os.path.join(_HERE, "libcalidrop.so")
_lib = None

OK, INVALID_ARG, UNSUPPORTED, WORKSPACE_TOO_SMALL, CUDA_ERROR, SCRATCH_LIMIT = 0, -1, -2, -3, -4, -5
STATIC_SCRATCH_BYTES = 4 << 20
MAX_LAYERS = 32

EXPORTS = [
    "calidrop_compress_workspace_bytes", "calidrop_compress", "calidrop_calibrate", "calidrop_gather_evicted",
    "calidrop_recalibrate", "calidrop_offload_evicted", "calidrop_reload_evicted",
    "calidrop_select_streaming", "calidrop_select_from_scores",
    "calidrop_accumulated_scores_workspace_bytes", "calidrop_accumulated_scores",
    "calidrop_compress_workspace_layout",
    "calidrop_decode_workspace_bytes", "calidrop_decode_workspace_init",
    "calidrop_decode_workspace_status_offset", "calidrop_decode",
    "calidrop_decode_batched", "calidrop_decode_static", "calidrop_compress_host", "calidrop_decode_host",
    "calidrop_status_string", "calidrop_version", "calidrop_launch_count",
]


class Params(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("B", "Hq", "Hkv", "D", "L", "window", "pool", "budget", "n_cal", "cap")] + \
               [("softmax_scale", C.c_float), ("theta1", C.c_float), ("theta2", C.c_float),
                ("calib_size", C.c_int32)]


class CompressLayout(C.Structure):
    _fields_ = [("vote_offset", C.c_size_t), ("pooled_offset", C.c_size_t), ("row_lse_offset", C.c_size_t),
                ("status_offset", C.c_size_t)]


class DecodeLayer(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("q", "k_new", "v_new", "K_kept", "V_kept", "O_c", "LSE_c", "C_q", "out", "lse_out", "flags")]


class CalidropError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)})")


def load():
    """Load libcalidrop.so (built in-tree by paper_2507_19906_b200/build.py)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is not built; run `python -m paper_2507_19906_b200.build` "
                          "(there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    lib.calidrop_compress_workspace_bytes.restype = C.c_size_t
    lib.calidrop_compress_workspace_bytes.argtypes = [C.POINTER(Params)]
    lib.calidrop_decode_workspace_bytes.restype = C.c_size_t
    lib.calidrop_decode_workspace_bytes.argtypes = [C.POINTER(Params), C.c_int32]
    lib.calidrop_compress_workspace_layout.restype = C.c_int
    lib.calidrop_compress_workspace_layout.argtypes = [C.POINTER(Params), C.POINTER(CompressLayout)]
    vp = C.c_void_p
    lib.calidrop_compress.restype = C.c_int
    lib.calidrop_compress.argtypes = [C.POINTER(Params)] + [vp] * 11 + [C.c_size_t, vp]
    lib.calidrop_gather_evicted.restype = C.c_int
    lib.calidrop_gather_evicted.argtypes = [C.POINTER(Params)] + [vp] * 7 + [C.c_size_t, vp]
    lib.calidrop_recalibrate.restype = C.c_int
    lib.calidrop_recalibrate.argtypes = [C.POINTER(Params), vp, vp, vp, C.c_int32, C.c_int32, vp, vp, vp, vp,
                                         C.c_size_t, vp]
    for f in (lib.calidrop_offload_evicted, lib.calidrop_reload_evicted):
        f.restype = C.c_int
        f.argtypes = [C.POINTER(Params), C.c_int32, vp, vp, vp, vp, vp, vp, vp]
    lib.calidrop_select_streaming.restype = C.c_int
    lib.calidrop_select_streaming.argtypes = [C.POINTER(Params), C.c_int32, vp, vp]
    lib.calidrop_accumulated_scores_workspace_bytes.restype = C.c_size_t
    lib.calidrop_accumulated_scores_workspace_bytes.argtypes = [C.POINTER(Params)]
    lib.calidrop_accumulated_scores.restype = C.c_int
    lib.calidrop_accumulated_scores.argtypes = [C.POINTER(Params), vp, vp, vp, vp, C.c_size_t, vp]
    lib.calidrop_select_from_scores.restype = C.c_int
    lib.calidrop_select_from_scores.argtypes = [C.POINTER(Params), vp, C.c_int32, vp, vp, C.c_size_t, vp]
    lib.calidrop_calibrate.restype = C.c_int
    lib.calidrop_calibrate.argtypes = [C.POINTER(Params)] + [vp] * 11 + [C.c_size_t, vp]
    lib.calidrop_decode_workspace_status_offset.restype = C.c_size_t
    lib.calidrop_decode_workspace_status_offset.argtypes = [C.POINTER(Params)]
    lib.calidrop_decode_workspace_init.restype = C.c_int
    lib.calidrop_decode_workspace_init.argtypes = [vp, C.c_size_t, vp]
    lib.calidrop_decode.restype = C.c_int
    lib.calidrop_decode.argtypes = [C.POINTER(Params)] + [vp] * 5 + [C.c_int32] + [vp] * 7 + [C.c_size_t, vp]
    lib.calidrop_decode_batched.restype = C.c_int
    lib.calidrop_decode_batched.argtypes = [C.POINTER(Params), C.c_int32, C.POINTER(DecodeLayer), C.c_int32,
                                            vp, C.c_size_t, vp]
    lib.calidrop_decode_static.restype = C.c_int
    lib.calidrop_decode_static.argtypes = [C.POINTER(Params)] + [vp] * 5 + [C.c_int32] + [vp] * 7
    lib.calidrop_compress_host.restype = C.c_int
    lib.calidrop_compress_host.argtypes = [C.POINTER(Params)] + [vp] * 18 + [C.c_size_t, vp]
    lib.calidrop_decode_host.restype = C.c_int
    lib.calidrop_decode_host.argtypes = [C.POINTER(Params)] + [vp] * 11 + [C.c_int32] + [vp] * 7 + [C.c_size_t, vp]
    lib.calidrop_status_string.restype = C.c_char_p
    lib.calidrop_status_string.argtypes = [C.c_int]
    lib.calidrop_version.restype = C.c_int
    lib.calidrop_launch_count.restype = C.c_uint64
    _lib = lib
    return lib


def make_params(*, B, Hq, Hkv, L=1, window=1, pool=1, budget=1, n_cal=1, cap, D=128,
                softmax_scale=0.0, theta1=0.7, theta2=0.85, calib_size=0) -> Params:
    return Params(B=B, Hq=Hq, Hkv=Hkv, D=D, L=L, window=window, pool=pool, budget=budget,
                  n_cal=n_cal, cap=cap, softmax_scale=softmax_scale, theta1=theta1, theta2=theta2,
                  calib_size=calib_size)


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_contiguous(), "tensors passed to the library must be contiguous"
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _check(rc, where):
    if rc != OK:
        raise CalidropError(rc, where)


def status_string(status: int) -> str:
    return load().calidrop_status_string(status).decode()


def calidrop_version() -> int:
    return load().calidrop_version()


def calidrop_launch_count() -> int:
    return int(load().calidrop_launch_count())


def calidrop_compress_workspace_bytes(p: Params) -> int:
    return int(load().calidrop_compress_workspace_bytes(C.byref(p)))


def calidrop_decode_workspace_bytes(p: Params, kv_len_max: int) -> int:
    return int(load().calidrop_decode_workspace_bytes(C.byref(p), kv_len_max))


def calidrop_decode_workspace_status_offset(p: Params) -> int:
    return int(load().calidrop_decode_workspace_status_offset(C.byref(p)))


def calidrop_compress_workspace_layout(p: Params) -> CompressLayout:
    out = CompressLayout()
    _check(load().calidrop_compress_workspace_layout(C.byref(p), C.byref(out)), "calidrop_compress_workspace_layout")
    return out


def calidrop_compress(p, Q_obs, K, V, lse_obs, kept_idx, K_kept, V_kept, O_c, LSE_c, C_q, workspace,
                      check=True) -> int:
    rc = load().calidrop_compress(C.byref(p), _ptr(Q_obs), _ptr(K), _ptr(V), _ptr(lse_obs), _ptr(kept_idx),
                                  _ptr(K_kept), _ptr(V_kept), _ptr(O_c), _ptr(LSE_c), _ptr(C_q),
                                  _ptr(workspace), workspace.numel() * workspace.element_size(), _stream())
    if check:
        _check(rc, "calidrop_compress")
    return rc


def calidrop_calibrate(p, Q_obs, K, V, lse_obs, kept_idx, K_kept, V_kept, O_c, LSE_c, C_q, workspace,
                       check=True) -> int:
    rc = load().calidrop_calibrate(C.byref(p), _ptr(Q_obs), _ptr(K), _ptr(V), _ptr(lse_obs), _ptr(kept_idx),
                                   _ptr(K_kept), _ptr(V_kept), _ptr(O_c), _ptr(LSE_c), _ptr(C_q),
                                   _ptr(workspace), workspace.numel() * workspace.element_size(), _stream())
    if check:
        _check(rc, "calidrop_calibrate")
    return rc


def calidrop_gather_evicted(p, K, V, kept_idx, evict_idx, K_evict, V_evict, workspace, check=True) -> int:
    rc = load().calidrop_gather_evicted(C.byref(p), _ptr(K), _ptr(V), _ptr(kept_idx), _ptr(evict_idx),
                                        _ptr(K_evict), _ptr(V_evict), _ptr(workspace),
                                        workspace.numel() * workspace.element_size(), _stream())
    if check:
        _check(rc, "calidrop_gather_evicted")
    return rc


def calidrop_recalibrate(p, q, K_evict, V_evict, n_evict, slot, O_c, LSE_c, C_q, workspace, check=True) -> int:
    rc = load().calidrop_recalibrate(C.byref(p), _ptr(q), _ptr(K_evict), _ptr(V_evict), int(n_evict), int(slot),
                                     _ptr(O_c), _ptr(LSE_c), _ptr(C_q), _ptr(workspace),
                                     workspace.numel() * workspace.element_size(), _stream())
    if check:
        _check(rc, "calidrop_recalibrate")
    return rc


def calidrop_select_streaming(p, n_sink, kept_idx, check=True) -> int:
    rc = load().calidrop_select_streaming(C.byref(p), int(n_sink), _ptr(kept_idx), _stream())
    if check:
        _check(rc, "calidrop_select_streaming")
    return rc


def calidrop_accumulated_scores_workspace_bytes(p: Params) -> int:
    return int(load().calidrop_accumulated_scores_workspace_bytes(C.byref(p)))


def calidrop_accumulated_scores(p, Q_full, K, scores, workspace, check=True) -> int:
    rc = load().calidrop_accumulated_scores(C.byref(p), _ptr(Q_full), _ptr(K), _ptr(scores), _ptr(workspace),
                                            workspace.numel() * workspace.element_size(), _stream())
    if check:
        _check(rc, "calidrop_accumulated_scores")
    return rc


def calidrop_select_from_scores(p, scores, tail, kept_idx, workspace, check=True) -> int:
    rc = load().calidrop_select_from_scores(C.byref(p), _ptr(scores), int(tail), _ptr(kept_idx), _ptr(workspace),
                                            workspace.numel() * workspace.element_size(), _stream())
    if check:
        _check(rc, "calidrop_select_from_scores")
    return rc


def _handle(x):
    """A CUDA stream or event of torch (or a raw handle, or None) as the integer the C-ABI takes."""
    if x is None:
        return None
    if isinstance(x, torch.cuda.Stream):
        return x.cuda_stream
    if isinstance(x, torch.cuda.Event):
        h = x.cuda_event                      # exists once the event has been recorded
        return h.value if hasattr(h, "value") else int(h)
    return int(x)


def calidrop_offload_evicted(p, n_evict, K_evict, V_evict, K_host, V_host, copy_stream, wait_event=None,
                             done_event=None, check=True) -> int:
    rc = load().calidrop_offload_evicted(C.byref(p), int(n_evict), _ptr(K_evict), _ptr(V_evict), _ptr(K_host),
                                         _ptr(V_host), _handle(copy_stream), _handle(wait_event), _handle(done_event))
    if check:
        _check(rc, "calidrop_offload_evicted")
    return rc


def calidrop_reload_evicted(p, n_evict, K_host, V_host, K_evict, V_evict, copy_stream, wait_event=None,
                            done_event=None, check=True) -> int:
    rc = load().calidrop_reload_evicted(C.byref(p), int(n_evict), _ptr(K_host), _ptr(V_host), _ptr(K_evict),
                                        _ptr(V_evict), _handle(copy_stream), _handle(wait_event), _handle(done_event))
    if check:
        _check(rc, "calidrop_reload_evicted")
    return rc


def calidrop_decode_workspace_init(workspace) -> int:
    rc = load().calidrop_decode_workspace_init(_ptr(workspace), workspace.numel() * workspace.element_size(),
                                               _stream())
    _check(rc, "calidrop_decode_workspace_init")
    return rc


def calidrop_decode(p, q, k_new, v_new, K_kept, V_kept, kv_len, O_c, LSE_c, C_q, out, lse_out, flags,
                    workspace, check=True) -> int:
    rc = load().calidrop_decode(C.byref(p), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(K_kept), _ptr(V_kept),
                                int(kv_len), _ptr(O_c), _ptr(LSE_c), _ptr(C_q), _ptr(out), _ptr(lse_out),
                                _ptr(flags), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                _stream())
    if check:
        _check(rc, "calidrop_decode")
    return rc


def calidrop_decode_static(p, q, k_new, v_new, K_kept, V_kept, kv_len, O_c, LSE_c, C_q, out, lse_out, flags,
                           check=True) -> int:
    """calidrop_decode with the library's built-in scratch: no workspace argument, nothing allocated."""
    rc = load().calidrop_decode_static(C.byref(p), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(K_kept),
                                       _ptr(V_kept), int(kv_len), _ptr(O_c), _ptr(LSE_c), _ptr(C_q), _ptr(out),
                                       _ptr(lse_out), _ptr(flags), _stream())
    if check:
        _check(rc, "calidrop_decode_static")
    return rc


def make_decode_layers(layers):
    """Pack a list of dicts of tensors into the HOST array calidrop_decode_batched takes."""
    arr = (DecodeLayer * len(layers))()
    for i, d in enumerate(layers):
        for name, _ in DecodeLayer._fields_:
            setattr(arr[i], name, _ptr(d.get(name)))
    return arr


def calidrop_decode_batched(p, layer_array, kv_len, workspace, check=True) -> int:
    rc = load().calidrop_decode_batched(C.byref(p), len(layer_array), layer_array, int(kv_len), _ptr(workspace),
                                        workspace.numel() * workspace.element_size(), _stream())
    if check:
        _check(rc, "calidrop_decode_batched")
    return rc


def calidrop_compress_host(p, Q_obs_h, K_h, V_h, lse_obs_h, kept_idx_h, O_c_h, LSE_c_h,
                           Q_obs, K, V, lse_obs, kept_idx, K_kept, V_kept, O_c, LSE_c, C_q, workspace,
                           check=True) -> int:
    rc = load().calidrop_compress_host(
        C.byref(p), _ptr(Q_obs_h), _ptr(K_h), _ptr(V_h), _ptr(lse_obs_h), _ptr(kept_idx_h), _ptr(O_c_h),
        _ptr(LSE_c_h), _ptr(Q_obs), _ptr(K), _ptr(V), _ptr(lse_obs), _ptr(kept_idx), _ptr(K_kept), _ptr(V_kept),
        _ptr(O_c), _ptr(LSE_c), _ptr(C_q), _ptr(workspace), workspace.numel() * workspace.element_size(),
        _stream())
    if check:
        _check(rc, "calidrop_compress_host")
    return rc


def calidrop_decode_host(p, q_h, k_new_h, v_new_h, out_h, lse_out_h, flags_h, q, k_new, v_new, K_kept, V_kept,
                         kv_len, O_c, LSE_c, C_q, out, lse_out, flags, workspace, check=True) -> int:
    rc = load().calidrop_decode_host(
        C.byref(p), _ptr(q_h), _ptr(k_new_h), _ptr(v_new_h), _ptr(out_h), _ptr(lse_out_h), _ptr(flags_h),
        _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(K_kept), _ptr(V_kept), int(kv_len), _ptr(O_c), _ptr(LSE_c),
        _ptr(C_q), _ptr(out), _ptr(lse_out), _ptr(flags), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _stream())
    if check:
        _check(rc, "calidrop_decode_host")
    return rc


# ------------------------------------------------------------------ convenience allocation
@dataclass
class LayerState:
    """Caller-owned device buffers of one attention layer (allocated with torch)."""
    p: Params
    kept_idx: torch.Tensor
    K_kept: torch.Tensor
    V_kept: torch.Tensor
    O_c: torch.Tensor
    LSE_c: torch.Tensor
    C_q: torch.Tensor
    ws_compress: torch.Tensor
    ws_decode: torch.Tensor
    n_kept: int


def alloc_layer_state(p: Params, device="cuda") -> LayerState:
    n_kept = min(p.budget, p.L)
    u8 = dict(dtype=torch.uint8, device=device)
    bf = dict(dtype=torch.bfloat16, device=device)
    st = LayerState(
        p=p,
        kept_idx=torch.empty((p.B, p.Hkv, n_kept), dtype=torch.int32, device=device),
        K_kept=torch.zeros((p.B, p.Hkv, p.cap, p.D), **bf),
        V_kept=torch.zeros((p.B, p.Hkv, p.cap, p.D), **bf),
        O_c=torch.empty((p.B, p.Hq, p.n_cal, p.D), dtype=torch.float32, device=device),
        LSE_c=torch.empty((p.B, p.Hq, p.n_cal), dtype=torch.float32, device=device),
        C_q=torch.empty((p.B, p.Hq, p.n_cal, p.D), **bf),
        ws_compress=torch.empty((max(calidrop_compress_workspace_bytes(p), 256),), **u8),
        ws_decode=torch.zeros((max(calidrop_decode_workspace_bytes(p, p.cap), 256),), **u8),
        n_kept=n_kept,
    )
    return st
