"""ctypes binding of libbebop.so.  Same names as the C ABI (include/bebop.h).

Argument marshalling only: tensors are torch CUDA tensors whose device pointers
are handed to the library, outputs are allocated here when not supplied, and the
call is enqueued on torch's current stream.  Nothing is computed in Python.
"""
import ctypes as C
import os
from typing import Optional

import torch

BEBOP_F32, BEBOP_BF16 = 0, 1
_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libbebop.so")
_lib = None


class BebopError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__("bebop status %d: %s" % (code, msg))
        self.code = code


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Load libbebop.so (never builds, never falls back)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError("%s is missing: build it with `python -m paper_2606_12370_b200.build` "
                          "(there is no CPU fallback)" % _LIB_PATH)
    lib = C.CDLL(_LIB_PATH)
    vp, i64, i32, f32, sz = C.c_void_p, C.c_int64, C.c_int, C.c_float, C.c_size_t
    lib.bebop_workspace_bytes.restype = sz
    lib.bebop_workspace_bytes.argtypes = [i32, i32, i32, i32]
    lib.bebop_verify.restype = i32
    lib.bebop_verify.argtypes = [vp, i64, vp, i64, vp, vp, vp, f32, vp, vp, i32, i32, i32, i32,
                                 vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.bebop_tv.restype = i32
    lib.bebop_tv.argtypes = [vp, i64, vp, i64, vp, f32, i32, i32, i32, vp, vp, vp, vp, sz, vp]
    lib.bebop_tv_static.restype = i32
    lib.bebop_tv_static.argtypes = [vp, i64, vp, i64, vp, f32, i32, i32, i32, vp, vp, vp, vp]
    lib.bebop_greedy_verify.restype = i32
    lib.bebop_greedy_verify.argtypes = [vp, i64, vp, vp, i32, i32, i32, i32, vp, vp, vp, vp, sz, vp]
    lib.bebop_debug_force_general_path.restype = None
    lib.bebop_debug_force_general_path.argtypes = [i32]
    lib.bebop_debug_set_timing_events.restype = None
    lib.bebop_debug_set_timing_events.argtypes = [vp, vp]
    lib.bebop_debug_last_kernel.restype = C.c_int
    lib.bebop_debug_last_kernel.argtypes = []
    lib.bebop_debug_set_draw_kappa.restype = None
    lib.bebop_debug_set_draw_kappa.argtypes = [f32]
    lib.bebop_debug_expire_wait.restype = None
    lib.bebop_debug_expire_wait.argtypes = [i32]
    lib.bebop_debug_fallback_offset.restype = sz
    lib.bebop_debug_fallback_offset.argtypes = [i32, i32, i32, i32]
    lib.bebop_status_string.restype = C.c_char_p
    lib.bebop_status_string.argtypes = [i32]
    _lib = lib
    return lib


def bebop_status_string(code: int) -> str:
    return load_library().bebop_status_string(int(code)).decode()


def _check(code: int):
    if code != 0:
        raise BebopError(code, bebop_status_string(code))


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return BEBOP_F32
    if t.dtype == torch.bfloat16:
        return BEBOP_BF16
    raise BebopError(3, "logits must be float32 or bfloat16")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _rows(t: torch.Tensor, ndim: int):
    """(pointer, ld) of a [.., R, V] tensor whose rows are equally spaced."""
    if not t.is_cuda:
        raise BebopError(8, "tensors must live on a CUDA device (no CPU fallback)")
    assert t.dim() == ndim and t.stride(-1) == 1, "vocabulary must be contiguous"
    ld = t.stride(-2)
    if ndim == 3 and t.shape[0] > 1:
        assert t.stride(0) == t.shape[1] * ld, "rows of the batch must be equally spaced"
    return C.c_void_p(t.data_ptr()), int(ld)


def bebop_debug_force_general_path(on) -> None:
    load_library().bebop_debug_force_general_path(int(on))


def bebop_debug_last_kernel() -> int:
    """What the last bebop_verify / bebop_tv / bebop_greedy_verify call ran: 1 general kernels, 2 pipelined kernel, 3 fused kernel."""
    return int(load_library().bebop_debug_last_kernel())


def bebop_debug_set_draw_kappa(kappa) -> None:
    """Factor of the fast draw's error bound (built-in 4; negative restores it; 0 keeps every fp32 draw)."""
    load_library().bebop_debug_set_draw_kappa(float(kappa))


def bebop_debug_expire_wait(which) -> None:
    """The next call lets device-side wait `which` (1: re-draw list, 2: accept scan) give up at once; 0 = off."""
    load_library().bebop_debug_expire_wait(int(which))


def bebop_debug_set_timing_events(start, stop) -> None:
    """torch.cuda.Event pair (enable_timing=True, already recorded once) bracketing the main (pipelined) kernel; None, None = off."""
    lib = load_library()
    if start is None:
        lib.bebop_debug_set_timing_events(None, None)
    else:
        lib.bebop_debug_set_timing_events(C.c_void_p(start.cuda_event), C.c_void_p(stop.cuda_event))


def bebop_debug_fallback_offset(B: int, K: int, V: int, dt: int) -> int:
    return int(load_library().bebop_debug_fallback_offset(B, K, V, dt))


def bebop_workspace_bytes(B: int, K: int, V: int, dt: int) -> int:
    return int(load_library().bebop_workspace_bytes(B, K, V, dt))


# Tests set this so that an output the library failed to write cannot pass as a left-over of an
# earlier call in recycled memory.
POISON_OUTPUTS = False


def _new(shape, dtype, dev):
    if POISON_OUTPUTS:
        return torch.full(shape if isinstance(shape, tuple) else (shape,), -77, dtype=dtype, device=dev)
    return torch.empty(shape, dtype=dtype, device=dev)


def _workspace(B, K, V, dt, device, workspace):
    need = bebop_workspace_bytes(B, K, V, dt)
    if workspace is None:
        workspace = torch.zeros(max(need, 256), dtype=torch.uint8, device=device)
    return workspace, workspace.numel() * workspace.element_size()


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def bebop_verify(target_logits, draft_logits, draft_tokens, u_accept, u_final, draft_len=None,
                 temperature=None, temperature_all=1.0, out=None, workspace=None,
                 want_tv=True, want_probs=True, want_status=True):
    """Chain rejection-sampling verification.  Returns a dict of CUDA tensors:
    accept_len [B] i32, out_tokens [B,K+1] i32, tv / p_draft / q_draft [B,K] f32,
    row_status [B] i32 (the optional ones are None when not requested)."""
    lib = load_library()
    B, K1, V = target_logits.shape
    K = K1 - 1
    dt = _dt(target_logits)
    assert draft_logits.dtype == target_logits.dtype and tuple(draft_logits.shape) == (B, K, V)
    dev = target_logits.device
    tp, ldt = _rows(target_logits, 3)
    dp, ldd = _rows(draft_logits, 3)
    o = out or {}
    def get(name, shape, dtype, want=True):
        if name in o and o[name] is not None:
            return o[name]
        return _new(shape, dtype, dev) if want else None
    res = dict(
        accept_len=get("accept_len", (B,), torch.int32), out_tokens=get("out_tokens", (B, K + 1), torch.int32),
        tv=get("tv", (B, K), torch.float32, want_tv), p_draft=get("p_draft", (B, K), torch.float32, want_probs),
        q_draft=get("q_draft", (B, K), torch.float32, want_probs),
        row_status=get("row_status", (B,), torch.int32, want_status))
    ws, wsb = _workspace(B, K, V, dt, dev, workspace)
    for t in (draft_tokens, u_accept, u_final):
        assert t.is_cuda and t.is_contiguous()
    assert draft_tokens.dtype == torch.int32 and u_accept.dtype == torch.float32 and u_final.dtype == torch.float32
    if draft_len is not None:
        assert draft_len.dtype == torch.int32 and draft_len.is_contiguous()
    if temperature is not None:
        assert temperature.dtype == torch.float32 and temperature.is_contiguous()
    _check(lib.bebop_verify(tp, ldt, dp, ldd, _ptr(draft_tokens), _ptr(draft_len), _ptr(temperature),
                            float(temperature_all), _ptr(u_accept), _ptr(u_final), B, K, V, dt,
                            _ptr(res["accept_len"]), _ptr(res["out_tokens"]), _ptr(res["tv"]),
                            _ptr(res["p_draft"]), _ptr(res["q_draft"]), _ptr(res["row_status"]),
                            _ptr(ws), wsb, _stream()))
    res["workspace"] = ws
    return res


def bebop_tv(target_logits, draft_logits, temperature=None, temperature_all=1.0, workspace=None,
             want_s_aux=True, want_status=True):
    """TV distance (and the auxiliary S) of N paired rows [N,V]."""
    lib = load_library()
    N, V = target_logits.shape
    dt = _dt(target_logits)
    assert draft_logits.dtype == target_logits.dtype and tuple(draft_logits.shape) == (N, V)
    dev = target_logits.device
    tp, ldt = _rows(target_logits, 2)
    dp, ldd = _rows(draft_logits, 2)
    tv = _new(N, torch.float32, dev)
    s_aux = _new(N, torch.float32, dev) if want_s_aux else None
    st = _new(N, torch.int32, dev) if want_status else None
    ws, wsb = _workspace(N, 1, V, dt, dev, workspace)
    _check(lib.bebop_tv(tp, ldt, dp, ldd, _ptr(temperature), float(temperature_all), N, V, dt,
                        _ptr(tv), _ptr(s_aux), _ptr(st), _ptr(ws), wsb, _stream()))
    return dict(tv=tv, s_aux=s_aux, row_status=st)


def bebop_tv_static(target_logits, draft_logits, temperature=None, temperature_all=1.0, want_s_aux=True):
    """bebop_tv with the library's built-in scratch instead of a workspace (no allocation in the call)."""
    lib = load_library()
    N, V = target_logits.shape
    dt = _dt(target_logits)
    assert draft_logits.dtype == target_logits.dtype and tuple(draft_logits.shape) == (N, V)
    dev = target_logits.device
    tp, ldt = _rows(target_logits, 2)
    dp, ldd = _rows(draft_logits, 2)
    tv = _new(N, torch.float32, dev)
    s_aux = _new(N, torch.float32, dev) if want_s_aux else None
    st = _new(N, torch.int32, dev)
    _check(lib.bebop_tv_static(tp, ldt, dp, ldd, _ptr(temperature), float(temperature_all), N, V, dt,
                               _ptr(tv), _ptr(s_aux), _ptr(st), _stream()))
    return dict(tv=tv, s_aux=s_aux, row_status=st)


def bebop_greedy_verify(target_logits, draft_tokens, draft_len=None, workspace=None):
    """Greedy-draft mode: accept while x_k equals the target argmax."""
    lib = load_library()
    B, K1, V = target_logits.shape
    K = K1 - 1
    dt = _dt(target_logits)
    dev = target_logits.device
    tp, ldt = _rows(target_logits, 3)
    assert draft_tokens.dtype == torch.int32 and draft_tokens.is_contiguous() and draft_tokens.is_cuda
    acc = _new(B, torch.int32, dev)
    out = _new((B, K + 1), torch.int32, dev)
    st = _new(B, torch.int32, dev)
    ws, wsb = _workspace(B, K, V, dt, dev, workspace)
    _check(lib.bebop_greedy_verify(tp, ldt, _ptr(draft_tokens), _ptr(draft_len), B, K, V, dt,
                                   _ptr(acc), _ptr(out), _ptr(st), _ptr(ws), wsb, _stream()))
    return dict(accept_len=acc, out_tokens=out, row_status=st)
