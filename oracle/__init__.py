"""ctypes binding of the fp64 CPU oracle (oracle/bebop_oracle.c).

TEST INFRASTRUCTURE ONLY.  Importable by tests, by the smoke check and by the
benchmark's CPU-baseline / reference arm; the product package never imports it.
Arrays are numpy; logits are float32 (bf16 inputs are widened exactly by the
caller before they get here).
"""
import ctypes as C
import os

import numpy as np

from .build import build as _build

_lib = None

ST_NONFINITE, ST_EMPTY_ROW, ST_BAD_TOKEN, ST_ZERO_RESID, ST_BAD_TEMP = 1, 2, 4, 8, 16
ST_FATAL = ST_NONFINITE | ST_EMPTY_ROW | ST_BAD_TOKEN | ST_BAD_TEMP
FLAG_MARGIN = 1e-5  # a draw whose accept or CDF margin is below this is "flagged"


def lib():
    """The oracle library.  BEBOP_ORACLE_LIB (a path) replaces it: the mutation test points it at deliberately
    broken builds to show that the pins notice."""
    global _lib
    if _lib is None:
        _lib = C.CDLL(os.environ.get("BEBOP_ORACLE_LIB") or _build())
        _lib.oracle_num_threads.restype = C.c_int
    return _lib


def _p(a, ct):
    return None if a is None else a.ctypes.data_as(C.POINTER(ct))


def _rows(a, ndim):
    a = np.asarray(a)
    assert a.dtype == np.float32 and a.ndim == ndim, (a.dtype, a.shape)
    ok = a.strides[-1] == 4 and a.strides[-2] % 4 == 0 and a.strides[-2] >= 4 * a.shape[-1]
    if ndim == 3 and a.strides[0] != a.shape[1] * a.strides[1]:
        ok = False
    return a if ok else np.ascontiguousarray(a)


def num_threads():
    return int(lib().oracle_num_threads())


def softmax(z, tau=1.0):
    """softmax(z/tau) of one row in fp64 -> (prob[V], status)."""
    z = np.ascontiguousarray(z, dtype=np.float32)
    out = np.zeros(z.shape[0], dtype=np.float64)
    st = lib().oracle_softmax(_p(z, C.c_float), C.c_int64(z.shape[0]), C.c_double(tau),
                              _p(out, C.c_double))
    return out, int(st)


def tv3(p, q):
    """The three equal forms of d_TV for probability rows p, q (fp64)."""
    p = np.ascontiguousarray(p, dtype=np.float64)
    q = np.ascontiguousarray(q, dtype=np.float64)
    out = np.zeros(3, dtype=np.float64)
    lib().oracle_tv3(_p(p, C.c_double), _p(q, C.c_double), C.c_int64(p.shape[0]), _p(out, C.c_double))
    return out


def verify(target, draft, draft_tokens, u_accept, u_final, draft_len=None, temperature=None,
           temperature_all=1.0, nthreads=0):
    """Algorithm 3 per sequence.  target [B,K+1,V] f32, draft [B,K,V] f32.

    Returns a dict: accept_len [B] i32, out_tokens [B,K+1] i32, tv/p_draft/q_draft
    [B,K] f64, row_status [B] i32, margin_acc [B,K], margin_cdf [B], margin_cdf_t [B],
    flagged [B] bool (any evaluated margin below FLAG_MARGIN).
    """
    target = _rows(target, 3)
    B, K1, V = target.shape
    K = K1 - 1
    draft = _rows(draft, 3) if K > 0 else np.zeros((B, 0, V), np.float32)
    assert draft.shape == (B, K, V)
    ld_t = target.strides[1] // 4
    if K > 0:
        ld_d = draft.strides[1] // 4
    else:
        ld_d = V
    tok = np.ascontiguousarray(draft_tokens, dtype=np.int32).reshape(B, K)
    ua = np.ascontiguousarray(u_accept, dtype=np.float32).reshape(B, K)
    uf = np.ascontiguousarray(u_final, dtype=np.float32).reshape(B)
    dl = None if draft_len is None else np.ascontiguousarray(draft_len, dtype=np.int32).reshape(B)
    tp = None if temperature is None else np.ascontiguousarray(temperature, dtype=np.float32).reshape(B)
    o = dict(
        accept_len=np.zeros(B, np.int32), out_tokens=np.zeros((B, K + 1), np.int32),
        tv=np.zeros((B, K), np.float64), p_draft=np.zeros((B, K), np.float64),
        q_draft=np.zeros((B, K), np.float64), row_status=np.zeros(B, np.int32),
        margin_acc=np.zeros((B, K), np.float64), margin_cdf=np.zeros(B, np.float64),
        margin_cdf_t=np.zeros(B, np.float64))
    rc = lib().oracle_verify(
        _p(target, C.c_float), C.c_int64(ld_t), _p(draft, C.c_float), C.c_int64(ld_d),
        _p(tok, C.c_int32), _p(dl, C.c_int32), _p(tp, C.c_float), C.c_float(temperature_all),
        _p(ua, C.c_float), _p(uf, C.c_float), C.c_int(B), C.c_int(K), C.c_int64(V),
        _p(o["accept_len"], C.c_int32), _p(o["out_tokens"], C.c_int32), _p(o["tv"], C.c_double),
        _p(o["p_draft"], C.c_double), _p(o["q_draft"], C.c_double), _p(o["row_status"], C.c_int32),
        _p(o["margin_acc"], C.c_double), _p(o["margin_cdf"], C.c_double),
        _p(o["margin_cdf_t"], C.c_double), C.c_int(nthreads))
    if rc != 0:
        raise MemoryError("oracle_verify")
    o["flagged"] = (o["margin_acc"].min(axis=1, initial=np.inf) < FLAG_MARGIN) | (o["margin_cdf"] < FLAG_MARGIN)
    return o


def tv(target, draft, temperature=None, temperature_all=1.0, nthreads=0):
    """TV and the auxiliary S of N paired rows.  target, draft: [N,V] f32."""
    target = _rows(target, 2)
    draft = _rows(draft, 2)
    N, V = target.shape
    assert draft.shape == (N, V)
    tp = None if temperature is None else np.ascontiguousarray(temperature, dtype=np.float32).reshape(N)
    o = dict(tv=np.zeros(N, np.float64), s_aux=np.zeros(N, np.float64),
             row_status=np.zeros(N, np.int32), tv3=np.zeros((N, 3), np.float64))
    rc = lib().oracle_tv(_p(target, C.c_float), C.c_int64(target.strides[0] // 4),
                         _p(draft, C.c_float), C.c_int64(draft.strides[0] // 4),
                         _p(tp, C.c_float), C.c_float(temperature_all), C.c_int(N), C.c_int64(V),
                         _p(o["tv"], C.c_double), _p(o["s_aux"], C.c_double),
                         _p(o["row_status"], C.c_int32), _p(o["tv3"], C.c_double), C.c_int(nthreads))
    if rc != 0:
        raise MemoryError("oracle_tv")
    return o


def greedy_verify(target, draft_tokens, draft_len=None, nthreads=0):
    """Greedy-draft mode: accept while x_k == argmax target row (lowest index on ties)."""
    target = _rows(target, 3)
    B, K1, V = target.shape
    K = K1 - 1
    tok = np.ascontiguousarray(draft_tokens, dtype=np.int32).reshape(B, K)
    dl = None if draft_len is None else np.ascontiguousarray(draft_len, dtype=np.int32).reshape(B)
    o = dict(accept_len=np.zeros(B, np.int32), out_tokens=np.zeros((B, K + 1), np.int32),
             row_status=np.zeros(B, np.int32))
    lib().oracle_greedy_verify(_p(target, C.c_float), C.c_int64(target.strides[1] // 4),
                               _p(tok, C.c_int32), _p(dl, C.c_int32), C.c_int(B), C.c_int(K),
                               C.c_int64(V), _p(o["accept_len"], C.c_int32),
                               _p(o["out_tokens"], C.c_int32), _p(o["row_status"], C.c_int32),
                               C.c_int(nthreads))
    return o
