"""Helpers shared by the GPU parity tests: run the oracle on (a sample of) the
stored inputs and compare the CUDA outputs with it under the stated bar."""
import math

import numpy as np
import torch

import oracle

TOL = {"f32": 1e-5, "bf16": 2e-3}       # absolute, on TV and on gathered probabilities
MAX_FLAGGED_FRACTION = 1e-4


def to_np(t):
    return None if t is None else t.detach().cpu().numpy()


def oracle_on(x, idx=None, nthreads=0, chunk=32):
    """Run the fp64 oracle on sequences `idx` (all when None) of a generated input set,
    `chunk` sequences at a time so that the widened host copies stay small."""
    B = x["target"].shape[0]
    idx = np.arange(B) if idx is None else np.asarray(idx)
    parts = []
    for i0 in range(0, len(idx), chunk):
        sel = torch.as_tensor(idx[i0:i0 + chunk], device=x["target"].device)
        tgt = x["target"][sel].float().cpu().numpy()
        drf = x["draft"][sel].float().cpu().numpy()
        pick = lambda t: None if t is None else to_np(t[sel])
        parts.append(oracle.verify(tgt, drf, pick(x["draft_tokens"]), pick(x["u_accept"]), pick(x["u_final"]),
                                   draft_len=pick(x["draft_len"]), temperature=pick(x["temperature"]),
                                   temperature_all=x["temperature_all"], nthreads=nthreads))
    return {k: np.concatenate([p[k] for p in parts]) for k in parts[0]}


def compare_verify(got, ref, dtype, idx=None, context=""):
    """got: dict of CUDA tensors for the whole batch; ref: oracle dict for `idx`.
    Integer outputs must match exactly on unflagged draws; flagged draws must be rare."""
    sel = slice(None) if idx is None else np.asarray(idx)
    g = {k: (None if v is None else to_np(v)[sel]) for k, v in got.items() if k != "workspace"}
    flagged = ref["flagged"]
    ok = ~flagged
    bad_len = (g["accept_len"] != ref["accept_len"]) & ok
    bad_tok = (g["out_tokens"] != ref["out_tokens"]).any(axis=1) & ok
    assert not bad_len.any(), "%s accept_len mismatch at %s" % (context, np.nonzero(bad_len)[0][:8])
    assert not bad_tok.any(), "%s token mismatch at %s: got %s want %s margins %s" % (
        context, np.nonzero(bad_tok)[0][:8], g["out_tokens"][bad_tok][:4], ref["out_tokens"][bad_tok][:4],
        ref["margin_cdf"][bad_tok][:4])
    draws = int(np.isfinite(ref["margin_acc"]).sum() + np.isfinite(ref["margin_cdf"]).sum())
    assert int(flagged.sum()) <= math.ceil(MAX_FLAGGED_FRACTION * draws), (context, int(flagged.sum()), draws)
    tol = TOL[dtype]
    if g.get("tv") is not None:
        err = np.abs(g["tv"] - ref["tv"]).max(initial=0.0)
        assert err <= tol, "%s tv error %g" % (context, err)
    for k in ("p_draft", "q_draft"):
        if g.get(k) is not None:
            err = np.abs(g[k] - ref[k]).max(initial=0.0)
            assert err <= tol, "%s %s error %g" % (context, k, err)
    if g.get("row_status") is not None:
        np.testing.assert_array_equal(g["row_status"], ref["row_status"], err_msg=context)
    return dict(flagged=int(flagged.sum()), draws=draws,
                mismatch_flagged=int(((g["accept_len"] != ref["accept_len"]) |
                                      (g["out_tokens"] != ref["out_tokens"]).any(axis=1)).sum()))


def check_properties(got, x):
    """Invariants that hold at any size (used where the oracle only sees a sample)."""
    cfg = x["cfg"]
    acc = to_np(got["accept_len"]).astype(np.int64)
    out = to_np(got["out_tokens"])
    tok = to_np(x["draft_tokens"])
    L = np.full(cfg.B, cfg.K) if x["draft_len"] is None else to_np(x["draft_len"]).astype(np.int64)
    assert ((acc >= 0) & (acc <= L)).all()
    cols = np.arange(cfg.K + 1)[None, :]
    assert (out[:, :cfg.K][cols[:, :cfg.K] < acc[:, None]] == tok[cols[:, :cfg.K] < acc[:, None]]).all()
    emitted = out[np.arange(cfg.B), acc]
    assert ((emitted >= 0) & (emitted < cfg.V)).all()
    assert (out[cols > acc[:, None]] == -1).all()
    if got.get("tv") is not None:
        tv = to_np(got["tv"])
        assert np.isfinite(tv).all() and (tv >= 0).all() and (tv <= 1).all()
        assert (tv[cols[:, :cfg.K] >= L[:, None]] == 0).all()
