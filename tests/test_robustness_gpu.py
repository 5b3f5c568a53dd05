"""GPU tests of what surrounds the arithmetic: optional outputs with the dependent kernel launch, the bounded
device-side waits (made to run out by a test hook: nothing is trapped or hung), the workspace bounds (sentinel
words on both sides of the workspace), signed zeros in the greedy mode, and the fast draw's error bound over many
seeds."""
import numpy as np
import pytest
import torch

import bebop_gen as G
import oracle
import paper_2606_12370_b200 as P
from parity import TOL, compare_verify, oracle_on, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda"
PATHS = {"pipe": 2, "general": 1, "fuse": 3}


def run_verify(x, **kw):
    return P.bebop_verify(x["target"], x["draft"], x["draft_tokens"], x["u_accept"], x["u_final"],
                          draft_len=x["draft_len"], temperature=x["temperature"],
                          temperature_all=x["temperature_all"], **kw)


# ------------------------------------------------------- optional outputs and the dependent launch
def test_tv_without_a_status_buffer():
    """bebop_tv with row_status = NULL: the kernel behind the main kernel still has to wait for it, or the
    results could be read (and the workspace cleared by the next call) while they are being written."""
    cfg = G.Config("tvns", 24, 2, 151936, "bf16", 2.0, True, 0.8, 1.0, seed=61)
    x = G.make_inputs(cfg, DEV)
    tgt = x["target"][:, :2].reshape(48, cfg.V)
    drf = x["draft"].reshape(48, cfg.V)
    ws = torch.empty(P.bebop_workspace_bytes(48, 1, cfg.V, 1), dtype=torch.uint8, device=DEV)
    ref = oracle.tv(tgt.float().cpu().numpy(), drf.float().cpu().numpy())
    for _ in range(3):                                   # back to back on one workspace
        got = P.bebop_tv(tgt, drf, workspace=ws, want_status=False)
        host = got["tv"].cpu()                           # a copy enqueued right behind the call
        assert got["row_status"] is None
        assert np.abs(host.numpy() - ref["tv"]).max() <= TOL["bf16"]
        assert np.abs(to_np(got["s_aux"]) - ref["s_aux"]).max() <= TOL["bf16"]


def test_verify_with_tv_and_without_status_twice_on_one_workspace():
    cfg = G.Config("vns", 40, 3, 65536, "bf16", 3.0, True, 1.0, 1.0, seed=62)
    x = G.make_inputs(cfg, DEV)
    ref = oracle_on(x)
    got = run_verify(x, want_status=False)
    for _ in range(2):
        got = run_verify(x, want_status=False, workspace=got["workspace"])
        tv_host = got["tv"].cpu()
        assert got["row_status"] is None
        compare_verify(got, ref, cfg.dtype)
        assert np.abs(tv_host.numpy() - ref["tv"]).max() <= TOL["bf16"]


# ------------------------------------------------------------------------- bounded waits
@pytest.mark.parametrize("path", ["pipe", "fuse"])
@pytest.mark.parametrize("which", [1, 2])
def test_a_wait_that_runs_out_returns_with_the_status_bit(which, path):
    """The hook makes one device-side wait give up as if its bound had run out (1: the re-draw kernel's wait for the
    list of sequences; 2: the main kernel's wait for what other CTAs deliver -- a sequence's accept scan in the
    pipelined kernel, a unit's softmax partials in the fused one).  The call must return, every row must say so,
    and the next call on the same workspace must be normal again."""
    cfg = G.Config("wait", 64, 3, 8192, "bf16", 2.0, True, 1.0, 1.0, seed=63)
    x = G.make_inputs(cfg, DEV)
    P.bebop_debug_force_general_path(PATHS[path])
    ok = run_verify(x)
    torch.cuda.synchronize()
    P.bebop_debug_expire_wait(which)
    bad = run_verify(x, workspace=ok["workspace"])
    torch.cuda.synchronize()                              # returns: nothing hangs
    assert (to_np(bad["row_status"]) & 32 == 32).all()
    again = run_verify(x, workspace=ok["workspace"])
    torch.cuda.synchronize()
    assert (to_np(again["row_status"]) & 32 == 0).all()
    for k in ("accept_len", "out_tokens", "tv", "row_status"):
        assert torch.equal(again[k], ok[k]), k
    compare_verify(again, oracle_on(x), cfg.dtype)
    P.bebop_debug_force_general_path(0)


# ----------------------------------------------------------------------- workspace bounds
GUARD = 4096


def _guarded(nbytes):
    buf = torch.full((nbytes + 2 * GUARD,), 0xA5, dtype=torch.uint8, device=DEV)
    return buf, buf[GUARD:GUARD + nbytes]


def _intact(buf, nbytes):
    return bool((buf[:GUARD] == 0xA5).all()) and bool((buf[GUARD + nbytes:] == 0xA5).all())


@pytest.mark.parametrize("path", ["pipe", "general", "fuse"])
@pytest.mark.parametrize("dtype,B,K,V", [("f32", 9, 2, 1000), ("bf16", 9, 2, 8), ("bf16", 5, 32, 4096), ("f32", 3, 1, 70001),
                                          ("bf16", 7, 3, 3 * 151936 // 2), ("bf16", 300, 1, 2040)])
def test_kernels_stay_inside_the_workspace(path, dtype, B, K, V):
    """4 KB of sentinel bytes before and after exactly bebop_workspace_bytes: every entry point, every path."""
    P.bebop_debug_force_general_path(PATHS[path])
    try:
        cfg = G.Config("guard", B, K, V, dtype, 2.0, V >= 16, 0.7, 1.0, ragged=K > 1, seed=64)
        per16 = 4 if dtype == "f32" else 8
        x = G.make_inputs(cfg, DEV, pad_ld=(-V) % per16)           # rows must start on 16-byte boundaries
        dt = 0 if dtype == "f32" else 1
        n = P.bebop_workspace_bytes(B, K, V, dt)
        buf, ws = _guarded(n)
        run_verify(x, workspace=ws)
        run_verify(x, workspace=ws, want_tv=False)
        P.bebop_greedy_verify(x["target"], x["draft_tokens"], draft_len=x["draft_len"], workspace=ws)
        torch.cuda.synchronize()
        assert _intact(buf, n), "verify / greedy wrote outside the workspace"
        N = B * K
        n2 = P.bebop_workspace_bytes(N, 1, V, dt)
        buf2, ws2 = _guarded(n2)
        ld = x["target"].stride(1)                                   # any N rows with one stride will do here
        P.bebop_tv(torch.as_strided(x["target"], (N, V), (ld, 1)), torch.as_strided(x["draft"], (N, V), (ld, 1)), workspace=ws2)
        torch.cuda.synchronize()
        assert _intact(buf2, n2), "bebop_tv wrote outside the workspace"
    finally:
        P.bebop_debug_force_general_path(0)


# --------------------------------------------------------------------------- greedy, signed zeros
@pytest.mark.parametrize("path", ["pipe", "general"])
def test_greedy_lowest_index_among_signed_zeros(path):
    """A row whose maximum is zero with both signs present: -0.0 at a low index, +0.0 later (in another warp's and
    another slice's range).  The two are equal, so the lowest index wins."""
    P.bebop_debug_force_general_path(PATHS[path])
    try:
        B, K, V = 4, 2, 6000
        tgt = torch.full((B, K + 1, V), -1.0, dtype=torch.bfloat16, device=DEV)
        tgt[:, :, 3] = -0.0
        tgt[:, 0, 700] = 0.0
        tgt[:, 1, 5000] = 0.0
        tgt[1, 2, 3] = -1.0; tgt[1, 2, 40] = 0.0; tgt[1, 2, 41] = -0.0
        tok = torch.full((B, K), 3, dtype=torch.int32, device=DEV)
        got = P.bebop_greedy_verify(tgt, tok)
        ref = oracle.greedy_verify(tgt.float().cpu().numpy(), to_np(tok))
        for k in ("accept_len", "out_tokens", "row_status"):
            np.testing.assert_array_equal(to_np(got[k]), ref[k], err_msg=k)
        assert (to_np(got["accept_len"]) == 2).all() and to_np(got["out_tokens"])[1, 2] == 40
    finally:
        P.bebop_debug_force_general_path(0)


# ------------------------------------------------------------- the fast draw's bound over many seeds
@pytest.mark.parametrize("path", ["pipe", "fuse"])
def test_fast_draw_bound_over_many_seeds_and_temperatures(path):
    """bebop_verify against the oracle on more than 5,000 sequences at V = 151936: 24 seeds, four temperatures, the
    peaked (rollout) and the flat (high-entropy) recipe, residual and bonus draws.  No unflagged mismatch is allowed,
    flagged draws stay below 1e-4, and the share of sequences the fp64 re-draw had to decide is reported.  Both
    kernels that keep fast draws: they bound the error in different ways (the pipelined one from the rows' sums of
    squares, the fused one from the rows' largest probabilities)."""
    P.bebop_debug_force_general_path(PATHS[path])
    B, K, V = 224, 3, 151936
    seen = flagged = draws = redrawn = bonus = 0
    kappas = (0.0, 0.25, 1.0)                                # how much room the built-in factor 4 leaves
    wrong = {k: 0 for k in kappas}; kept = {k: 0 for k in kappas}
    for seed in range(24):
        tau = (0.6, 0.7, 1.0, 1.2)[seed % 4]
        flat = (seed // 4) % 2 == 1
        cfg = G.Config("cert", B, K, V, "bf16", 1.0 if flat else 3.0, not flat, 1.5 if flat else 1.0, tau, seed=1000 + seed)
        x = G.make_inputs(cfg, DEV)
        if seed % 3 == 0:                                   # a third of the batches: short drafts, so more bonus draws
            x["draft_len"] = torch.tensor([i % 2 for i in range(B)], dtype=torch.int32, device=DEV)
        got = run_verify(x)
        torch.cuda.synchronize()
        off = P.bebop_debug_fallback_offset(B, K, V, 1)
        redrawn += int(got["workspace"][off:off + 4].view(torch.int32).item())
        ref = oracle_on(x)
        res = compare_verify(got, ref, cfg.dtype, context="seed %d tau %.1f %s" % (seed, tau, "flat" if flat else "peaked"))
        L = np.full(B, K) if x["draft_len"] is None else to_np(x["draft_len"])
        bonus += int((ref["accept_len"] == L).sum())
        seen += B; flagged += res["flagged"]; draws += res["draws"]
        ok = ~ref["flagged"]
        for kap in kappas:                                  # the same batch with a smaller factor: which draws go wrong?
            P.bebop_debug_set_draw_kappa(kap)
            try:
                g2 = run_verify(x, workspace=got["workspace"])
                torch.cuda.synchronize()
            finally:
                P.bebop_debug_set_draw_kappa(-1.0)
            kept[kap] += B - int(g2["workspace"][off:off + 4].view(torch.int32).item())
            wrong[kap] += int(((to_np(g2["out_tokens"]) != ref["out_tokens"]).any(axis=1) & ok).sum())
    P.bebop_debug_force_general_path(0)
    print("\nfast-draw bound (%s kernel): %d sequences (%d bonus draws), %d draws, %d flagged by the oracle (%.2e), "
          "%d re-drawn in fp64 (%.2f %%), 0 unflagged mismatches"
          % (path, seen, bonus, draws, flagged, flagged / draws, redrawn, 100.0 * redrawn / seen))
    for kap in kappas:
        print("  factor %.2f: %d of %d draws kept in fp32, %d of them differ from the oracle" % (kap, kept[kap], seen, wrong[kap]))
    assert seen >= 5000 and flagged <= 1e-4 * draws + 1
    assert wrong[1.0] == 0, "a quarter of the built-in factor already lets a wrong token through"


# ------------------------------------------------------------------ which kernel runs
def test_the_library_chooses_the_kernel_by_shape():
    """Left alone, bebop_tv goes through the fused kernel (up to 32 slices per row), bebop_verify through the fused
    kernel on small vocabularies and small calls and through the pipelined kernel on large ones; the hook overrides."""
    P.bebop_debug_force_general_path(0)
    small = G.make_inputs(G.Config("d1", 400, 3, 8192, "bf16", 2.0, True, 1.0, 1.0, seed=71), DEV)
    large = G.make_inputs(G.Config("d2", 200, 3, 151936, "bf16", 2.0, True, 1.0, 1.0, seed=72), DEV)
    run_verify(small); assert P.bebop_debug_last_kernel() == 3
    run_verify(large); assert P.bebop_debug_last_kernel() == 2
    P.bebop_tv(large["target"][:, 0], large["draft"][:, 0]); assert P.bebop_debug_last_kernel() == 3
    P.bebop_greedy_verify(large["target"], large["draft_tokens"]); assert P.bebop_debug_last_kernel() == 2
    for mode, want in ((1, 1), (2, 2), (3, 3), (0, 3)):
        P.bebop_debug_force_general_path(mode)
        run_verify(small)
        assert P.bebop_debug_last_kernel() == want
    P.bebop_debug_force_general_path(0)
    torch.cuda.synchronize()
