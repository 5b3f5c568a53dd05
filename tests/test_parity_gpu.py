"""GPU parity: the CUDA path (through the C ABI) against the fp64 oracle on the
same seeded tensors, sequence by sequence.  Full-size configurations are compared
on every sequence when the host has at least 8 cores (the oracle then needs a few
seconds), otherwise on an evenly spaced sample plus size-independent invariants."""
import numpy as np
import pytest
import torch

import bebop_gen as G
import oracle
import paper_2606_12370_b200 as P
from parity import TOL, check_properties, compare_verify, oracle_on, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda"


PATHS = {"pipe": 2, "general": 1, "fuse": 3}


@pytest.fixture(autouse=True, params=["pipe", "general", "fuse"])
def kernel_path(request):
    """Every test runs three times: through the pipelined kernel and through the fused kernel where the shape admits
    them, and through the general split-row kernels.  (Left alone, the library picks the faster of the first two for
    the shape: the other GPU test files run that way.)"""
    P.bebop_debug_force_general_path(PATHS[request.param])
    yield request.param
    P.bebop_debug_force_general_path(0)


def run_verify(x, **kw):
    return P.bebop_verify(x["target"], x["draft"], x["draft_tokens"], x["u_accept"], x["u_final"],
                          draft_len=x["draft_len"], temperature=x["temperature"],
                          temperature_all=x["temperature_all"], **kw)


def full_check(cfg, pad_ld=0, draft_mode="sample", sample=None):
    x = G.make_inputs(cfg, DEV, draft_mode=draft_mode, pad_ld=pad_ld)
    got = run_verify(x)
    torch.cuda.synchronize()
    check_properties(got, x)
    idx = None
    if sample is not None and sample < cfg.B and oracle.num_threads() < 8:
        idx = np.unique(np.linspace(0, cfg.B - 1, sample).astype(np.int64))
    ref = oracle_on(x, idx)
    return compare_verify(got, ref, cfg.dtype, idx, context=cfg.name), x, got


# ------------------------------------------------------------ the five configs
def test_config1_tiny():
    full_check(G.get_config("tiny"))


def test_config2_rollout():
    full_check(G.get_config("rollout"), sample=32)


def test_config3_high_entropy_sampled_and_greedy():
    cfg = G.get_config("high_entropy")
    full_check(cfg, sample=24)
    x = G.make_inputs(cfg, DEV, draft_mode="argmax")
    got = P.bebop_greedy_verify(x["target"], x["draft_tokens"])
    torch.cuda.synchronize()
    idx = np.unique(np.linspace(0, cfg.B - 1, 48).astype(np.int64))
    ref = oracle.greedy_verify(x["target"][torch.as_tensor(idx, device=DEV)].float().cpu().numpy(),
                               to_np(x["draft_tokens"])[idx])
    for k in ("accept_len", "out_tokens", "row_status"):
        np.testing.assert_array_equal(to_np(got[k])[idx], ref[k])
    # whole batch against torch's own argmax where the maximum is unique
    tgt = x["target"]
    mx = tgt.max(dim=-1, keepdim=True).values
    first = G.first_argmax(tgt.float())
    acc = to_np(got["accept_len"]).astype(np.int64)
    emitted = to_np(got["out_tokens"])[np.arange(cfg.B), acc]
    assert (emitted == to_np(first)[np.arange(cfg.B), acc]).all()
    del mx


def test_config4_large_vocab():
    full_check(G.get_config("large_vocab"), sample=16)


def test_config5_full_batch_ragged():
    full_check(G.get_config("full_batch"), sample=40)


def test_headline_shape():
    full_check(G.get_config("headline"), sample=24)


# ------------------------------------------------------------------ edge cases
@pytest.mark.parametrize("dtype,V,pad", [("f32", 1000, 24), ("f32", 8, 0), ("bf16", 1003, 5),
                                          ("bf16", 8, 0), ("f32", 4099, 1), ("bf16", 40000, 0),
                                          ("f32", 70001, 3), ("bf16", 3 * 151936 // 2, 0)])
def test_ragged_vocab_and_padding(dtype, V, pad):
    cfg = G.Config("edge", 9, 2, V, dtype, 2.0, V >= 16, 0.7, 0.9, seed=11)
    full_check(cfg, pad_ld=pad)


@pytest.mark.parametrize("K", [1, 2, 7, 32])
def test_draft_counts(K):
    cfg = G.Config("k", 6, K, 2048, "bf16", 1.0, False, 0.2, 1.0, ragged=K > 1, seed=K)
    full_check(cfg)


def test_many_short_sequences_finish_in_quick_succession():
    """Rows of one slice: every task completes a row, and a CTA's publisher completes sequences (accept scan,
    draw set-up, the draw task mailed to its own producer) as fast as it publishes."""
    cfg = G.Config("short", 3000, 1, 2040, "bf16", 2.0, True, 1.0, 1.0, seed=31)
    full_check(cfg, sample=256)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_every_sequence_goes_to_the_fp64_redraw(dtype, kernel_path):
    """A target u * Z next to zero sits inside the error bound of the fp32 prefix sum, so no fast draw is kept:
    every sequence is listed while the pipelined kernel still runs, and the re-draw kernel has more work items
    than CTAs.  The token is the first one with residual mass (bonus rows: with probability), exactly."""
    cfg = G.Config("redraw_all", 600, 2, 20000, dtype, 2.0, True, 1.0, 1.0, seed=41)
    x = G.make_inputs(cfg, DEV)
    x["draft_len"] = torch.tensor([i % 3 for i in range(cfg.B)], dtype=torch.int32, device=DEV)
    x["u_final"] = torch.full((cfg.B,), 1e-30, dtype=torch.float32, device=DEV)
    got = run_verify(x)
    got = run_verify(x, workspace=got["workspace"])     # the second call finds the first call's records there
    torch.cuda.synchronize()
    if kernel_path != "general":
        off = P.bebop_debug_fallback_offset(cfg.B, cfg.K, cfg.V, 0 if dtype == "f32" else 1)
        assert int(got["workspace"][off:off + 4].view(torch.int32).item()) == cfg.B
    check_properties(got, x)
    idx = np.unique(np.linspace(0, cfg.B - 1, 96).astype(np.int64))
    ref = oracle_on(x, idx)
    # (the oracle flags every one of these draws as a near-tie of the inverse CDF, which it is; the first token
    # with mass is unique all the same, so the comparison is exact here)
    assert np.array_equal(to_np(got["accept_len"])[idx], ref["accept_len"])
    assert np.array_equal(to_np(got["out_tokens"])[idx], ref["out_tokens"])
    assert np.abs(to_np(got["tv"])[idx] - ref["tv"]).max() <= TOL[dtype]


def test_all_draft_lengths_including_zero():
    cfg = G.Config("len", 10, 4, 4096, "f32", 2.0, False, 0.3, 1.0, seed=5)
    x = G.make_inputs(cfg, DEV)
    x["draft_len"] = torch.tensor([0, 1, 2, 3, 4, 0, 4, 2, 1, 3], dtype=torch.int32, device=DEV)
    got = run_verify(x)
    check_properties(got, x)
    compare_verify(got, oracle_on(x), cfg.dtype)


def test_identical_distributions_accept_everything():
    cfg = G.Config("same", 8, 3, 5000, "bf16", 2.0, False, 0.0, 1.0, seed=2)
    x = G.make_inputs(cfg, DEV)
    x["draft"].copy_(x["target"][:, :3])
    got = run_verify(x)
    assert (to_np(got["accept_len"]) == 3).all()
    assert float(got["tv"].abs().max()) < 1e-6
    compare_verify(got, oracle_on(x), cfg.dtype)


def test_disjoint_supports_and_masked_vocab():
    cfg = G.Config("mask", 6, 2, 2048, "f32", 1.0, False, 0.5, 1.0, seed=3)
    x = G.make_inputs(cfg, DEV)
    x["target"][:, :, :1024] = float("-inf")         # p lives on the upper half
    x["draft"][:3, :, 1024:] = float("-inf")         # q on the lower half for 3 sequences
    x["draft_tokens"][:3] = torch.randint(0, 1024, (3, 2), device=DEV, dtype=torch.int32)
    got = run_verify(x)
    ref = oracle_on(x)
    compare_verify(got, ref, cfg.dtype)
    assert np.allclose(to_np(got["tv"])[:3], 1.0, atol=1e-6)
    assert (to_np(got["accept_len"])[:3] == 0).all()


def test_status_bits():
    cfg = G.Config("st", 8, 2, 1024, "f32", 1.0, False, 0.5, 1.0, seed=4)
    x = G.make_inputs(cfg, DEV)
    x["target"][1, 0, 17] = float("nan")
    x["draft"][2, 1, :] = float("-inf")
    x["draft_tokens"][3, 1] = 1024
    x["temperature"] = torch.ones(8, device=DEV)
    x["temperature"][4] = 0.0
    x["target"][5, 1, 5] = float("inf")
    # sequence 6: p == q with the drafted token masked in both -> zero residual at a reject
    x["draft"][6] = x["target"][6, :2]
    x["target"][6, 0, 9] = float("-inf"); x["draft"][6, 0, 9] = float("-inf")
    x["draft_tokens"][6, 0] = 9
    # sequence 7: NaN only in the bonus row, all drafts accepted (q == p)
    x["draft"][7] = x["target"][7, :2]
    x["target"][7, 2, 100] = float("nan")
    got = run_verify(x)
    ref = oracle_on(x)
    compare_verify(got, ref, cfg.dtype)
    st = to_np(got["row_status"])
    assert st[1] & 1 and st[2] & 2 and st[3] & 4 and st[4] & 16 and st[5] & 1 and st[6] == 8 and st[7] & 1
    assert st[0] == 0


def test_ties_in_logits_coarse_values():
    # coarse integer-valued logits: many exactly tied probabilities
    cfg = G.Config("tie", 12, 3, 512, "bf16", 1.0, False, 0.0, 1.0, seed=6)
    x = G.make_inputs(cfg, DEV)
    g = torch.Generator(device=DEV).manual_seed(1)
    x["target"].copy_(torch.randint(-2, 3, x["target"].shape, generator=g, device=DEV).to(torch.bfloat16))
    x["draft"].copy_(torch.randint(-2, 3, x["draft"].shape, generator=g, device=DEV).to(torch.bfloat16))
    got = run_verify(x)
    compare_verify(got, oracle_on(x), cfg.dtype)
    gx = G.make_inputs(cfg, DEV, draft_mode="argmax")
    gx["target"].copy_(x["target"])
    gg = P.bebop_greedy_verify(gx["target"], gx["draft_tokens"])
    rr = oracle.greedy_verify(gx["target"].float().cpu().numpy(), to_np(gx["draft_tokens"]))
    for k in ("accept_len", "out_tokens", "row_status"):
        np.testing.assert_array_equal(to_np(gg[k]), rr[k])


def test_optional_outputs_may_be_null():
    cfg = G.get_config("tiny")
    x = G.make_inputs(cfg, DEV)
    a = run_verify(x)
    b = run_verify(x, want_tv=False, want_probs=False, want_status=False)
    assert b["tv"] is None and b["p_draft"] is None and b["row_status"] is None
    assert torch.equal(a["accept_len"], b["accept_len"]) and torch.equal(a["out_tokens"], b["out_tokens"])


def test_without_tv_same_tokens_on_a_large_vocabulary():
    """Without a TV output the second sweep reads only the rows a token is drawn from: tokens, accept
    lengths, probabilities and status must not change (ragged lengths, bonus and residual draws)."""
    cfg = G.Config("notv", 24, 4, 40000, "bf16", 3.0, True, 1.0, 1.0, seed=21)
    x = G.make_inputs(cfg, DEV)
    x["draft_len"] = torch.tensor([(i * 7) % 5 for i in range(cfg.B)], dtype=torch.int32, device=DEV)
    a = run_verify(x)
    b = run_verify(x, want_tv=False)
    assert b["tv"] is None
    for k in ("accept_len", "out_tokens", "p_draft", "q_draft", "row_status"):
        assert torch.equal(a[k], b[k]), k


@pytest.mark.parametrize("dtype,K,V", [("f32", 3, 1000), ("bf16", 32, 4096), ("bf16", 1, 70000)])
def test_without_tv_matches_the_oracle(dtype, K, V):
    """The shortened second sweep (tv = NULL) against the oracle directly: ragged lengths with L = 0, every K."""
    cfg = G.Config("notv2", 12, K, V, dtype, 2.0, V > 5000, 1.0, 1.0, seed=23 + K)
    x = G.make_inputs(cfg, DEV)
    x["draft_len"] = torch.tensor([(i * 5) % (K + 1) for i in range(cfg.B)], dtype=torch.int32, device=DEV)
    got = run_verify(x, want_tv=False)
    torch.cuda.synchronize()
    assert got["tv"] is None
    compare_verify(got, oracle_on(x, None), cfg.dtype, None, context=cfg.name)


def test_deterministic_and_stream_ordered():
    cfg = G.Config("det", 16, 3, 32768, "bf16", 3.0, True, 1.0, 1.0, seed=8)
    x = G.make_inputs(cfg, DEV)
    a = run_verify(x)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        b = run_verify(x)
    s.synchronize()
    for k in a:
        if k != "workspace":
            assert torch.equal(a[k], b[k]), k


# ------------------------------------------------------------------- bebop_tv
@pytest.mark.parametrize("dtype,V", [("f32", 1024), ("bf16", 151936), ("bf16", 1003 + 5)])
def test_tv_entry_point(dtype, V):
    cfg = G.Config("tv", 10, 2, V, dtype, 2.0, V > 5000, 0.8, 1.0, seed=13)
    x = G.make_inputs(cfg, DEV)
    tgt = x["target"][:, :2].reshape(20, V)
    drf = x["draft"].reshape(20, V)
    temp = torch.linspace(0.6, 1.2, 20, device=DEV)
    got = P.bebop_tv(tgt, drf, temperature=temp)
    ref = oracle.tv(tgt.float().cpu().numpy(), drf.float().cpu().numpy(), temperature=to_np(temp))
    assert np.abs(to_np(got["tv"]) - ref["tv"]).max() <= TOL[dtype]
    assert np.abs(to_np(got["s_aux"]) - ref["s_aux"]).max() <= TOL[dtype]
    np.testing.assert_array_equal(to_np(got["row_status"]), ref["row_status"])


@pytest.mark.parametrize("dtype,N,V", [("bf16", 20000, 8), ("f32", 9001, 40), ("bf16", 3000, 2056)])
def test_tv_many_short_rows(dtype, N, V):
    """More row pairs than there are warps to complete them (every warp completes several), rows of one slice,
    some of them masked, empty or poisoned, per-row temperatures."""
    gen = torch.Generator(device=DEV).manual_seed(77)
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    tgt = (2.0 * torch.randn(N, V, generator=gen, device=DEV)).to(tdt)
    drf = (tgt.float() + 0.8 * torch.randn(N, V, generator=gen, device=DEV)).to(tdt)
    tgt[5, V // 2:] = float("-inf")
    drf[6, :] = float("-inf")                  # an empty draft row
    tgt[7, 3] = float("nan")
    drf[N - 1, :] = tgt[N - 1, :]              # the last row pair: identical rows
    temp = 0.6 + 0.6 * torch.rand(N, generator=gen, device=DEV)
    got = P.bebop_tv(tgt, drf, temperature=temp)
    ref = oracle.tv(tgt.float().cpu().numpy(), drf.float().cpu().numpy(), temperature=to_np(temp))
    np.testing.assert_array_equal(to_np(got["row_status"]), ref["row_status"])
    ok = ref["row_status"] == 0
    assert np.abs(to_np(got["tv"]) - ref["tv"])[ok].max() <= TOL[dtype]
    assert np.abs(to_np(got["s_aux"]) - ref["s_aux"])[ok].max() <= TOL[dtype]
    assert float(got["tv"][N - 1]) == 0.0


# ---------------------------------------------------------------------- greedy
@pytest.mark.parametrize("dtype,V,K", [("f32", 1000, 3), ("bf16", 151936, 3), ("bf16", 8, 1), ("bf16", 4096, 32)])
def test_greedy_entry_point(dtype, V, K):
    cfg = G.Config("g", 12, K, V, dtype, 1.0, False, 0.3, 1.0, ragged=K > 1, seed=17)
    x = G.make_inputs(cfg, DEV, draft_mode="argmax", pad_ld=(8 - V % 8) % 8)
    x["target"][0, 0, 3] = float("nan")
    x["draft_tokens"][1, 0] = -1
    got = P.bebop_greedy_verify(x["target"], x["draft_tokens"], draft_len=x["draft_len"])
    ref = oracle.greedy_verify(x["target"].float().cpu().numpy(), to_np(x["draft_tokens"]),
                               draft_len=to_np(x["draft_len"]))
    for k in ("accept_len", "out_tokens", "row_status"):
        np.testing.assert_array_equal(to_np(got[k]), ref[k], err_msg=k)
    assert to_np(got["row_status"])[0] & 1 and to_np(got["row_status"])[1] & 4


def test_not_cuda_tensor_is_rejected():
    cfg = G.get_config("tiny")
    x = G.make_inputs(cfg, "cpu")
    with pytest.raises(P.BebopError):
        run_verify(x)
