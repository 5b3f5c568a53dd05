"""bebop_tv_static (built-in scratch, no workspace argument) against bebop_tv, through the C ABI.
Collected last by name; passes alone and after the other GPU tests."""
import pytest
import torch

pytestmark = pytest.mark.gpu


def _inputs(seed, N, V, dtype):
    g = torch.Generator(device="cuda").manual_seed(seed)
    tgt = (2.0 * torch.randn(N, V, generator=g, device="cuda")).to(dtype)
    drf = (tgt.float() + 0.7 * torch.randn(N, V, generator=g, device="cuda")).to(dtype)
    tau = 0.6 + 0.6 * torch.rand(N, generator=g, device="cuda")
    return tgt, drf, tau


@pytest.mark.parametrize("dtype,N,V", [(torch.float32, 5, 1000), (torch.bfloat16, 48, 151936)])
def test_static_equals_workspace_two_calls_in_a_row(dtype, N, V):
    import paper_2606_12370_b200 as P
    P.bebop_debug_force_general_path(0)
    for call in range(2):                       # the second call re-uses the scratch the first one left
        tgt, drf, tau = _inputs(100 + call, N, V, dtype)
        if call == 1:
            tgt[1, 7:] = float("-inf")          # masked vocabulary
            drf[2, :] = tgt[2, :]               # identical rows: TV exactly 0
            tgt[3, 5] = float("nan")            # status bit
        P.bebop_debug_force_general_path(1)     # bebop_tv through the same split-row kernels: bit for bit
        want = P.bebop_tv(tgt, drf, temperature=tau)
        P.bebop_debug_force_general_path(0)     # and through the pipelined kernel: to rounding
        fast = P.bebop_tv(tgt, drf, temperature=tau)
        got = P.bebop_tv_static(tgt, drf, temperature=tau)
        torch.cuda.synchronize()
        assert torch.equal(got["row_status"], want["row_status"]) and torch.equal(got["row_status"], fast["row_status"])
        assert torch.equal(got["tv"].view(torch.int32), want["tv"].view(torch.int32))          # bit for bit
        assert torch.equal(got["s_aux"].view(torch.int32), want["s_aux"].view(torch.int32))
        assert float((got["tv"] - fast["tv"]).abs().max()) <= 1e-5
        assert float((got["s_aux"] - fast["s_aux"]).abs().max()) <= 1e-5
        if call == 1:
            assert float(got["tv"][2]) == 0.0 and int(got["row_status"][3]) & 1


def test_static_against_the_oracle():
    """One small comparison with the fp64 oracle, so that this entry point does not stand on bebop_tv alone."""
    import numpy as np
    import oracle
    import paper_2606_12370_b200 as P
    tgt, drf, tau = _inputs(7, 12, 4100, torch.float32)
    got = P.bebop_tv_static(tgt, drf, temperature=tau)
    ref = oracle.tv(tgt.cpu().numpy(), drf.cpu().numpy(), temperature=tau.cpu().numpy())
    assert np.abs(got["tv"].cpu().numpy() - ref["tv"]).max() <= 1e-5
    assert np.abs(got["s_aux"].cpu().numpy() - ref["s_aux"]).max() <= 1e-5
    assert (got["row_status"].cpu().numpy() == ref["row_status"]).all()


def test_static_limit_is_where_the_header_says():
    """The largest shape the built-in scratch takes (rows in one slice: 24 bytes per row pair in two 256-byte aligned
    arrays of one MiB together, i.e. 43,680 row pairs) runs and equals bebop_tv; one row pair more is refused."""
    import paper_2606_12370_b200 as P
    N, V = 43680, 8
    tgt, drf, tau = _inputs(9, N + 1, V, torch.bfloat16)
    got = P.bebop_tv_static(tgt[:N], drf[:N], temperature=tau[:N])
    P.bebop_debug_force_general_path(1)
    want = P.bebop_tv(tgt[:N], drf[:N], temperature=tau[:N])
    P.bebop_debug_force_general_path(0)
    torch.cuda.synchronize()
    assert torch.equal(got["tv"].view(torch.int32), want["tv"].view(torch.int32))
    with pytest.raises(P.BebopError) as e:
        P.bebop_tv_static(tgt, drf, temperature=tau)
    assert e.value.code == 9


def test_static_rejects_what_does_not_fit():
    import paper_2606_12370_b200 as P
    N, V = 50000, 1024                           # 50,000 row pairs x 1 slice x 24 B > 1 MiB
    tgt = torch.zeros(N, V, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(P.BebopError) as e:
        P.bebop_tv_static(tgt, tgt)
    assert e.value.code == 9 and "built-in scratch" in str(e.value)
    r = P.bebop_tv(tgt, tgt)                     # the workspace entry point takes the same shape
    torch.cuda.synchronize()
    assert float(r["tv"].abs().max()) == 0.0
