"""Pins for the fp64 CPU oracle: closed forms, invariants, library routines,
statistical identities and brute force.  None of these re-types the oracle's
own formula; each would fail for a plausible slip (dropped term, wrong sign,
off-by-one position, swapped p and q)."""
import os
from fractions import Fraction

import numpy as np
import pytest
import scipy.special
import scipy.stats

import oracle

RNG = np.random.default_rng(12345)
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def u_open(shape, rng):
    return ((2 * rng.integers(0, 1 << 23, size=shape) + 1) * 2.0 ** -24).astype(np.float32)


def logits_of(prob):
    with np.errstate(divide="ignore"):
        return np.log(np.asarray(prob, dtype=np.float64)).astype(np.float32)


# ---------------------------------------------------------------- softmax / TV
def test_softmax_matches_scipy():
    for V, tau in [(7, 1.0), (1000, 0.7), (4096, 1.3)]:
        z = (RNG.standard_normal(V) * 3).astype(np.float32)
        p, st = oracle.softmax(z, tau)
        ref = scipy.special.softmax(z.astype(np.float64) / tau)
        assert st == 0
        np.testing.assert_allclose(p, ref, rtol=1e-13, atol=0)
        assert abs(p.sum() - 1.0) < 1e-14


def test_softmax_masked_and_status():
    z = np.array([0.0, -np.inf, 1.0, -np.inf], np.float32)
    p, st = oracle.softmax(z, 1.0)
    assert st == 0 and p[1] == 0.0 and p[3] == 0.0
    np.testing.assert_allclose(p[[0, 2]], scipy.special.softmax([0.0, 1.0]), rtol=1e-15)
    assert oracle.softmax(np.full(5, -np.inf, np.float32))[1] == oracle.ST_EMPTY_ROW
    assert oracle.softmax(np.array([0, np.nan], np.float32))[1] == oracle.ST_NONFINITE
    assert oracle.softmax(np.array([0, np.inf], np.float32))[1] == oracle.ST_NONFINITE


def test_tv_three_forms_agree_and_bounds():
    for V in (5, 333, 20000):
        zp = (RNG.standard_normal(V) * 2).astype(np.float32)
        zq = (zp + RNG.standard_normal(V)).astype(np.float32)
        p, _ = oracle.softmax(zp)
        q, _ = oracle.softmax(zq)
        t = oracle.tv3(p, q)
        assert np.ptp(t) < 1e-12
        assert 0.0 < t[0] < 1.0
        # symmetry and the triangle-free sanity: TV(p,q) == TV(q,p)
        assert abs(oracle.tv3(q, p)[2] - t[2]) < 1e-15
        assert abs(oracle.tv3(q, p)[0] - t[0]) < 1e-12
        # Pinsker: TV <= sqrt(KL(p||q) / 2)
        kl = float(np.sum(p * (np.log(p) - np.log(q))))
        assert t[0] <= np.sqrt(kl / 2) + 1e-12
        # against numpy's own expression of the definition
        assert abs(t[2] - 0.5 * np.abs(p - q).sum()) < 1e-13


def test_tv_special_cases():
    z = (RNG.standard_normal(100)).astype(np.float32)
    o = oracle.tv(z[None], z[None])
    assert o["tv"][0] == 0.0 and abs(o["s_aux"][0] - 1.0) < 1e-14
    # disjoint supports -> TV = 1
    a = z.copy(); b = z.copy()
    a[:50] = -np.inf; b[50:] = -np.inf
    o = oracle.tv(a[None], b[None])
    assert abs(o["tv"][0] - 1.0) < 1e-15 and o["row_status"][0] == 0


def test_restated_formulas_agree():
    """The same expressions typed again in numpy.  This guards against typos only: it pins nothing (a formula
    restated is still the same formula), and the mutation test does not count it."""
    z = (RNG.standard_normal(100)).astype(np.float32)
    zq = (z + RNG.standard_normal(100)).astype(np.float32)
    o = oracle.tv(z[None], zq[None], temperature_all=0.8)
    p = scipy.special.softmax(z.astype(np.float64) / np.float64(np.float32(0.8)))
    q = scipy.special.softmax(zq.astype(np.float64) / np.float64(np.float32(0.8)))
    assert abs(o["s_aux"][0] - q[q <= p].sum()) < 1e-13
    assert abs(o["tv"][0] - np.maximum(p - q, 0).sum()) < 1e-13


def test_s_aux_is_the_scalar_of_the_tv_gradient():
    """Eq. tv_grad (App. A): d TV / d z_j = -q_j (1[q_j <= p_j] - S) / tau for a draft logit z_j, with S the
    oracle's s_aux.  The left side is a central finite difference of the oracle's own TV, so a wrong S (summed over
    the wrong set, or p in place of q) shows as a wrong gradient in every coordinate."""
    rng = np.random.default_rng(99)
    h = 2.0 ** -12
    for V, tau in [(8, 1.0), (32, 0.7), (17, 1.3), (32, 0.5)]:
        # logits on a grid of 2^-12, so that z +- h is exact in float32
        zp = (rng.integers(-8192, 8192, V) * h).astype(np.float32)
        zq = (zp.astype(np.float64) + rng.integers(-4096, 4096, V) * h).astype(np.float32)
        taud = np.float64(np.float32(tau))
        base = oracle.tv(zp[None], zq[None], temperature_all=tau)
        p, _ = oracle.softmax(zp, taud)
        q, _ = oracle.softmax(zq, taud)
        assert np.abs(p - q).min() > 1e-4 * q.min()          # no coordinate sits on the kink q = p
        S = base["s_aux"][0]
        plus = np.repeat(zq[None], V, 0); minus = plus.copy()
        plus[np.arange(V), np.arange(V)] += np.float32(h)
        minus[np.arange(V), np.arange(V)] -= np.float32(h)
        tgt = np.repeat(zp[None], V, 0)
        fd = (oracle.tv(tgt, plus, temperature_all=tau)["tv"] - oracle.tv(tgt, minus, temperature_all=tau)["tv"]) / (2 * h)
        want = -q * ((q <= p).astype(np.float64) - S) / taud
        np.testing.assert_allclose(fd, want, rtol=0, atol=1e-7)
        # Prop. 3: the gradient of every coordinate is bounded by q_j / tau
        assert (np.abs(fd) <= q / taud + 1e-7).all()


def _frac(tok):
    return None if tok == "*" else float(Fraction(tok))


def test_golden_dyadic_s_aux_and_margins():
    """tests/golden/dyadic_margins.txt: S of Eq. tv_grad, the accept margin, both CDF margins and the flag on a
    four-token case worked out by hand, including a draw that must be flagged and one that must not."""
    rows, scal, cases = {}, {}, []
    for line in open(os.path.join(GOLDEN, "dyadic_margins.txt")):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        if f[0] == "case":
            cases.append(f[1:])
        elif len(f) == 5:
            rows[f[0]] = [Fraction(x) for x in f[1:]]
        else:
            scal[f[0]] = float(Fraction(f[1]))
    z = {k: np.log2(np.array([float(x) for x in v])).astype(np.float32) for k, v in rows.items()}
    tau = 1.0 / np.log(2.0)
    o = oracle.tv(z["p"][None], z["q"][None], temperature_all=tau)
    assert abs(o["tv"][0] - scal["tv"]) < 1e-6 and abs(o["s_aux"][0] - scal["s_aux"]) < 1e-6
    tgt = np.stack([z["p"], z["bonus"]])[None]
    for name, tok, ua, uf, n, y, m_acc, m_cdf, m_cdf_t, flagged in cases:
        r = oracle.verify(tgt, z["q"][None, None], np.array([[int(tok)]], np.int32),
                          np.array([[_frac(ua)]], np.float32), np.array([_frac(uf)], np.float32), temperature_all=tau)
        assert abs(r["tv"][0, 0] - scal["tv"]) < 1e-6, name          # per-position TV of the verify call itself
        if n != "*":
            assert r["accept_len"][0] == int(n), name
        if y != "*":
            assert r["out_tokens"][0, r["accept_len"][0]] == int(y), name
        for key, want in (("margin_acc", m_acc), ("margin_cdf", m_cdf), ("margin_cdf_t", m_cdf_t)):
            if want != "*":
                got = r[key][0, 0] if key == "margin_acc" else r[key][0]
                assert abs(got - _frac(want)) < 2e-6, (name, key, got, want)
        assert bool(r["flagged"][0]) == bool(int(flagged)), name


def test_golden_rank_swap_example():
    rows, exp = {}, {}
    for line in open(os.path.join(GOLDEN, "tv_rank_swap.txt")):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        if len(f) == 5:
            rows[f[0]] = [float(x) for x in f[1:]]
        else:
            exp[f[0]] = float(f[1])
    q = logits_of(rows["q"])
    for tag in ("old", "new"):
        zp = logits_of(rows["p_" + tag])
        o = oracle.tv(zp[None], q[None])
        assert abs(o["tv"][0] - exp["tv_" + tag]) < 1e-7
        tok = np.array([[int(np.argmax(rows["q"]))]], np.int32)
        tgt = np.stack([zp, zp])[None]
        g = oracle.greedy_verify(tgt, tok)
        assert g["accept_len"][0] == int(exp["greedy_accept_" + tag])
        # rejection sampling: the drafted old top-1 is accepted iff u < p/q
        ratio = rows["p_" + tag][0] / rows["q"][0]
        for u, want in ((0.5, 1), (min(0.99, ratio + 0.03), 1 if ratio >= 1 else 0)):
            r = oracle.verify(tgt, q[None, None], tok, np.array([[u]], np.float32), np.array([0.5], np.float32))
            assert r["accept_len"][0] == want


def test_shift_and_scale_invariance():
    B, K, V = 6, 2, 257
    tgt = (RNG.standard_normal((B, K + 1, V)) * 2).astype(np.float32)
    drf = (tgt[:, :K] + RNG.standard_normal((B, K, V))).astype(np.float32)
    tok = RNG.integers(0, V, (B, K)).astype(np.int32)
    ua, uf = u_open((B, K), RNG), u_open((B,), RNG)
    a = oracle.verify(tgt, drf, tok, ua, uf)
    # scaling logits and temperature by the same power of two is exact
    b = oracle.verify(tgt * 4, drf * 4, tok, ua, uf, temperature_all=4.0)
    for k in ("accept_len", "out_tokens"):
        np.testing.assert_array_equal(a[k], b[k])
    np.testing.assert_array_equal(a["tv"], b["tv"])
    # adding a constant to a row changes nothing beyond rounding
    c = oracle.verify(tgt + 8, drf - 16, tok, ua, uf)
    ok = ~(a["flagged"] | c["flagged"])
    np.testing.assert_array_equal(a["accept_len"][ok], c["accept_len"][ok])
    np.testing.assert_array_equal(a["out_tokens"][ok], c["out_tokens"][ok])
    np.testing.assert_allclose(a["tv"], c["tv"], atol=1e-6)


# ------------------------------------------------------- accept rule and draws
def _replicated(zt, zd, n):
    K = zd.shape[0]
    V = zt.shape[1]
    tgt = np.broadcast_to(zt, (n, K + 1, V)).copy()
    drf = np.broadcast_to(zd, (n, K, V)).copy()
    return tgt, drf


def test_accept_probability_is_one_minus_tv():
    """Eq. (reject_sample): P(accept) = sum min(p,q) = 1 - TV, by simulation."""
    V, n = 16, 1_000_000
    rng = np.random.default_rng(7)
    zt = (rng.standard_normal((2, V)) * 1.5).astype(np.float32)
    zd = (zt[:1] + rng.standard_normal((1, V))).astype(np.float32)
    q = scipy.special.softmax(zd[0].astype(np.float64))
    tok = rng.choice(V, size=(n, 1), p=q).astype(np.int32)
    tgt, drf = _replicated(zt, zd, n)
    o = oracle.verify(tgt, drf, tok, u_open((n, 1), rng), u_open((n,), rng))
    alpha = 1.0 - o["tv"][0, 0]
    freq = (o["accept_len"] == 1).mean()
    sigma = np.sqrt(alpha * (1 - alpha) / n)
    assert 0.2 < alpha < 0.95
    assert abs(freq - alpha) < 4 * sigma


@pytest.mark.parametrize("K", [1, 3])
def test_output_tokens_follow_target_chi_squared(K):
    """Unbiasedness (Sec. 2.2): the token emitted at every position reached is
    distributed exactly as the target row of that position, bonus included."""
    V, n = 8, 1_000_000
    rng = np.random.default_rng(100 + K)
    zt = (rng.standard_normal((K + 1, V)) * 1.2).astype(np.float32)
    zd = (zt[:K] + rng.standard_normal((K, V)) * 0.8).astype(np.float32)
    tau = 0.9
    taud = np.float64(np.float32(tau))
    tok = np.stack([rng.choice(V, size=n, p=scipy.special.softmax(zd[k].astype(np.float64) / taud))
                    for k in range(K)], axis=1).astype(np.int32)
    tgt, drf = _replicated(zt, zd, n)
    o = oracle.verify(tgt, drf, tok, u_open((n, K), rng), u_open((n,), rng), temperature_all=tau)
    alphas = 1.0 - o["tv"][0]
    for j in range(K + 1):
        reached = o["accept_len"] >= j
        emitted = o["out_tokens"][reached, j]
        assert (emitted >= 0).all()
        p = scipy.special.softmax(zt[j].astype(np.float64) / taud)
        cnt = np.bincount(emitted, minlength=V)
        chi2 = float(((cnt - reached.sum() * p) ** 2 / (reached.sum() * p)).sum())
        assert chi2 < 24.32, (j, chi2)          # 7 dof, p = 1e-3
    # expected accept length E[L] = sum_j prod_{i<=j} alpha_i  (Sec. 2.4 / Eq. e2e_tv)
    expect = float(np.cumprod(alphas).sum())
    sd = o["accept_len"].std() / np.sqrt(n)
    assert abs(o["accept_len"].mean() - expect) < 4 * sd + 1e-9


def test_brute_force_measure_is_exactly_p():
    """V = 4, dyadic probabilities, midpoint grid over every uniform: the measure
    of {emitted token at position j = v}, in rational arithmetic, equals p_j(v)."""
    F = Fraction
    q1 = [F(4, 8), F(2, 8), F(1, 8), F(1, 8)]
    p1 = [F(2, 8), F(2, 8), F(2, 8), F(2, 8)]       # p/q = 1/2,1,1,1 ; residual (0,0,1,1)/8
    q2 = [F(4, 8), F(2, 8), F(1, 8), F(1, 8)]
    p2 = [F(0), F(3, 8), F(3, 8), F(2, 8)]          # masked token; residual (0,1,2,1)/8
    p3 = [F(1, 8), F(3, 8), F(2, 8), F(2, 8)]       # bonus row
    N = 16
    grid = ((np.arange(N) + 0.5) / N).astype(np.float32)
    u1, u2, uf, x1, x2 = np.meshgrid(grid, grid, grid, np.arange(4), np.arange(4), indexing="ij")
    n = u1.size
    tgt = np.broadcast_to(np.stack([logits_of(p1), logits_of(p2), logits_of(p3)]), (n, 3, 4)).copy()
    drf = np.broadcast_to(np.stack([logits_of(q1), logits_of(q2)]), (n, 2, 4)).copy()
    tok = np.stack([x1.ravel(), x2.ravel()], 1).astype(np.int32)
    ua = np.stack([u1.ravel(), u2.ravel()], 1)
    o = oracle.verify(tgt, drf, tok, ua, uf.ravel())
    w = np.array([q1[a] * q2[b] for a, b in tok], dtype=object) * F(1, N ** 3)
    targets = [p1, p2, p3]
    for j in range(3):
        reached = o["accept_len"] >= j
        mass_reached = sum(w[reached], F(0))
        for v in range(4):
            sel = reached & (o["out_tokens"][:, j] == v)
            assert sum(w[sel], F(0)) == targets[j][v] * mass_reached, (j, v)
    # the chain itself: P(accept_len >= 1) = sum min(p1,q1) = 3/4 exactly
    assert sum(w[o["accept_len"] >= 1], F(0)) == F(3, 4)


def test_inverse_cdf_matches_cumsum_searchsorted():
    """Bonus draw (L = 0) and residual draw against numpy cumsum + searchsorted."""
    B, V = 400, 513
    rng = np.random.default_rng(5)
    tgt = (rng.standard_normal((B, 2, V)) * 2).astype(np.float32)
    drf = (tgt[:, :1] + rng.standard_normal((B, 1, V))).astype(np.float32)
    uf = u_open((B,), rng)
    tok = rng.integers(0, V, (B, 1)).astype(np.int32)
    # L = 0: bonus from target row 0
    o = oracle.verify(tgt, drf, tok, u_open((B, 1), rng), uf, draft_len=np.zeros(B, np.int32))
    assert (o["accept_len"] == 0).all() and (o["tv"] == 0).all()
    # forced reject: u_accept close to 1 and p(x) < q(x) is not guaranteed, so use p(x)=0
    tgt2 = tgt.copy()
    tgt2[np.arange(B), 0, tok[:, 0]] = -np.inf
    o2 = oracle.verify(tgt2, drf, tok, u_open((B, 1), rng), uf)
    assert (o2["accept_len"] == 0).all()
    for b in range(B):
        p = scipy.special.softmax(tgt[b, 0].astype(np.float64))
        if o["margin_cdf"][b] > 1e-6:
            c = np.cumsum(p)
            assert o["out_tokens"][b, 0] == np.searchsorted(c, uf[b] * c[-1], side="left")
        p2 = scipy.special.softmax(tgt2[b, 0].astype(np.float64))
        q2 = scipy.special.softmax(drf[b, 0].astype(np.float64))
        if o2["margin_cdf"][b] > 1e-6:
            c = np.cumsum(np.maximum(p2 - q2, 0))
            assert o2["out_tokens"][b, 0] == np.searchsorted(c, uf[b] * c[-1], side="left")
            assert (o2["out_tokens"][b, 1:] == -1).all()


def test_identical_distributions_accept_everything():
    B, K, V = 50, 4, 100
    tgt = (RNG.standard_normal((B, K + 1, V)) * 2).astype(np.float32)
    drf = tgt[:, :K].copy()
    tok = RNG.integers(0, V, (B, K)).astype(np.int32)
    dl = RNG.integers(0, K + 1, B).astype(np.int32)
    o = oracle.verify(tgt, drf, tok, u_open((B, K), RNG), u_open((B,), RNG), draft_len=dl)
    np.testing.assert_array_equal(o["accept_len"], dl)
    assert (o["tv"] == 0).all()
    for b in range(B):
        np.testing.assert_array_equal(o["out_tokens"][b, : dl[b]], tok[b, : dl[b]])
        assert o["out_tokens"][b, dl[b]] >= 0
        assert (o["out_tokens"][b, dl[b] + 1:] == -1).all()


def test_gathered_probabilities_and_margins():
    B, K, V = 20, 3, 300
    tgt = (RNG.standard_normal((B, K + 1, V)) * 2).astype(np.float32)
    drf = (tgt[:, :K] + RNG.standard_normal((B, K, V))).astype(np.float32)
    tok = RNG.integers(0, V, (B, K)).astype(np.int32)
    ua = u_open((B, K), RNG)
    o = oracle.verify(tgt, drf, tok, ua, u_open((B,), RNG), temperature_all=0.5)
    for b in range(B):
        n = o["accept_len"][b]
        for k in range(K):
            p = scipy.special.softmax(tgt[b, k].astype(np.float64) / 0.5)
            q = scipy.special.softmax(drf[b, k].astype(np.float64) / 0.5)
            assert abs(o["p_draft"][b, k] - p[tok[b, k]]) < 1e-14
            assert abs(o["q_draft"][b, k] - q[tok[b, k]]) < 1e-14
            acc = ua[b, k] * q[tok[b, k]] < p[tok[b, k]]
            if k < n:
                assert acc
            if k == n:
                assert not acc
            assert np.isfinite(o["margin_acc"][b, k]) == (k <= n)


# --------------------------------------------------------------------- greedy
def test_greedy_reduces_to_leading_argmax_match():
    B, K, V = 64, 5, 50
    # coarse values -> many tied maxima; numpy argmax returns the first one
    tgt = RNG.integers(-3, 4, (B, K + 1, V)).astype(np.float32)
    g = tgt.argmax(axis=2)
    tok = g[:, :K].astype(np.int32).copy()
    flip = RNG.random((B, K)) < 0.3
    tok[flip] = (tok[flip] + 1) % V
    dl = RNG.integers(0, K + 1, B).astype(np.int32)
    o = oracle.greedy_verify(tgt, tok, draft_len=dl)
    for b in range(B):
        n = 0
        while n < dl[b] and tok[b, n] == g[b, n]:
            n += 1
        assert o["accept_len"][b] == n
        assert o["out_tokens"][b, n] == g[b, n]
        np.testing.assert_array_equal(o["out_tokens"][b, :n], tok[b, :n])
        assert (o["out_tokens"][b, n + 1:] == -1).all()


# ------------------------------------------------------------- status / ragged
def test_status_bits_and_fatal_rows():
    B, K, V = 6, 2, 40
    tgt = RNG.standard_normal((B, K + 1, V)).astype(np.float32)
    drf = RNG.standard_normal((B, K, V)).astype(np.float32)
    tok = RNG.integers(0, V, (B, K)).astype(np.int32)
    tgt[1, 0, 3] = np.nan
    drf[2, 1, :] = -np.inf
    tok[3, 1] = V
    temp = np.ones(B, np.float32); temp[4] = 0.0
    o = oracle.verify(tgt, drf, tok, u_open((B, K), RNG), u_open((B,), RNG), temperature=temp)
    assert o["row_status"][0] == 0 and o["out_tokens"][0, o["accept_len"][0]] >= 0
    assert o["row_status"][1] & oracle.ST_NONFINITE
    assert o["row_status"][2] & oracle.ST_EMPTY_ROW
    assert o["row_status"][3] & oracle.ST_BAD_TOKEN
    assert o["row_status"][4] & oracle.ST_BAD_TEMP
    for b in (1, 2, 3, 4):
        assert o["accept_len"][b] == 0 and (o["out_tokens"][b] == -1).all() and (o["tv"][b] == 0).all()
    assert o["row_status"][5] == 0


def test_zero_residual_falls_back_to_target():
    V = 6
    z = RNG.standard_normal(V).astype(np.float32)
    z[2] = -np.inf                       # p(x) = q(x) = 0 for the drafted token, p == q elsewhere
    tgt = np.stack([z, z])[None]
    o = oracle.verify(tgt, z[None, None], np.array([[2]], np.int32), np.array([[0.5]], np.float32),
                      np.array([0.4], np.float32))
    assert o["accept_len"][0] == 0 and o["row_status"][0] == oracle.ST_ZERO_RESID
    c = np.cumsum(scipy.special.softmax(z.astype(np.float64)))
    assert o["out_tokens"][0, 0] == np.searchsorted(c, 0.4 * c[-1])


def test_threads_do_not_change_results():
    B, K, V = 16, 2, 200
    tgt = RNG.standard_normal((B, K + 1, V)).astype(np.float32)
    drf = RNG.standard_normal((B, K, V)).astype(np.float32)
    tok = RNG.integers(0, V, (B, K)).astype(np.int32)
    ua, uf = u_open((B, K), RNG), u_open((B,), RNG)
    a = oracle.verify(tgt, drf, tok, ua, uf, nthreads=1)
    b = oracle.verify(tgt, drf, tok, ua, uf, nthreads=4)
    for k in a:
        np.testing.assert_array_equal(a[k], b[k])
