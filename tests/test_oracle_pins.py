"""Pins for the float64 oracle: closed forms, invariants, library cross-checks and
brute force on tiny inputs.  None of these tests touches the CUDA path."""
import math

import numpy as np
import pytest

import oracle

LN2 = math.log(2.0)
rng = np.random.default_rng(1234)


def rand_dist(V, sparsity=0.0):
    p = rng.random(V) ** 3
    if sparsity:
        p[rng.random(V) < sparsity] = 0.0
        p[rng.integers(V)] += 0.1
    return p / p.sum()


def bf16_bits(x):
    """float array -> bf16 bits (round to nearest even), as the generator would store it."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return u.astype(np.uint16)


# ------------------------------------------------------------------ softmax / entropy

def test_softmax_golden_and_shift(golden):
    c = golden["entropy_of_softmax_log1234"]
    p, lse = oracle.softmax(c["z"])
    assert np.allclose(p, c["expect"]["p"], atol=1e-15)
    assert abs(lse - c["expect"]["lse"]) < 1e-14
    assert abs(oracle.entropy(p) - c["expect"]["H"]) < 1e-14
    z = rng.normal(size=1000) * 5
    p0, l0 = oracle.softmax(z)
    p1, l1 = oracle.softmax(z + 37.5)
    assert np.allclose(p0, p1, atol=1e-15) and abs(l1 - l0 - 37.5) < 1e-12
    assert abs(p0.sum() - 1.0) < 1e-13


def test_softmax_matches_scipy():
    from scipy.special import logsumexp, softmax
    z = rng.normal(size=5000) * 4
    p, lse = oracle.softmax(z)
    assert np.allclose(p, softmax(z), rtol=1e-13, atol=0)
    assert abs(lse - logsumexp(z)) < 1e-12


def test_softmax_minus_inf_and_nan():
    p, lse = oracle.softmax([0.0, -np.inf, 1.0, -np.inf])
    assert p[1] == 0.0 and p[3] == 0.0 and abs(p.sum() - 1) < 1e-15
    p, lse = oracle.softmax([-np.inf] * 4)
    assert np.isnan(lse) and np.isnan(p).all()
    p, lse = oracle.softmax([0.0, np.nan, 1.0])
    assert np.isnan(lse)


@pytest.mark.parametrize("V", [4, 1000, 128256])
def test_entropy_uniform_is_ln_v(V):
    assert abs(oracle.entropy(np.full(V, 1.0 / V)) - math.log(V)) < 1e-10
    p, _ = oracle.softmax(np.full(V, 3.25))
    assert abs(oracle.entropy(p) - math.log(V)) < 1e-10


def test_entropy_onehot_and_golden(golden):
    e = np.zeros(17)
    e[5] = 1.0
    assert oracle.entropy(e) == 0.0
    c = golden["entropy_dyadic"]
    assert abs(oracle.entropy(c["p"]) - c["expect"]["H"]) < 1e-15


def test_entropy_equals_lse_minus_mean_logit():
    z = rng.normal(size=3000) * 3
    p, lse = oracle.softmax(z)
    assert abs(oracle.entropy(p) - (lse - float(np.dot(p, z)))) < 1e-11


def test_entropy_matches_scipy():
    from scipy.stats import entropy
    p = rand_dist(4096, 0.3)
    assert abs(oracle.entropy(p) - entropy(p)) < 1e-12


# ------------------------------------------------------------------ CE / KL / JSD / distance

def test_kl_is_ce_minus_h(golden):
    c = golden["kl_ce_dyadic_vs_uniform"]
    assert abs(oracle.cross_entropy(c["p"], c["q"]) - c["expect"]["CE"]) < 1e-15
    assert abs(oracle.kl(c["p"], c["q"]) - c["expect"]["KL"]) < 1e-15
    for _ in range(5):
        p, q = rand_dist(500), rand_dist(500)
        assert abs(oracle.kl(p, q) - (oracle.cross_entropy(p, q) - oracle.entropy(p))) < 1e-12
    # asymmetric: a transposed operand would be caught here
    p, q = np.array([0.9, 0.1]), np.array([0.5, 0.5])
    assert abs(oracle.kl(p, q) - (0.9 * math.log(1.8) + 0.1 * math.log(0.2))) < 1e-15
    assert abs(oracle.kl(q, p) - (0.5 * math.log(0.5 / 0.9) + 0.5 * math.log(5.0))) < 1e-15


def test_jsd_golden(golden):
    for name in ("jsd_half_vs_onehot", "jsd_dyadic_vs_uniform", "jsd_disjoint"):
        c = golden[name]
        J = oracle.jsd(c["p"], c["q"])
        assert abs(J - c["expect"]["JSD"]) < 1e-15, name
        if "d" in c["expect"]:
            assert abs(oracle.js_distance(J) - c["expect"]["d"]) < 1e-15, name


def test_jsd_zero_symmetric_bounded():
    for V in (4, 64, 5000):
        p, q = rand_dist(V, 0.2), rand_dist(V, 0.2)
        assert oracle.jsd(p, p) == 0.0
        assert oracle.js_distance(oracle.jsd(p, p)) == 0.0
        assert abs(oracle.jsd(p, q) - oracle.jsd(q, p)) < 1e-15
        assert 0.0 <= oracle.jsd(p, q) <= LN2
    # disjoint supports: exactly ln 2, distance exactly 1
    p = np.zeros(100)
    q = np.zeros(100)
    p[:50] = rand_dist(50)
    q[50:] = rand_dist(50)
    assert abs(oracle.jsd(p, q) - LN2) < 1e-15
    assert oracle.js_distance(LN2) == 1.0
    assert oracle.js_distance(LN2 + 1e-9) == 1.0 and oracle.js_distance(-1e-12) == 0.0


def test_distance_ends_are_exact_whatever_the_rounding_of_the_sum():
    """Sec. 4.4: d is exactly 0 for coinciding rows and exactly 1 for rows that share no
    token, also where the float64 sum of V terms misses 0 or ln 2 in its last bits."""
    r = np.random.default_rng(7)
    missed = 0
    for V in (100, 5001, 128256):
        p = np.zeros(V)
        q = np.zeros(V)
        cut = V // 3
        p[:cut] = r.random(cut) ** 4
        q[cut:] = r.random(V - cut) ** 4
        p /= p.sum()
        q /= q.sum()
        missed += oracle.jsd(p, q) != LN2            # the plain sum need not hit ln 2
        d, J = oracle.js_distance_rows(p, q)
        assert d == 1.0 and J == LN2
        assert oracle.js_distance_rows(q, p) == (1.0, LN2)
        d, J = oracle.js_distance_rows(p, p.copy())
        assert d == 0.0 and J == 0.0
        # one shared token of tiny mass: no longer disjoint, the sum decides (just below 1)
        q2 = q.copy()
        q2[0] = 1e-9
        q2 /= q2.sum()
        d, J = oracle.js_distance_rows(p, q2)
        assert J == oracle.jsd(p, q2) and d == oracle.js_distance(J) and 1.0 - 1e-6 < d <= 1.0
        # ordinary pair: the plain definitions
        a, b = rand_dist(V, 0.1), rand_dist(V, 0.1)
        d, J = oracle.js_distance_rows(a, b)
        assert J == oracle.jsd(a, b) and d == oracle.js_distance(J) and 0.0 < d < 1.0
    assert missed > 0, "the case this rule exists for did not occur"
    d, J = oracle.js_distance_rows([0.5, np.nan], [0.5, 0.5])
    assert math.isnan(d) and math.isnan(J)


def test_jsd_two_printed_forms_agree():
    for V in (4, 333, 20000):
        p, q = rand_dist(V, 0.1), rand_dist(V, 0.1)
        assert abs(oracle.jsd(p, q) - oracle.jsd_entropy_form(p, q)) < 1e-12
        m = 0.5 * (p + q)
        assert abs(oracle.jsd(p, q) - 0.5 * (oracle.kl(p, m) + oracle.kl(q, m))) < 1e-13


def test_js_distance_matches_scipy_base2():
    from scipy.spatial.distance import jensenshannon
    for V in (4, 1000):
        p, q = rand_dist(V), rand_dist(V)
        assert abs(oracle.js_distance(oracle.jsd(p, q)) - jensenshannon(p, q, base=2)) < 1e-12


def test_js_distance_is_sqrt_and_metric():
    assert abs(oracle.js_distance(0.3) - math.sqrt(0.3 / LN2)) < 1e-15
    for V in (4, 16, 64):
        for _ in range(50):
            a, b, c = rand_dist(V, 0.2), rand_dist(V, 0.2), rand_dist(V, 0.2)
            d = lambda x, y: oracle.js_distance(oracle.jsd(x, y))
            assert d(a, c) <= d(a, b) + d(b, c) + 1e-12


# ------------------------------------------------------------------ inverse CDF

def brute_inv_cdf(p, u):
    c = 0.0
    for v, pv in enumerate(p):
        c += pv
        if c > u:
            return v
    return max(v for v, pv in enumerate(p) if pv > 0)


def test_inv_cdf_bruteforce_v4():
    p = np.array([0.1, 0.2, 0.3, 0.4])
    for u, want in [(0.0, 0), (0.05, 0), (0.11, 1), (0.29, 1), (0.31, 2), (0.59, 2), (0.61, 3),
                    (0.999, 3)]:
        assert oracle.inv_cdf(p, u)[0] == want
    for u in np.linspace(0, 0.99999, 997):
        for pp in (p, np.array([0.0, 0.5, 0.0, 0.5]), np.array([0.25] * 4)):
            assert oracle.inv_cdf(pp, u)[0] == brute_inv_cdf(pp, u)


def test_inv_cdf_margin_zero_mass_and_fallback():
    p = np.array([0.0, 0.5, 0.0, 0.5])
    v, m = oracle.inv_cdf(p, 0.3)
    assert v == 1 and abs(m - 0.2) < 1e-15
    v, m = oracle.inv_cdf(p, 0.5)      # C_1 = 0.5 is not > 0.5; token 2 has no mass
    assert v == 3 and abs(m - 0.0) < 1e-15
    # rounding leaves total mass below u: fall back to the last token with mass
    p = np.array([0.3, 0.3, 0.3999999, 0.0])
    assert oracle.inv_cdf(p, 0.99999999)[0] == 2


def test_inv_cdf_histogram():
    p = rand_dist(16)
    us = (np.arange(200000) + 0.5) / 200000
    counts = np.bincount([oracle.inv_cdf(p, u)[0] for u in us[::10]], minlength=16)
    assert np.abs(counts / counts.sum() - p).max() < 2e-4


# ------------------------------------------------------------------ KDE and Bayes

def test_kde_golden(golden):
    c = golden["kde_three_point"]
    L = c["list"]
    assert abs(oracle.sample_std(L) - c["expect"]["std"]) < 1e-15
    assert abs(oracle.kde_bandwidth(L, 0) - c["expect"]["h_silverman"]) < 1e-15
    assert abs(oracle.kde_bandwidth(L, 1) - c["expect"]["h_scott"]) < 1e-15
    assert abs(oracle.kde(L, 0.4) - c["expect"]["f_0.4"]) < 1e-14
    assert abs(oracle.kde(L, 0.2) - c["expect"]["f_0.2"]) < 1e-14
    assert abs(oracle.kde(L, 0.6) - c["expect"]["f_0.2"]) < 1e-14   # symmetric list


def test_kde_integrates_to_one_and_matches_scipy():
    from scipy.stats import gaussian_kde
    L = rng.random(40) * 0.8 + 0.1
    xs = np.linspace(-2, 3, 20001)
    f = np.array([oracle.kde(L, x) for x in xs])
    assert abs(np.trapezoid(f, xs) - 1.0) < 1e-6
    for rule, name in ((0, "silverman"), (1, "scott")):
        g = gaussian_kde(L, bw_method=name)
        for x in (0.0, 0.13, 0.5, 0.77, 1.0):
            assert abs(oracle.kde(L, x, rule) - g(x)[0]) < 1e-12 * max(1.0, g(x)[0])


def test_accept_prob_properties():
    L = rng.random(30)
    for d in (0.1, 0.5, 0.9):
        # identical densities: posterior equals the prior
        assert abs(oracle.accept_prob(L, L, d) - 0.5) < 1e-14
    LA, LR = rng.random(50) * 0.5, 0.4 + rng.random(20) * 0.6
    for d in (0.05, 0.3, 0.45, 0.7, 0.95):
        pa = oracle.accept_prob(LA, LR, d)
        pr = oracle.accept_prob(LR, LA, d)         # roles swapped: P(R|d)
        assert abs(pa + pr - 1.0) < 1e-13
        fa, fr = oracle.kde(LA, d), oracle.kde(LR, d)
        assert abs(pa - 50 * fa / (50 * fa + 20 * fr)) < 1e-14
    assert oracle.accept_prob(LA, LR, 0.1) > 0.9 and oracle.accept_prob(LA, LR, 0.9) < 0.1


def test_accept_prob_cold_start():
    L = rng.random(10)
    assert oracle.accept_prob([], [], 0.3) == 0.0
    assert oracle.accept_prob(L, [], 0.3) == 0.0
    assert oracle.accept_prob(L, [0.4], 0.3) == 0.0
    assert oracle.accept_prob([0.2], L, 0.3) == 0.0
    assert oracle.accept_prob(L, [0.4, 0.4], 0.3) == 0.0          # zero deviation
    assert oracle.accept_prob(L, L, 0.3, min_samples=11) == 0.0
    assert oracle.accept_prob(L, L, 0.3, min_samples=10) == 0.5


# ------------------------------------------------------------------ draft step

def test_draft_step_strict_stop_and_sample():
    z = np.zeros(4, dtype=np.float32)
    r = oracle.draft_step(z, 0.6, 0.0)
    assert abs(r["H"] - math.log(4)) < 1e-15 and r["stop"] and r["token"] == 2
    assert not oracle.draft_step(z, 0.6, r["H"])["stop"]              # H == T_G: strict >
    assert oracle.draft_step(z, 0.6, np.nextafter(r["H"], 0))["stop"]
    zb = bf16_bits(np.log([1, 2, 3, 4]))
    r = oracle.draft_step(zb, 0.35, 10.0)
    zw = oracle.widen(zb)
    p, lse = oracle.softmax(zw)
    assert abs(r["H"] - oracle.entropy(p)) < 1e-15 and abs(r["lse"] - lse) < 1e-15
    assert r["token"] == brute_inv_cdf(p, 0.35) and not r["stop"]


def test_widen_bf16_exact():
    x = np.array([1.0, -2.5, 0.15625, -np.inf, 3.0e38], dtype=np.float32)
    b = bf16_bits(x)
    w = oracle.widen(b)
    assert w[0] == 1.0 and w[1] == -2.5 and w[2] == 0.15625 and w[3] == -np.inf
    assert abs(w[4] / 3.0e38 - 1) < 2 ** -8


# ------------------------------------------------------------------ Algorithm 1, brute force

def py_alg1_round(state, zd, zt, x, ut, ua, min_samples=2):
    """Independent statement of Alg. 1's verify + update with numpy/scipy routines.

    state: dict with python lists LE, LA, LR and float T_G.  Uses scipy's softmax,
    Jensen-Shannon distance and gaussian_kde, none of which the oracle calls."""
    from scipy.spatial.distance import jensenshannon
    from scipy.special import softmax
    from scipy.stats import gaussian_kde
    K = len(x)
    P = [softmax(np.asarray(r, dtype=np.float64)) for r in zt]
    Q = [softmax(np.asarray(r, dtype=np.float64)) for r in zd]
    y = [brute_inv_cdf(P[i], float(ut[i])) for i in range(K + 1)]
    w = K
    for i in range(K):
        d = float(jensenshannon(P[i], Q[i], base=2))
        LA, LR = state["LA"], state["LR"]
        if len(LA) >= max(2, min_samples) and len(LR) >= max(2, min_samples) \
                and np.std(LA) > 0 and np.std(LR) > 0:
            fa = gaussian_kde(LA, bw_method="silverman")(d)[0]
            fr = gaussian_kde(LR, bw_method="silverman")(d)[0]
            na, nr = len(LA), len(LR)
            den = fa * na + fr * nr
            pa = fa * na / den if den > 0 else 0.0
        else:
            pa = 0.0
        if x[i] != y[i] and float(ua[i]) >= pa:
            q = Q[i]
            state["LE"].append(float(-(q[q > 0] * np.log(q[q > 0])).sum()))
            if 0 < d < 1:
                LR.append(d)
            w = i
            break
        if 0 < d < 1:
            LA.append(d)
    if state["LE"]:
        state["T_G"] = float(np.mean(state["LE"]))
    return w, y[w]


def test_alg1_trajectory_against_independent_python():
    V, K, rounds = 48, 6, 60
    r = np.random.default_rng(7)
    st = oracle.SequenceState(capacity=1024, min_samples=8)   # longer cold start: more rejections
    py = dict(LE=[], LA=[], LR=[], T_G=0.0)
    n_rej = 0
    for t in range(rounds):
        zd = (r.normal(size=(K, V)) * 2).astype(np.float32)
        zt = (zd + r.normal(size=(K, V)) * r.choice([0.1, 0.5, 1.5], size=(K, 1))).astype(np.float32)
        zt = np.concatenate([zt, r.normal(size=(1, V)).astype(np.float32)])
        ut = r.random(K + 1).astype(np.float32)
        ua = r.random(K).astype(np.float32)
        # draft tokens: mostly agree with the target sample so that windows vary
        x = np.array([brute_inv_cdf(oracle.softmax(zt[i].astype(np.float64))[0], float(ut[i]))
                      if r.random() < 0.8 else int(r.integers(V)) for i in range(K)])
        out = oracle.verify_round(st, zd, zt, x, ut, ua)
        w, tok = py_alg1_round(py, zd, zt, x, ut, ua, min_samples=8)
        assert out["accept_len"] == w and out["next_token"] == tok, t
        LE, LA, LR = st.lists()
        assert np.allclose(LE, py["LE"], atol=1e-12) and len(LE) == len(py["LE"])
        assert np.allclose(LA, py["LA"], atol=1e-12) and len(LA) == len(py["LA"])
        assert np.allclose(LR, py["LR"], atol=1e-12) and len(LR) == len(py["LR"])
        assert abs(st.T_G.value - py["T_G"]) < 1e-12
        n_rej += out["rejected"]
    assert 5 < n_rej < rounds and st.nA.value > 20 and st.nR.value > 5   # both regimes exercised


def test_tg_is_running_mean_and_zero_until_first_rejection():
    V, K = 32, 3
    r = np.random.default_rng(3)
    st = oracle.SequenceState(capacity=256, min_samples=1000)   # stay in the token-match regime
    Hs = []
    for t in range(12):
        zd = r.normal(size=(K, V)).astype(np.float32)
        zt = r.normal(size=(K + 1, V)).astype(np.float32)
        ut = r.random(K + 1).astype(np.float32)
        y = [oracle.inv_cdf(oracle.softmax(zt[i].astype(np.float64))[0], ut[i])[0] for i in range(K)]
        x = np.array(y)
        if t >= 4:                       # from round 4 on, break the match at position t % K
            x[t % K] = (y[t % K] + 1) % V
        out = oracle.verify_round(st, zd, zt, x, ut, np.zeros(K, dtype=np.float32) + 0.5)
        if t < 4:
            assert out["accept_len"] == K and not out["rejected"] and st.T_G.value == 0.0
            assert out["next_token"] == out["y"][K]
        else:
            i = t % K
            assert out["accept_len"] == i and out["rejected"] and out["next_token"] == y[i]
            Hs.append(out["H_d"][i])
            assert abs(st.T_G.value - np.mean(Hs)) < 1e-13
    assert st.nE.value == 8


def test_boundary_distances_skip_kde_lists_but_entropy_is_recorded():
    V = 8
    st = oracle.SequenceState(capacity=64)
    same = np.array([[0.0, 1.0, 2.0, 3.0, -1.0, 0.5, 0.25, 2.5]], dtype=np.float32)
    zt = np.concatenate([same, same])
    # identical rows: d == 0; force a mismatch -> rejected (cold start P=0)
    y0 = oracle.inv_cdf(oracle.softmax(same[0].astype(np.float64))[0], 0.5)[0]
    out = oracle.verify_round(st, same, zt, [(y0 + 1) % V], [0.5, 0.5], [0.9])
    assert out["dist"][0] == 0.0 and out["rejected"] and out["accept_len"] == 0
    assert (st.nE.value, st.nA.value, st.nR.value) == (1, 0, 0)
    assert abs(st.T_G.value - out["H_d"][0]) < 1e-15
    # identical rows, matching token: accepted, still not recorded
    out = oracle.verify_round(st, same, zt, [y0], [0.5, 0.5], [0.9])
    assert out["accept_len"] == 1 and (st.nE.value, st.nA.value, st.nR.value) == (1, 0, 0)
    # disjoint supports: d == 1
    ninf = -np.inf
    zd = np.array([[0.0, 1.0, ninf, ninf, ninf, ninf, ninf, ninf]], dtype=np.float32)
    zt2 = np.array([[ninf, ninf, 0.0, 1.0, 2.0, ninf, ninf, ninf]] * 2, dtype=np.float32)
    out = oracle.verify_round(st, zd, zt2, [0], [0.5, 0.5], [0.9])
    assert out["dist"][0] == 1.0 and out["rejected"]
    assert (st.nE.value, st.nA.value, st.nR.value) == (2, 0, 0)


def test_unusable_rows_are_rejected_and_leave_the_state_alone():
    """A draft row with NaN (or a target row without a finite logit) has no entropy and no
    distance: the candidate is rejected on a token mismatch, nothing is appended and T_G
    keeps its value (a NaN in L_E^R would switch the stop check off for good)."""
    V = 8
    r = np.random.default_rng(5)
    st = oracle.SequenceState(capacity=64)
    zd = r.normal(size=(2, V)).astype(np.float32)
    zt = r.normal(size=(3, V)).astype(np.float32)
    out = oracle.verify_round(st, zd, zt, [V + 5, V + 5], [0.5, 0.5, 0.5], [0.9, 0.9])   # ordinary rejection first
    assert out["rejected"] and st.nE.value == 1
    T0, sizes = st.T_G.value, (st.nE.value, st.nA.value, st.nR.value)
    zd[0, 3] = np.nan
    out = oracle.verify_round(st, zd, zt, [V + 5, V + 5], [0.5, 0.5, 0.5], [0.9, 0.9])
    assert out["rejected"] and out["accept_len"] == 0 and math.isnan(out["H_d"][0]) and math.isnan(out["dist"][0])
    assert (st.nE.value, st.nA.value, st.nR.value) == sizes and st.T_G.value == T0
    zd[0, 3] = 0.0
    zt[0, :] = -np.inf
    out = oracle.verify_round(st, zd, zt, [V + 5, V + 5], [0.5, 0.5, 0.5], [0.9, 0.9])
    assert out["rejected"] and out["y"][0] == -1 and math.isnan(out["dist"][0])
    assert math.isfinite(out["H_d"][0])                      # the draft row itself is fine ...
    assert (st.nE.value, st.nA.value, st.nR.value) == sizes and st.T_G.value == T0   # ... but the position has no distance


def test_match_always_accepts_and_update_flag():
    V, K = 16, 4
    r = np.random.default_rng(11)
    st = oracle.SequenceState(capacity=64)
    zd = r.normal(size=(K, V)).astype(np.float32)
    zt = r.normal(size=(K + 1, V)).astype(np.float32)
    ut = r.random(K + 1).astype(np.float32)
    y = [oracle.inv_cdf(oracle.softmax(zt[i].astype(np.float64))[0], ut[i])[0] for i in range(K + 1)]
    out = oracle.verify_round(st, zd, zt, y[:K], ut, np.ones(K, dtype=np.float32) * 0.999,
                              update=False)
    assert out["accept_len"] == K and np.all(out["p_acc"] == 0.0)
    assert (st.nE.value, st.nA.value, st.nR.value) == (0, 0, 0)       # update=False leaves state
    out = oracle.verify_round(st, zd, zt, y[:K], ut, np.ones(K, dtype=np.float32) * 0.999)
    assert st.nA.value == K and list(out["y"]) == y


def test_in_round_appends_feed_later_candidates():
    """Candidate i sees the accepted distances d_1..d_{i-1} of the same round."""
    V, K = 16, 3
    r = np.random.default_rng(5)
    st = oracle.SequenceState(capacity=64)
    st.LA[:2] = [0.30, 0.34]
    st.nA.value = 2
    st.LR[:3] = [0.6, 0.7, 0.8]
    st.nR.value = 3
    zd = r.normal(size=(K, V)).astype(np.float32)
    zt = (zd + 0.7 * r.normal(size=(K, V))).astype(np.float32)
    zt = np.concatenate([zt, zd[:1]])
    ut = r.random(K + 1).astype(np.float32)
    y = [oracle.inv_cdf(oracle.softmax(zt[i].astype(np.float64))[0], ut[i])[0] for i in range(K)]
    out = oracle.verify_round(st, zd, zt, y, ut, np.full(K, 0.5, dtype=np.float32), update=False)
    d = out["dist"]
    for i in range(K):
        want = oracle.accept_prob(np.concatenate([[0.30, 0.34], d[:i]]), [0.6, 0.7, 0.8], d[i])
        stale = oracle.accept_prob([0.30, 0.34], [0.6, 0.7, 0.8], d[i])
        assert abs(out["p_acc"][i] - want) < 1e-15
        if i > 0:
            assert abs(want - stale) > 1e-6


def test_reject_rule_threshold_variant():
    st = oracle.SequenceState(capacity=64, reject_rule=1)
    st.LA[:3] = [0.1, 0.2, 0.3]
    st.nA.value = 3
    st.LR[:3] = [0.7, 0.8, 0.9]
    st.nR.value = 3
    z = np.array([[0.0, 0.2, -0.1, 0.05]], dtype=np.float32)
    zt = np.array([[0.1, 0.1, -0.1, 0.0]] * 2, dtype=np.float32)
    y0 = oracle.inv_cdf(oracle.softmax(zt[0].astype(np.float64))[0], 0.5)[0]
    out = oracle.verify_round(st, z, zt, [(y0 + 1) % 4], [0.5, 0.5], [0.999])
    assert out["p_acc"][0] > 0.5 and out["accept_len"] == 1     # small d: accepted although u is large


# ------------------------------------------------------------------ vanilla mode

def logits_of(p):
    with np.errstate(divide="ignore"):
        return np.log(np.asarray(p, dtype=np.float64)).astype(np.float32)


def test_vanilla_golden_alpha_and_residual(golden):
    c = golden["vanilla_reversed"]
    p, q = np.array(c["p"]), np.array(c["q"])
    zt = np.stack([logits_of(p), logits_of(p)])
    zd = logits_of(q)[None]
    for x in range(4):
        out = oracle.vanilla_round(zd, zt, [x], [0.9999], 0.1)
        assert abs(out["alpha"][0] - c["expect"]["alpha"][x]) < 1e-6
    # rejected (u_accept above alpha): the resample follows the residual [0,0,1/4,3/4]
    for ur, want in [(0.1, 2), (0.24, 2), (0.26, 3), (0.9, 3)]:
        out = oracle.vanilla_round(zd, zt, [0], [0.5], ur)
        assert out["accept_len"] == 0 and out["next_token"] == want
    # accepted everywhere: bonus row sampled with u_resample
    out = oracle.vanilla_round(zd, zt, [3], [0.5], 0.35)
    assert out["accept_len"] == 1 and out["next_token"] == 2


def test_vanilla_output_law_is_target_distribution():
    """Leviathan's identity: accept/resample reproduces p_t exactly (V=4 enumeration)."""
    r = np.random.default_rng(21)
    N = 120
    grid = (np.arange(N) + 0.5) / N
    for _ in range(2):
        p, q = rand_dist(4), rand_dist(4)
        zt = np.stack([logits_of(p), logits_of(p)])
        zd = logits_of(q)[None]
        pp = oracle.softmax(zt[0].astype(np.float64))[0]
        qq = oracle.softmax(zd[0].astype(np.float64))[0]
        law = np.zeros(4)
        for x in range(4):
            for ua in grid:
                acc = oracle.vanilla_round(zd, zt, [x], [ua], 0.5)
                if acc["accept_len"] == 1:
                    law[x] += qq[x] / N
                else:
                    for ur in grid:
                        tok = oracle.vanilla_round(zd, zt, [x], [ua], ur)["next_token"]
                        law[tok] += qq[x] / (N * N)
        assert np.abs(law - pp).max() < 2.5 / N


def test_vanilla_first_rejection_prefix():
    V, K = 8, 4
    r = np.random.default_rng(2)
    zd = r.normal(size=(K, V)).astype(np.float32)
    zt = np.concatenate([zd, zd[:1]])            # identical rows: alpha == 1 everywhere
    out = oracle.vanilla_round(zd, zt, [1, 2, 3, 4], [0.999] * K, 0.3)
    assert out["accept_len"] == K and np.all(out["alpha"] == 1.0)
    zt2 = zt.copy()
    zt2[2, 3] -= 20.0                            # token 3 at position 2 becomes very unlikely
    out = oracle.vanilla_round(zd, zt2, [1, 2, 3, 4], [0.5] * K, 0.3)
    assert out["accept_len"] == 2 and out["next_token"] != 3 and np.isnan(out["alpha"][3])


# ------------------------------------------------------------------ greedy decoding and the ablation variants

def test_argmax_hand_cases_and_ties_take_the_lowest_index():
    assert oracle.argmax(np.array([0.5, 2.0, -1.0, 2.0], dtype=np.float32)) == 1        # tie: lowest index
    assert oracle.argmax(np.array([3.0, 2.0, -1.0, 2.5], dtype=np.float32)) == 0
    assert oracle.argmax(np.array([-np.inf, -np.inf, -7.0, -np.inf], dtype=np.float32)) == 2
    assert oracle.argmax(np.array([-np.inf] * 4, dtype=np.float32)) == -1
    assert oracle.argmax(np.array([1.0, np.nan, 5.0, 0.0], dtype=np.float32)) == -1
    # bf16 rounds 1.001 and 1.002 to the same value: a tie once widened, lowest index again
    z = bf16_bits(np.array([0.0, 1.001, 1.002, 0.5]))
    assert oracle.argmax(z) == 1
    r = np.random.default_rng(3)
    for V in (5, 1000, 128256):
        z = r.normal(size=V).astype(np.float32)
        assert oracle.argmax(z) == int(np.argmax(z))
        p, _ = oracle.softmax(z.astype(np.float64))
        assert oracle.argmax(z) == int(np.argmax(p))          # the most probable token (Sec. 2.1.1)


def test_greedy_round_is_the_longest_matching_prefix():
    """Sec. 2.1.3: accept x_i only if it equals argmax p_i; stop at the first mismatch; the
    emitted token is the target's choice there (the bonus row's after a full match)."""
    zt = np.array([[0.0, 3.0, 1.0, 2.0],      # argmax 1
                   [5.0, 5.0, 1.0, 2.0],      # tie 0/1 -> 0
                   [0.0, 1.0, 9.0, 2.0],      # 2
                   [0.0, 1.0, 2.0, 7.0]],     # bonus row: 3
                  dtype=np.float32)
    o = oracle.greedy_round(zt, [1, 0, 2])                     # all match
    assert (o["accept_len"], o["next_token"]) == (3, 3) and list(o["argmax"]) == [1, 0, 2, 3]
    o = oracle.greedy_round(zt, [2, 0, 2])                     # fail at the first candidate
    assert (o["accept_len"], o["next_token"]) == (0, 1) and list(o["argmax"]) == [1, -2, -2, -2]
    o = oracle.greedy_round(zt, [1, 1, 2])                     # the tie goes to index 0, so 1 is a mismatch
    assert (o["accept_len"], o["next_token"]) == (1, 0)
    o = oracle.greedy_round(zt, [1, 0, 3])                     # fail at the last candidate
    assert (o["accept_len"], o["next_token"]) == (2, 2)
    o = oracle.greedy_round(zt[:1], [])                        # empty window: the bonus row decides
    assert (o["accept_len"], o["next_token"]) == (0, 1)
    # brute force on random small cases
    r = np.random.default_rng(9)
    for _ in range(200):
        K, V = int(r.integers(1, 6)), 4
        zt = r.integers(0, 3, size=(K + 1, V)).astype(np.float32)
        x = r.integers(0, V, size=K)
        am = [int(np.argmax(row)) for row in zt]
        w = next((i for i in range(K) if x[i] != am[i]), K)
        o = oracle.greedy_round(zt, x)
        assert (o["accept_len"], o["next_token"]) == (w, am[w])


def test_gen_only_feedback_is_the_running_mean_of_rejected_entropies():
    """Sec. 5 (Gen-Only) with Sec. 4.3: only a rejection feeds T_G, with the entropy of the
    rejected candidate; T_G is the mean of all of them; the distance lists stay empty."""
    st = oracle.SequenceState(capacity=32)
    H = [1.5, 0.25, 3.0, 2.0]
    oracle.gen_only_update(st, H, 4, 4)                        # nothing rejected
    assert st.nE.value == 0 and st.T_G.value == 0.0
    oracle.gen_only_update(st, H, 4, 2)                        # candidate 2 rejected
    assert st.nE.value == 1 and st.T_G.value == 3.0
    oracle.gen_only_update(st, H, 4, 0)
    assert st.nE.value == 2 and st.T_G.value == (3.0 + 1.5) / 2
    oracle.gen_only_update(st, [np.nan, 1.0], 2, 0)            # an unusable row records nothing
    assert st.nE.value == 2 and st.T_G.value == 2.25
    oracle.gen_only_update(st, H, 2, 3)                        # accept_len beyond the window: ignored
    assert st.nE.value == 2 and (st.nA.value, st.nR.value) == (0, 0)


# ------------------------------------------------------------------ adjusted distribution (Sec. 2.1.1)

def test_warp_identities_leave_the_row_alone():
    z = rng.normal(size=50) * 3
    for k, p in [(0, 1.0), (50, 1.0), (77, 1.0), (-1, 1.5)]:
        out, margin = oracle.warp(z, 1.0, k, p)
        assert np.array_equal(out, z) and margin == math.inf
    z32 = z.astype(np.float32)
    assert np.array_equal(oracle.warp(z32)[0], z32.astype(np.float64))
    assert np.array_equal(oracle.warp(bf16_bits(z32))[0], oracle.widen(bf16_bits(z32)))


def test_warp_golden_dyadic_row(golden):
    c = golden["warp_dyadic_v8"]
    e = c["expect"]
    z = np.log(np.array(c["p"]))
    p2 = oracle.softmax(oracle.warp(z, 2.0)[0])[0]
    assert p2[0] == pytest.approx(e["t2_p0"], abs=1e-14) and p2[7] == pytest.approx(e["t2_p7"], abs=1e-14)
    ph = oracle.softmax(oracle.warp(z, 0.5)[0])[0]
    assert ph[0] == pytest.approx(e["thalf_p0"], abs=1e-14) and ph[1] == pytest.approx(e["thalf_p1"], abs=1e-14)
    zk, _ = oracle.warp(z, 1.0, 3, 1.0)
    assert list(np.isfinite(zk)) == [True] * 3 + [False] * 5
    pk, lse = oracle.softmax(zk)
    assert lse == pytest.approx(e["topk3_lse"], abs=1e-14)
    assert oracle.entropy(pk) == pytest.approx(e["topk3_H"], abs=1e-14)
    assert pk[:3] == pytest.approx([4 / 7, 2 / 7, 1 / 7], abs=1e-15)
    zp, margin = oracle.warp(z, 1.0, 0, 0.8)
    assert np.array_equal(np.isfinite(zp), np.isfinite(zk)) and margin == pytest.approx(e["topp08_margin"], abs=1e-12)
    zq, _ = oracle.warp(z, 1.0, 0, 0.74)
    assert list(np.isfinite(zq)) == [True] * 2 + [False] * 6
    pq, lse = oracle.softmax(zq)
    assert lse == pytest.approx(e["topp074_lse"], abs=1e-14)
    assert oracle.entropy(pq) == pytest.approx(e["topp074_H"], abs=1e-14)


def test_warp_temperature_is_a_power_of_the_distribution():
    z = rng.normal(size=300) * 2
    p, _ = oracle.softmax(z)
    for T in (0.3, 0.7, 1.9):
        pT, lseT = oracle.softmax(oracle.warp(z, T)[0])
        ref = p ** (1.0 / T)
        assert np.allclose(pT, ref / ref.sum(), rtol=1e-12, atol=0)
        assert lseT == pytest.approx(np.log(np.exp(z / T - z.max() / T).sum()) + z.max() / T, abs=1e-12)


def test_warp_top_k_against_a_partition_and_ties_stay_together():
    z = rng.normal(size=1000)
    for k in (1, 2, 17, 999):
        out, _ = oracle.warp(z, 1.0, k, 1.0)
        kept = np.flatnonzero(np.isfinite(out))
        assert set(kept) == set(np.argpartition(-z, k - 1)[:k]) and np.array_equal(out[kept], z[kept])
    out, _ = oracle.warp(np.array([3.0, 2.0, 2.0, 1.0, 2.0]), 1.0, 2, 1.0)
    assert list(np.isfinite(out)) == [True, True, True, False, True]          # the tie at rank 2 is not split


def test_warp_top_p_against_an_independent_sort_and_is_minimal():
    """Tie-free rows: the kept set equals the ascending-cumsum rule (drop a token while the
    mass up to and including it, least probable first, is <= 1 - top_p); its mass reaches
    top_p and loses that property when its least probable token is removed."""
    for trial in range(20):
        z = rng.normal(size=400) * (1 + trial % 4)
        top_p = float(rng.uniform(0.05, 0.98))
        out, margin = oracle.warp(z, 1.0, 0, top_p)
        p, _ = oracle.softmax(z)
        order = np.argsort(p, kind="stable")
        csum = np.cumsum(p[order])
        if margin < 1e-9:
            continue
        ref_kept = set(order[csum > 1.0 - top_p])
        kept = np.flatnonzero(np.isfinite(out))
        assert set(kept) == ref_kept
        mass = p[kept].sum()
        assert mass >= top_p - 1e-12 and mass - p[kept].min() < top_p + 1e-12
    out, _ = oracle.warp(np.array([0.0, 0.0, 0.0, -1.0]), 1.0, 0, 0.3)
    assert list(np.isfinite(out)) == [True, True, True, False]                 # ties at the edge stay


def test_warp_steps_apply_in_order_temperature_top_k_top_p():
    z = rng.normal(size=200) * 2
    a, _ = oracle.warp(z, 0.6, 20, 0.7)
    b, _ = oracle.warp(oracle.warp(oracle.warp(z, 0.6)[0], 1.0, 20, 1.0)[0], 1.0, 0, 0.7)
    assert np.array_equal(a, b)
    c, _ = oracle.warp(oracle.warp(z, 1.0, 0, 0.7)[0], 0.6, 20, 1.0)         # another order: another set
    assert not np.array_equal(np.isfinite(a), np.isfinite(c))


def test_warp_unusable_row_is_scaled_and_not_cut():
    z = np.array([1.0, np.nan, 3.0, 2.0])
    out, _ = oracle.warp(z, 2.0, 1, 0.5)
    assert np.isnan(out[1]) and list(out[[0, 2, 3]]) == [0.5, 1.5, 1.0]
    out, _ = oracle.warp(np.full(4, -np.inf), 1.0, 2, 0.5)
    assert np.all(np.isneginf(out))


def test_warped_rows_put_mass_on_the_exact_ends_of_the_distance():
    """Sec. 4.4 observes many distances of exactly 0 or 1; cut supports are where they come
    from: top-1 rows coincide or are disjoint, wider cuts give distances strictly between."""
    zd, zt = rng.normal(size=64), rng.normal(size=64)
    zt[int(np.argmax(zd))] = zt.max() + 1.0                                   # same most probable token
    p, q = oracle.softmax(oracle.warp(zt, 1.0, 1)[0])[0], oracle.softmax(oracle.warp(zd, 1.0, 1)[0])[0]
    assert oracle.js_distance_rows(p, q)[0] == 0.0
    zt2 = zt.copy()
    zt2[int(np.argmin(zd))] = zt2.max() + 1.0
    p2 = oracle.softmax(oracle.warp(zt2, 1.0, 1)[0])[0]
    assert oracle.js_distance_rows(p2, q)[0] == 1.0
    p5, q5 = oracle.softmax(oracle.warp(zt, 1.0, 5)[0])[0], oracle.softmax(oracle.warp(zd, 1.0, 5)[0])[0]
    assert 0.0 < oracle.js_distance_rows(p5, q5)[0] < 1.0


def test_rounds_accept_warped_float64_rows():
    """The round functions take the warped rows as they are (float64): a draft step on a
    top-k row never samples a cut token, and the vanilla accept ratio is 0 for a candidate
    the target's cut removed."""
    z = (rng.normal(size=(1, 32)) * 2).astype(np.float32)
    zk, _ = oracle.warp(z, 0.8, 4, 1.0)
    for u in np.linspace(0.01, 0.99, 25):
        d = oracle.draft_step(zk[0], float(u), 0.0)
        assert np.isfinite(zk[0, d["token"]])
    zd = rng.normal(size=(1, 32))
    zt = np.stack([zd[0] + 0.1, rng.normal(size=32)])
    x = int(np.argmax(zd[0]))
    ztw = zt.copy()
    ztw[0, x] = -np.inf
    ov = oracle.vanilla_round(zd, ztw, [x], [0.5], 0.3)
    assert ov["alpha"][0] == 0.0 and ov["accept_len"] == 0 and ov["next_token"] != x


def test_warp_band_mass_counts_the_groups_near_the_top_p_decision():
    z = np.log(np.array([1 / 2, 1 / 4, 1 / 8, 1 / 16, 1 / 32, 1 / 64, 1 / 128, 1 / 128]))
    # the mass above tokens 0..5 is 0, 1/2, 3/4, 7/8, 15/16, 31/32: top_p = 0.76 is 0.01 from token 2's
    # decision, 0.115 from token 3's, 0.1775 from token 4's and 0.20875 from token 5's
    assert oracle.warp(z, 1.0, 0, 0.76, band=0.005)[2] == 0.0
    assert oracle.warp(z, 1.0, 0, 0.76, band=0.02)[2] == pytest.approx(1 / 8, abs=1e-15)
    assert oracle.warp(z, 1.0, 0, 0.76, band=0.12)[2] == pytest.approx(1 / 8 + 1 / 16, abs=1e-15)
    assert oracle.warp(z, 1.0, 0, 0.76, band=0.2)[2] == pytest.approx(1 / 8 + 1 / 16 + 1 / 32, abs=1e-15)
