"""Pins for the oracle's EGAE / Monte-Carlo return (Eq. 2, 3, 6 and R_t after Eq. 5)."""
import os

import numpy as np
import pytest
from scipy.signal import lfilter

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))


def brute_force_adv(r, v, b, e, trunc, boot, gamma, lam):
    """Eq. 6 taken literally: one explicit double sum per token."""
    out = np.zeros(len(r))
    for t in range(b, e):
        s = 0.0
        for k in range(t, e):
            if k + 1 < e:
                vn = v[k + 1]
            else:
                vn = (boot if boot is not None else v[e - 1]) if trunc else 0.0
            delta = r[k] + gamma * vn - v[k]
            s += (gamma * lam) ** (k - t) * delta
        out[t] = s
    return out


def random_case(rng, B, maxlen, gap=True):
    lens = rng.integers(1, maxlen + 1, B)
    gaps = rng.integers(0, 4, B) if gap else np.zeros(B, int)
    sb, se, pos = [], [], 0
    for L, g in zip(lens, gaps):
        pos += g
        sb.append(pos)
        pos += L
        se.append(pos)
    N = pos + 2
    r = rng.standard_normal(N).astype(np.float32)
    v = rng.standard_normal(N).astype(np.float32)
    tr = rng.integers(0, 2, B).astype(np.uint8)
    return r, v, np.array(sb, np.int32), np.array(se, np.int32), tr, N


def test_hand_example_fixture():
    rows = [l.split() for l in open(os.path.join(HERE, "golden", "egae_hand_example.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 2
    for row in rows:
        trunc = int(row[1])
        r = [float(x) for x in row[2:5]]
        A = [float(x) for x in row[5:8]]
        R = [float(x) for x in row[8:11]]
        adv, ret = oracle.egae(r, [0.5, 0.2, 0.1], [0], [3], [trunc], None, 1.0, 0.5)
        np.testing.assert_allclose(adv, A, atol=1e-12)
        np.testing.assert_allclose(ret, R, atol=1e-12)


@pytest.mark.parametrize("gamma,lam", [(1.0, 0.95), (0.99, 0.9), (1.0, 1.0), (0.9, 0.0), (0.97, 1.0)])
def test_matches_brute_force_sum(gamma, lam):
    rng = np.random.default_rng(7)
    r, v, sb, se, tr, N = random_case(rng, 6, 12)
    for boot in (None, rng.standard_normal(6).astype(np.float32)):
        adv, _ = oracle.egae(r, v, sb, se, tr, boot, gamma, lam)
        ref = np.zeros(N)
        for i in range(6):
            ref += brute_force_adv(r.astype(float), v.astype(float), sb[i], se[i], tr[i],
                                   None if boot is None else float(boot[i]), gamma, lam)
        np.testing.assert_allclose(adv, ref, rtol=1e-12, atol=1e-12)


def test_equals_textbook_gae_when_nothing_is_truncated():
    """Section 3.1: same form as GAE with T replaced by l.  Comparator: scipy's IIR filter run
    over the reversed TD residuals (y[n] = x[n] + gamma*lambda*y[n-1])."""
    rng = np.random.default_rng(11)
    r, v, sb, se, tr, N = random_case(rng, 5, 40)
    tr[:] = 0
    gamma, lam = 0.99, 0.95
    adv, ret = oracle.egae(r, v, sb, se, tr, None, gamma, lam)
    for b, e in zip(sb, se):
        vv = v[b:e].astype(float)
        vnext = np.append(vv[1:], 0.0)
        delta = r[b:e] + gamma * vnext - vv
        gae = lfilter([1.0], [1.0, -gamma * lam], delta[::-1])[::-1]
        np.testing.assert_allclose(adv[b:e], gae, rtol=1e-12, atol=1e-12)
        mc = lfilter([1.0], [1.0, -gamma], r[b:e].astype(float)[::-1])[::-1]
        np.testing.assert_allclose(ret[b:e], mc, rtol=1e-12, atol=1e-12)


def test_truncated_equals_gae_with_pseudo_reward():
    """A truncated segment is a finished one whose last reward is r + gamma*V_boot."""
    rng = np.random.default_rng(12)
    r, v, sb, se, tr, N = random_case(rng, 5, 30)
    tr[:] = 1
    gamma, lam = 0.98, 0.9
    adv, _ = oracle.egae(r, v, sb, se, tr, None, gamma, lam)
    r2 = r.astype(np.float64).copy()
    for b, e in zip(sb, se):
        r2[e - 1] += gamma * float(v[e - 1])
    for b, e in zip(sb, se):
        vv = v[b:e].astype(float)
        delta = r2[b:e] + gamma * np.append(vv[1:], 0.0) - vv
        gae = lfilter([1.0], [1.0, -gamma * lam], delta[::-1])[::-1]
        np.testing.assert_allclose(adv[b:e], gae, rtol=1e-12, atol=1e-12)


def test_gamma_lambda_one_is_reward_to_go_minus_value():
    rng = np.random.default_rng(13)
    r, v, sb, se, tr, N = random_case(rng, 8, 50)
    boot = rng.standard_normal(8).astype(np.float32)
    adv, ret = oracle.egae(r, v, sb, se, tr, boot, 1.0, 1.0)
    for i, (b, e) in enumerate(zip(sb, se)):
        rtg = np.cumsum(r[b:e].astype(float)[::-1])[::-1]
        vb = float(boot[i]) if tr[i] else 0.0
        np.testing.assert_allclose(adv[b:e], rtg + vb - v[b:e], rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(ret[b:e], rtg, rtol=1e-12, atol=1e-12)
        if not tr[i]:  # lambda=1 advantage plus value is the Monte-Carlo return
            np.testing.assert_allclose(adv[b:e] + v[b:e], ret[b:e], atol=1e-12)


def test_last_token_of_truncated_response():
    """V(s_l)=V(s_{l-1}) makes delta_{l-1} = r + (gamma-1) V(s_{l-1}); 0 for gamma=1, r=0."""
    rng = np.random.default_rng(14)
    r, v, sb, se, tr, N = random_case(rng, 6, 20)
    r[:] = 0
    tr[:] = 1
    adv, _ = oracle.egae(r, v, sb, se, tr, None, 1.0, 0.95)
    assert np.all(adv[se - 1] == 0.0)
    adv, _ = oracle.egae(r, v, sb, se, tr, None, 0.9, 0.95)
    np.testing.assert_allclose(adv[se - 1], (0.9 - 1.0) * v[se - 1].astype(float), atol=1e-15)


def test_lambda_zero_is_td_residual_and_outside_is_zero():
    rng = np.random.default_rng(15)
    r, v, sb, se, tr, N = random_case(rng, 6, 20)
    tr[:] = 0
    adv, ret = oracle.egae(r, v, sb, se, tr, None, 0.95, 0.0)
    inside = np.zeros(N, bool)
    for b, e in zip(sb, se):
        inside[b:e] = True
        vn = np.append(v[b + 1:e].astype(float), 0.0)
        np.testing.assert_allclose(adv[b:e], r[b:e] + 0.95 * vn - v[b:e], atol=1e-14)
    assert np.all(adv[~inside] == 0) and np.all(ret[~inside] == 0)


def test_single_terminal_reward_return_is_constant():
    r = np.zeros(10, np.float32)
    r[8] = -1.0
    v = np.zeros(10, np.float32)
    _, ret = oracle.egae(r, v, [2], [9], [0], None, 1.0, 0.95)
    assert np.all(ret[2:9] == -1.0) and ret[9] == 0 and np.all(ret[:2] == 0)


def test_empty_and_length_one_segments():
    r = np.array([0.5, 1.0, 0.25], np.float32)
    v = np.array([0.1, 0.2, 0.3], np.float32)
    adv, ret = oracle.egae(r, v, [0, 1, 2], [1, 1, 3], [0, 1, 1], None, 1.0, 0.95)
    assert adv[0] == pytest.approx(0.5 - np.float32(0.1))
    assert adv[1] == 0.0 and ret[1] == 0.0  # the empty segment selects nothing
    assert adv[2] == pytest.approx(0.25)


@pytest.mark.parametrize("gamma,lam", [(1.0, 0.95), (0.99, 0.9), (1.0, 1.0), (0.9, 0.0)])
def test_advantage_is_lambda_return_minus_value(gamma, lam):
    """A_t + V_t is the lambda-return: G_t = r_t + gamma ((1 - lambda) V_{t+1} + lambda G_{t+1}), with
    G = r + gamma V_next on the last token (V_next = 0, the bootstrap value, or the token's own
    value).  A second, textbook form of the same estimator, evaluated here token by token."""
    rng = np.random.default_rng(11)
    r, v, sb, se, tr, N = random_case(rng, 7, 40)
    boots = rng.standard_normal(7).astype(np.float32)
    for boot in (None, boots):
        adv, _ = oracle.egae(r, v, sb, se, tr, boot, gamma, lam)
        ref = np.zeros(N)
        for i in range(7):
            b, e = int(sb[i]), int(se[i])
            G = 0.0
            for t in range(e - 1, b - 1, -1):
                if t == e - 1:
                    vn = (float(v[t]) if boot is None else float(boot[i])) if tr[i] else 0.0
                    G = float(r[t]) + gamma * vn
                else:
                    G = float(r[t]) + gamma * ((1.0 - lam) * float(v[t + 1]) + lam * G)
                ref[t] = G - float(v[t])
        np.testing.assert_allclose(adv, ref, rtol=1e-11, atol=1e-11)
