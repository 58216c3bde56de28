"""Pins for the oracle's log-prob gather, clipped surrogate (Eq. 1) and value loss (Eq. 4-5)."""
import numpy as np
import pytest
import torch
from scipy.special import logsumexp

import oracle


def make(rng, R=7, V=13, scale=2.0):
    x = (scale * rng.standard_normal((R, V))).astype(np.float32)
    y = rng.integers(0, V, R).astype(np.int32)
    adv = rng.standard_normal(R).astype(np.float32)
    lp = x[np.arange(R), y] - logsumexp(x.astype(np.float64), axis=1)
    old = (lp + 0.25 * rng.standard_normal(R)).astype(np.float32)
    return x, y, adv, old


def test_logprob_against_scipy_and_normalisation():
    rng = np.random.default_rng(0)
    x, y, _, _ = make(rng, 9, 1001, 3.0)
    lp = oracle.logprob(x, y)
    ref = x[np.arange(9), y] - logsumexp(x.astype(np.float64), axis=1)
    np.testing.assert_allclose(lp, ref, rtol=0, atol=1e-12)
    # every column as target: probabilities sum to one
    for r in range(2):
        allp = [oracle.logprob(x[r:r + 1], np.array([v], np.int32))[0] for v in range(0, 1001)]
        assert abs(np.exp(allp).sum() - 1.0) < 1e-12
    # shift invariance and rows / strides
    lp2 = oracle.logprob(x + np.float32(8.0), y)
    np.testing.assert_allclose(lp2, lp, atol=1e-5)
    rows = np.array([5, 0, 8], np.int32)
    np.testing.assert_allclose(oracle.logprob(x, y, rows), ref[rows], atol=1e-12)
    big = np.zeros((9, 1100), np.float32)
    big[:, :1001] = x
    np.testing.assert_allclose(oracle.logprob(big[:, :1001], y), ref, atol=1e-12)


def test_logprob_bf16_and_extremes():
    rng = np.random.default_rng(1)
    xb = torch.from_numpy(2 * rng.standard_normal((4, 64)).astype(np.float32)).to(torch.bfloat16)
    bits = xb.view(torch.int16).numpy().view(np.uint16)
    y = rng.integers(0, 64, 4).astype(np.int32)
    ref = torch.log_softmax(xb.double(), dim=1)[torch.arange(4), torch.from_numpy(y).long()]
    np.testing.assert_allclose(oracle.logprob(bits, y), ref.numpy(), atol=1e-12)
    x = np.full((1, 10), -1e4, np.float32)
    x[0, 3] = 1e4
    assert oracle.logprob(x, np.array([3], np.int32))[0] == pytest.approx(0.0, abs=1e-12)
    assert oracle.logprob(x, np.array([4], np.int32))[0] == pytest.approx(-2e4)


def test_logprob_and_gradient_at_the_largest_magnitudes():
    """Closed forms at the largest finite bf16 / fp32 values, where adding log S to the maximum
    would lose it: a constant row is uniform (log-prob -log V, gradient factor*(1/V - onehot)) and one
    +max among -max is one-hot (log-prob 0, gradient 0)."""
    V = 40
    big = np.float32(3.3895313892515355e38)            # largest finite bf16
    x = np.zeros((3, V), np.float32)
    x[0, :] = big
    x[1, :] = -big
    x[1, 5] = big
    x[2, :] = -big
    y = np.array([7, 5, 0], np.int32)
    lp = oracle.logprob(x, y)
    np.testing.assert_allclose(lp, [-np.log(V), 0.0, -np.log(V)], rtol=0, atol=1e-12)
    adv = np.array([1.0, -1.0, 0.5], np.float32)
    out = oracle.policy_loss(x, y, None, None, lp.astype(np.float32), adv, 0.2, 0.2)
    onehot = np.zeros((3, V))
    onehot[np.arange(3), y] = 1.0
    p = np.stack([np.full(V, 1.0 / V), onehot[1], np.full(V, 1.0 / V)])
    rho = np.exp(lp - lp.astype(np.float32))
    np.testing.assert_allclose(out["dlogits"], (adv * rho / 3)[:, None] * (p - onehot), rtol=1e-12, atol=1e-18)
    # a constant row of float64 logits at 2^100: uniform as well
    np.testing.assert_allclose(oracle.logprob(np.full((1, V), 2.0 ** 100), y[:1]), [-np.log(V)], atol=1e-12)


def test_entropy_and_kl_statistics():
    """Forward-only statistics against torch's float64 softmax (-sum p log p), closed forms (uniform
    row: log V; one-hot row: 0; two equal maxima among -inf: log 2), bounds, shift invariance, and
    the KL estimate against its definition mean(old_logp - logp) with an index map."""
    rng = np.random.default_rng(11)
    R, V = 12, 257
    x = (3.0 * rng.standard_normal((R, V))).astype(np.float32)
    y = rng.integers(0, V, R).astype(np.int32)
    out = oracle.logprob_stats(x, y)
    xt = torch.tensor(x, dtype=torch.float64)
    lp = torch.log_softmax(xt, dim=1)
    ref_h = -(lp.exp() * lp).sum(dim=1).numpy()
    np.testing.assert_allclose(out["entropy"], ref_h, rtol=0, atol=1e-12)
    np.testing.assert_allclose(out["logp"], lp[torch.arange(R), torch.tensor(y).long()].numpy(), atol=1e-12)
    assert abs(out["mean_entropy"] - ref_h.mean()) < 1e-12 and out["mean_kl"] == 0.0
    assert np.all(out["entropy"] > 0) and np.all(out["entropy"] < np.log(V))
    np.testing.assert_allclose(oracle.logprob_stats(x + np.float32(16.0), y)["entropy"], out["entropy"], atol=1e-4)
    # closed forms
    special = np.full((3, V), -np.inf, np.float32)
    special[0, :] = 0.7                       # uniform
    special[1, 5] = 2.0                       # one-hot: every other entry has probability 0
    special[2, [3, 200]] = -1.5               # two equal entries
    h = oracle.logprob_stats(special, np.array([0, 5, 3], np.int32))
    np.testing.assert_allclose(h["entropy"], [np.log(V), 0.0, np.log(2.0)], atol=1e-12)
    np.testing.assert_allclose(h["logp"], [-np.log(V), 0.0, -np.log(2.0)], atol=1e-12)
    # rows, index map and the KL estimate
    rows = np.array([7, 2, 9, 0], np.int32)
    aux = np.array([1, 30, 5, 12], np.int32)
    old = rng.standard_normal(40).astype(np.float32)
    sub = oracle.logprob_stats(x, y, rows, aux, old)
    np.testing.assert_allclose(sub["entropy"], ref_h[rows], atol=1e-12)
    assert abs(sub["mean_kl"] - np.mean(old[aux].astype(np.float64) - sub["logp"])) < 1e-12
    on_policy = out["logp"].astype(np.float32)
    assert abs(oracle.logprob_stats(x, y, None, None, on_policy)["mean_kl"]) < 1e-7
    # bf16 storage
    xb = torch.from_numpy(x).to(torch.bfloat16)
    bits = xb.view(torch.int16).numpy().view(np.uint16)
    lpb = torch.log_softmax(xb.double(), dim=1)
    np.testing.assert_allclose(oracle.logprob_stats(bits, y)["entropy"], -(lpb.exp() * lpb).sum(dim=1).numpy(), atol=1e-12)


def torch_policy_loss(x, y, old, adv, el, eh, denom):
    """Eq. 1 restated with autograd as an independent comparator (float64)."""
    xt = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    lp = torch.log_softmax(xt, dim=1)[torch.arange(len(y)), torch.tensor(y).long()]
    rho = torch.exp(lp - torch.tensor(old, dtype=torch.float64))
    A = torch.tensor(adv, dtype=torch.float64)
    obj = torch.minimum(rho * A, torch.clamp(rho, 1 - el, 1 + eh) * A)
    loss = -(obj.sum() / denom)
    loss.backward()
    return loss.item(), xt.grad.numpy(), (-obj).detach().numpy()


@pytest.mark.parametrize("el,eh", [(0.2, 0.2), (0.2, 0.28), (1e9, 1e9)])
def test_policy_loss_matches_autograd(el, eh):
    rng = np.random.default_rng(2)
    x, y, adv, old = make(rng, 40, 17)
    out = oracle.policy_loss(x, y, None, None, old, adv, el, eh)
    loss, grad, tl = torch_policy_loss(x, y, old, adv, el, eh, 40)
    assert out["loss"] == pytest.approx(loss, rel=1e-12)
    np.testing.assert_allclose(out["token_loss"], tl, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(out["dlogits"], grad, rtol=1e-10, atol=1e-14)
    np.testing.assert_allclose(out["dlogits"].sum(axis=1), 0, atol=1e-14)
    if el < 1:
        assert out["clip_lo"] + out["clip_hi"] > 0          # the case does exercise the clip
        rho = np.exp(out["logp"] - old)
        lo = (rho < 1 - el) & (adv < 0)
        hi = (rho > 1 + eh) & (adv > 0)
        assert out["clip_lo"] == lo.sum() and out["clip_hi"] == hi.sum()
        assert np.all(out["dlogits"][lo | hi] == 0)
    else:
        assert out["clip_lo"] == out["clip_hi"] == 0


def test_policy_loss_finite_differences():
    rng = np.random.default_rng(3)
    x, y, adv, old = make(rng, 5, 8)
    x = x.astype(np.float32)
    out = oracle.policy_loss(x, y, None, None, old, adv, 0.2, 0.28)
    rho = np.exp(out["logp"] - old)
    assert np.all(np.abs(rho - 0.8) > 1e-3) and np.all(np.abs(rho - 1.28) > 1e-3)
    h = 2.0 ** -10          # exactly representable perturbation of fp32 inputs
    for r in range(5):
        for v in range(8):
            xp, xm = x.copy(), x.copy()
            xp[r, v] += h
            xm[r, v] -= h
            assert xp[r, v] - xm[r, v] == 2 * h
            lp = oracle.policy_loss(xp, y, None, None, old, adv, 0.2, 0.28, want_dlogits=False)["loss"]
            lm = oracle.policy_loss(xm, y, None, None, old, adv, 0.2, 0.28, want_dlogits=False)["loss"]
            fd = (lp - lm) / (2 * h)
            assert out["dlogits"][r, v] == pytest.approx(fd, abs=2e-6)


def test_policy_loss_on_policy_special_case_and_indexing():
    rng = np.random.default_rng(4)
    x, y, adv, _ = make(rng, 6, 11)
    lp = oracle.logprob(x, y)
    # old == new (to fp32 rounding): ratio 1, loss = -mean(A), gradient (A/n)(p - onehot)
    out = oracle.policy_loss(x, y, None, None, lp.astype(np.float32), adv, 0.2, 0.2)
    assert out["loss"] == pytest.approx(-adv.astype(float).mean(), rel=1e-6)
    p = np.exp(x.astype(float) - logsumexp(x.astype(float), axis=1, keepdims=True))
    onehot = np.eye(11)[y]
    np.testing.assert_allclose(out["dlogits"], adv[:, None] / 6 * (p - onehot), rtol=1e-6, atol=1e-9)
    # rows / aux_idx / denom
    rows = np.array([4, 1], np.int32)
    aux = np.array([9, 2], np.int32)
    old_big = np.zeros(12, np.float32)
    adv_big = np.zeros(12, np.float32)
    old_big[aux] = lp[rows] + 0.1
    adv_big[aux] = adv[rows]
    o2 = oracle.policy_loss(x, y, rows, aux, old_big, adv_big, 0.2, 0.2, denom=10.0)
    l, g, _ = torch_policy_loss(x[rows], y[rows], old_big[aux], adv_big[aux], 0.2, 0.2, 10.0)
    assert o2["loss"] == pytest.approx(l, rel=1e-12)
    np.testing.assert_allclose(o2["dlogits"], g, rtol=1e-10, atol=1e-14)


def test_policy_loss_tie_on_clip_edge_keeps_gradient():
    x = np.zeros((1, 4), np.float32)
    y = np.array([0], np.int32)
    lp = float(oracle.logprob(x, y)[0])
    old = np.array([lp], np.float32)
    # ratio is exp(lp - fp32(lp)): make eps so that the edge equals the ratio exactly
    rho = np.exp(lp - float(old[0]))
    out = oracle.policy_loss(x, y, None, None, old, np.array([1.0], np.float32), 1 - rho, rho - 1)
    assert out["clip_lo"] == out["clip_hi"] == 0 and np.any(out["dlogits"] != 0)
    out = oracle.policy_loss(x, y, None, None, old, np.zeros(1, np.float32), 0.2, 0.2)
    assert out["loss"] == 0 and np.all(out["dlogits"] == 0)
    out = oracle.policy_loss(x[:0], y[:0], None, None, old, old, 0.2, 0.2)
    assert out["loss"] == 0.0


def torch_value_loss(v, vo, R, idx, xl, xh, denom):
    vt = torch.tensor(v, dtype=torch.float64, requires_grad=True)
    vo = torch.tensor(vo, dtype=torch.float64)
    R = torch.tensor(R, dtype=torch.float64)
    ix = torch.tensor(idx).long()
    vc = torch.maximum(torch.minimum(vt, vo + xh), vo - xl)
    l = 0.5 * torch.maximum((vt - R) ** 2, (vc - R) ** 2)
    loss = l[ix].sum() / denom
    loss.backward()
    return loss.item(), vt.grad.numpy()


@pytest.mark.parametrize("xl,xh", [(0.5, 0.6), (0.05, 0.02), (1e9, 1e9)])
def test_value_loss_matches_autograd_and_fd(xl, xh):
    rng = np.random.default_rng(5)
    N = 60
    v = rng.standard_normal(N).astype(np.float32)
    vo = (v + 0.3 * rng.standard_normal(N)).astype(np.float32)
    R = rng.choice([-1.0, 1.0], N).astype(np.float32)
    idx = np.sort(rng.choice(N, 25, replace=False)).astype(np.int32)
    loss, dv = oracle.value_loss(v, vo, R, idx, xl, xh)
    l, g = torch_value_loss(v, vo, R, idx, xl, xh, 25)
    assert loss == pytest.approx(l, rel=1e-12)
    np.testing.assert_allclose(dv, g, rtol=1e-12, atol=1e-15)
    off = np.ones(N, bool)
    off[idx] = False
    assert np.all(dv[off] == 0)
    if xl > 1e8:
        assert loss == pytest.approx(0.5 * np.mean((v[idx].astype(float) - R[idx]) ** 2), rel=1e-12)
        np.testing.assert_allclose(dv[idx], (v[idx].astype(float) - R[idx]) / 25, rtol=1e-12)
    h = 2.0 ** -12
    for p in idx[:8]:
        vp, vm = v.copy(), v.copy()
        vp[p] += h
        vm[p] -= h
        fd = (oracle.value_loss(vp, vo, R, idx, xl, xh)[0] - oracle.value_loss(vm, vo, R, idx, xl, xh)[0]) / (vp[p] - vm[p])
        kink = min(abs(v[p] - (vo[p] - xl)), abs(v[p] - (vo[p] + xh)))
        if kink > 2 * h:
            assert dv[p] == pytest.approx(fd, abs=1e-4)


def test_value_loss_empty_and_denominator():
    v = np.array([0.3, -0.2], np.float32)
    loss, dv = oracle.value_loss(v, v, v, np.zeros(0, np.int32), 0.5, 0.6)
    assert loss == 0 and np.all(dv == 0)
    loss, dv = oracle.value_loss(v, v, np.zeros(2, np.float32), np.array([1], np.int32), 0.5, 0.6, denom=4.0)
    assert loss == pytest.approx(0.5 * float(v[1]) ** 2 / 4) and dv[1] == pytest.approx(float(v[1]) / 4)


def test_lmhead_rows_equal_matmul():
    rng = np.random.default_rng(6)
    M, K, V = 5, 24, 40
    H = torch.from_numpy(rng.standard_normal((M, K)).astype(np.float32)).to(torch.bfloat16)
    W = torch.from_numpy(0.1 * rng.standard_normal((K, V)).astype(np.float32)).to(torch.bfloat16)
    hb = H.view(torch.int16).numpy().view(np.uint16)
    wb = W.view(torch.int16).numpy().view(np.uint16)
    rows = np.array([3, 0], np.int32)
    x = oracle.lmhead_logits_rows(hb, wb, rows)
    ref = (H.double() @ W.double()).numpy()
    np.testing.assert_allclose(x, ref[rows], rtol=1e-13, atol=1e-13)
    dx = rng.standard_normal((M, V))
    np.testing.assert_allclose(oracle.lmhead_dhidden_rows(dx, wb), dx @ W.double().numpy().T, rtol=1e-12, atol=1e-13)
    cols = [7, 1, 39]
    np.testing.assert_allclose(oracle.lmhead_dweight_cols(hb, dx[:, cols]),
                               (H.double().numpy().T @ dx)[:, cols], rtol=1e-12, atol=1e-13)


def test_float64_logits_give_the_float32_results_on_representable_values():
    """The LM-head tests hand the loss routine float64 logits; on values that float32 holds exactly
    the two input types must agree to the last bit."""
    rng = np.random.default_rng(9)
    n, V = 7, 33
    x32 = rng.standard_normal((n, V)).astype(np.float32)
    t = rng.integers(0, V, n).astype(np.int32)
    old = (-3.0 + 0.1 * rng.standard_normal(n)).astype(np.float32)
    adv = rng.standard_normal(n).astype(np.float32)
    a = oracle.policy_loss(x32, t, None, None, old, adv, 0.2, 0.28)
    b = oracle.policy_loss(x32.astype(np.float64), t, None, None, old, adv, 0.2, 0.28)
    assert a["loss"] == b["loss"] and np.array_equal(a["logp"], b["logp"])
    assert np.array_equal(a["dlogits"], b["dlogits"])
    assert np.array_equal(oracle.logprob(x32, t), oracle.logprob(x32.astype(np.float64), t))
