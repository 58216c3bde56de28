"""GPU parity: CUDA path (through the C ABI) against the float64 oracle, element by element, on
small seeded inputs that still span several tiles, ragged tails and the edge cases."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_15050_b200 import synth
from gpu_util import (DEV, adv_close, dev, run_egae, run_policy, run_select, run_value,
                      worst_relative_error)

pytestmark = pytest.mark.gpu

LOGP_ATOL = 2e-3       # per-token log-probs and losses from bf16 logits, fp32 accumulation
ADV_RTOL = 1e-5        # fp32 advantages


def f32(x):
    return float(np.float32(x))


# ------------------------------------------------------------------------------------------------
# selection
# ------------------------------------------------------------------------------------------------
def check_select(c, tail_drop=0, pm=None, vm=None, tail_drop_seq=None):
    pol, val, cn = run_select(c, tail_drop, pm, vm, tail_drop_seq=tail_drop_seq)
    rp, rv = oracle.select_tokens(c["seq_begin"], c["prompt_len"], c["prev_len"], c["new_len"],
                                  c["truncated"], tail_drop, pm, vm, tail_drop_seq=tail_drop_seq)
    assert cn[2] == 0 and cn[3] == 0
    assert cn[0] == len(rp) and cn[1] == len(rv)
    assert np.array_equal(pol, rp) and np.array_equal(val, rv)
    return cn


def test_select_config1():
    cn = check_select(synth.config1())
    assert cn[0] == 170 and cn[1] == 42


@pytest.mark.parametrize("seed", range(4))
def test_select_random_multi_tile(seed):
    rng = np.random.default_rng(seed)
    B = int(rng.integers(1, 60))
    prompt = rng.integers(0, 300, B)
    prev = rng.integers(0, 500, B) * rng.integers(0, 2, B)
    new = rng.integers(0, 700, B)
    trunc = rng.integers(0, 2, B).astype(np.uint8)
    sb, _, _ = synth.pack(prompt, prev, new)
    c = dict(seq_begin=sb, prompt_len=prompt, prev_len=prev, new_len=new, truncated=trunc)
    N = int(sb[-1])
    check_select(c, tail_drop=int(rng.integers(0, 40)))
    pm = rng.integers(0, 2, max(N, 1)).astype(np.uint8)
    vm = rng.integers(0, 2, max(N, 1)).astype(np.uint8)
    check_select(c, 3, pm, vm)
    check_select(c, 0, pm, None)


def test_select_edge_cases():
    z = np.zeros(1, np.int32)
    # one sequence, everything selected; all truncated; all prompt; empty sequences; tile-aligned end
    for prompt, prev, new, trunc in [([0], [0], [4096], [0]), ([0], [0], [8192], [1]),
                                     ([5000], [0], [0], [0]), ([0, 0, 3], [0, 0, 0], [0, 0, 1], [0, 1, 0]),
                                     ([1], [4094], [1], [0]), ([7], [0], [1], [1])]:
        sb, _, _ = synth.pack(prompt, prev, new)
        c = dict(seq_begin=sb, prompt_len=np.array(prompt), prev_len=np.array(prev),
                 new_len=np.array(new), truncated=np.array(trunc, np.uint8))
        check_select(c)
        check_select(c, tail_drop=2)


def test_select_per_sequence_tail_drop():
    """One count per sequence (Section 3.2 leaves the number of excluded latest tokens open): random
    ragged batches over several tiles, counts larger than a sequence, the array overriding the scalar,
    and a negative entry (read as 0, reported)."""
    for seed in range(3):
        rng = np.random.default_rng(100 + seed)
        B = int(rng.integers(2, 80))
        prompt = rng.integers(0, 300, B)
        prev = rng.integers(0, 500, B) * rng.integers(0, 2, B)
        new = rng.integers(0, 900, B)
        trunc = rng.integers(0, 2, B).astype(np.uint8)
        sb, _, _ = synth.pack(prompt, prev, new)
        c = dict(seq_begin=sb, prompt_len=prompt, prev_len=prev, new_len=new, truncated=trunc)
        N = int(sb[-1])
        td = rng.integers(0, 1000, B).astype(np.int32)
        cn = check_select(c, 5, tail_drop_seq=td)
        assert cn[0] == int(np.sum(np.maximum(0, new - trunc.astype(np.int64) * td)))
        pm = rng.integers(0, 2, max(N, 1)).astype(np.uint8)
        vm = rng.integers(0, 2, max(N, 1)).astype(np.uint8)
        check_select(c, 0, pm, vm, tail_drop_seq=td)
        same = run_select(c, 0, tail_drop_seq=np.full(B, 7, np.int32))
        scalar = run_select(c, 7)
        assert np.array_equal(same[0], scalar[0]) and np.array_equal(same[1], scalar[1])
        if trunc.any():
            neg = td.copy()
            neg[int(np.argmax(trunc))] = -3
            pol, val, cn = run_select(c, 0, tail_drop_seq=neg)
            rp, rv = oracle.select_tokens(sb, prompt, prev, new, trunc, 0, tail_drop_seq=neg)
            assert cn[2] == 4 and np.array_equal(pol, rp) and np.array_equal(val, rv)


def test_select_run_to_run_identical_and_config4():
    c = synth.config4(B=600, hi=32768)
    a1 = run_select(c, 16, c["extra_policy_mask"], c["extra_value_mask"])
    a2 = run_select(c, 16, c["extra_policy_mask"], c["extra_value_mask"])
    assert np.array_equal(a1[0], a2[0]) and np.array_equal(a1[1], a2[1])
    check_select(c, 16, c["extra_policy_mask"], c["extra_value_mask"])
    check_select(c, 0)
    td = np.random.default_rng(7).integers(0, 64, c["B"]).astype(np.int32)
    check_select(c, 0, c["extra_policy_mask"], c["extra_value_mask"], tail_drop_seq=td)


# ------------------------------------------------------------------------------------------------
# EGAE
# ------------------------------------------------------------------------------------------------
def check_egae(B, r, v, sb, se, tr, boot, gamma, lam):
    adv, ret, status = run_egae(B, r, v, sb, se, tr, boot, gamma, lam)
    ra, rr = oracle.egae(r, v, sb, se, tr, boot, f32(gamma), f32(lam))
    assert status == 0
    assert adv_close(adv, ra, sb, se, ADV_RTOL) <= 1.0
    assert adv_close(ret, rr, sb, se, ADV_RTOL) <= 1.0
    print("worst relative error where |exact| >= 1: advantages %.2e, returns %.2e"
          % (worst_relative_error(adv, ra), worst_relative_error(ret, rr)))
    return adv, ret


def test_egae_nonfinite_inputs_are_read_as_zero_and_reported():
    """A NaN / infinite reward or value inside a segment is read as 0 (so every output stays finite
    and equals the oracle's result on the cleaned arrays) and raises the status bit; the same
    garbage outside every segment is ignored."""
    from paper_2506_15050_b200 import binding as b
    rng = np.random.default_rng(61)
    N = 3 * 2048 + 300
    r = rng.standard_normal(N).astype(np.float32)
    v = rng.standard_normal(N).astype(np.float32)
    sb, se = np.array([10, 2500, 5000], np.int32), np.array([2400, 4990, N - 7], np.int32)
    tr = np.array([1, 0, 1], np.uint8)
    boot = np.array([0.3, np.nan, np.inf], np.float32)      # boot[1] belongs to a finished response: unused
    r[2450], v[3], v[N - 2] = np.nan, np.inf, np.nan         # outside every segment: ignored
    adv, ret, st = run_egae(3, r, v, sb, se, tr, np.array([0.3, np.nan, 0.5], np.float32), 0.99, 0.95)
    ra, rr = oracle.egae(r, v, sb, se, tr, np.array([0.3, 0.0, 0.5], np.float32), f32(0.99), f32(0.95))
    assert st == 0 and adv_close(adv, ra, sb, se, ADV_RTOL) <= 1.0 and adv_close(ret, rr, sb, se, ADV_RTOL) <= 1.0
    bad_r, bad_v = r.copy(), v.copy()
    bad_r[100], bad_r[2047], bad_v[2048], bad_v[4989], bad_v[5000] = np.nan, np.inf, -np.inf, np.nan, np.inf
    clean_r, clean_v = bad_r.copy(), bad_v.copy()
    clean_r[[100, 2047]] = 0
    clean_v[[2048, 4989, 5000]] = 0
    for bt in (boot, None):
        adv, ret, st = run_egae(3, bad_r, bad_v, sb, se, tr, bt, 0.99, 0.95)
        clean_boot = None if bt is None else np.array([0.3, 0.0, 0.0], np.float32)
        ra, rr = oracle.egae(clean_r, clean_v, sb, se, tr, clean_boot, f32(0.99), f32(0.95))
        assert st == b.DEV_NONFINITE
        assert np.all(np.isfinite(adv)) and np.all(np.isfinite(ret))
        assert adv_close(adv, ra, sb, se, ADV_RTOL) <= 1.0 and adv_close(ret, rr, sb, se, ADV_RTOL) <= 1.0


def test_lookback_waits_give_up_cleanly():
    """The bounded waits of the two look-back kernels, made to run out on the host's say-so: tiles
    do not publish and a look-back gives up after four polls.  Both calls must come back with
    TPPO_DEV_WAIT_TIMEOUT, finite in-bounds outputs and a usable device; with the hooks cleared the
    same calls are exact again."""
    from paper_2506_15050_b200 import binding as b
    c = synth.config4(B=300)
    try:
        b.tppo_test_hooks(4, True)
        adv, ret, st = run_egae(c["B"], c["rewards"], c["values"], c["seg_begin"], c["seg_end"],
                                c["truncated"], c["bootstrap"], 1.0, 0.95)
        assert st & b.DEV_WAIT_TIMEOUT and np.all(np.isfinite(adv)) and np.all(np.isfinite(ret))
        pol, val, cn = run_select(c, 0, c["extra_policy_mask"], c["extra_value_mask"], strict=False)
        assert cn[2] & b.DEV_WAIT_TIMEOUT
        assert np.all((pol >= 0) & (pol < c["N"])) and np.all((val >= 0) & (val < c["N"]))
    finally:
        b.tppo_test_hooks(-1, False)
    check_egae(c["B"], c["rewards"], c["values"], c["seg_begin"], c["seg_end"], c["truncated"],
               c["bootstrap"], 1.0, 0.95)
    check_select(c, 0, c["extra_policy_mask"], c["extra_value_mask"])


def test_egae_config1_and_truncated_tail_is_zero():
    c = synth.config1()
    adv, ret = check_egae(c["B"], c["rewards"], c["values"], c["seg_begin"], c["seg_end"],
                          c["truncated"], None, c["gamma"], c["lam"])
    for i in (1, 3):   # gamma=1, no reward: the last token of a truncated response has A = 0
        assert adv[c["seg_end"][i] - 1] == 0.0


@pytest.mark.parametrize("gamma,lam", [(1.0, 0.95), (1.0, 1.0), (0.99, 0.9), (0.999, 1.0), (0.9, 0.0)])
def test_egae_random_ragged(gamma, lam):
    rng = np.random.default_rng(5)
    B = 37
    lens = rng.integers(0, 9000, B)
    lens[3] = 2048          # tile-aligned lengths and a length-1 segment
    lens[4] = 4096
    lens[5] = 1
    gaps = rng.integers(0, 50, B)
    sb = np.cumsum(gaps + np.concatenate([[0], lens[:-1]])).astype(np.int32)
    se = (sb + lens).astype(np.int32)
    N = int(se[-1]) + 13
    r = rng.standard_normal(N).astype(np.float32)      # dense (process) rewards
    v = rng.standard_normal(N).astype(np.float32)
    tr = rng.integers(0, 2, B).astype(np.uint8)
    boot = rng.standard_normal(B).astype(np.float32)
    check_egae(B, r, v, sb, se, tr, boot, gamma, lam)
    check_egae(B, r, v, sb, se, tr, None, gamma, lam)


def test_egae_edge_cases():
    rng = np.random.default_rng(6)
    r = rng.standard_normal(5000).astype(np.float32)
    v = rng.standard_normal(5000).astype(np.float32)
    one = lambda *a: np.array(a, np.int32)
    check_egae(1, r, v, one(0), one(5000), np.array([1], np.uint8), None, 1.0, 0.95)   # B = 1
    check_egae(1, r, v, one(0), one(5000), np.array([0], np.uint8), None, 1.0, 1.0)
    check_egae(1, r[:1], v[:1], one(0), one(1), np.array([1], np.uint8), None, 1.0, 0.95)
    check_egae(3, r, v, one(10, 10, 4000), one(10, 2048, 4001), np.array([0, 1, 0], np.uint8), None, 0.97, 0.9)
    adv, ret, st = run_egae(0, r[:100], v[:100], np.zeros(0, np.int32), np.zeros(0, np.int32),
                            np.zeros(0, np.uint8), None, 1.0, 0.95)
    assert st == 0 and np.all(adv == 0) and np.all(ret == 0)
    a1 = run_egae(1, r, v, one(3), one(4999), np.array([1], np.uint8), None, 1.0, 0.95)
    a2 = run_egae(1, r, v, one(3), one(4999), np.array([1], np.uint8), None, 1.0, 0.95)
    assert np.array_equal(a1[0], a2[0]) and np.array_equal(a1[1], a2[1])     # run-to-run identical
    _, _, st = run_egae(1, r, v, one(3), one(6000), np.array([1], np.uint8), None, 1.0, 0.95)
    assert st == 8      # segment end beyond N is reported, not followed


def test_egae_segment_ends_at_every_offset_of_a_run():
    """A thread evaluates sixteen consecutive positions; the end of one segment and the start of the
    next are placed at every offset inside such a run and across the tile edge (2048), with the
    three kinds of boundary value (finished, truncated with and without a bootstrap array)."""
    rng = np.random.default_rng(8)
    N = 3 * 2048 + 77
    r = rng.standard_normal(N).astype(np.float32)
    v = rng.standard_normal(N).astype(np.float32)
    for e1 in list(range(2030, 2067)) + [4095, 4096, 4097]:
        for gap in (0, 1, 5):
            sb = np.array([3, e1 + gap], np.int32)
            se = np.array([e1, N - 2], np.int32)
            boot = rng.standard_normal(2).astype(np.float32)
            for tr in ((0, 1), (1, 0)):
                check_egae(2, r, v, sb, se, np.array(tr, np.uint8), boot, 0.99, 0.95)
            check_egae(2, r, v, sb, se, np.array([1, 1], np.uint8), None, 1.0, 0.95)


def test_egae_long_response_dense_rewards_keeps_the_tolerance():
    """One response of 131072 tokens with a reward on every token and no decay (gamma = lambda = 1,
    and gamma just below 1): sums over the whole response, where single-precision accumulation
    over the length would lose the tolerance."""
    rng = np.random.default_rng(9)
    N = 131072 + 50
    r = (0.5 + rng.standard_normal(N)).astype(np.float32)
    v = rng.standard_normal(N).astype(np.float32)
    sb, se = np.array([20], np.int32), np.array([N - 30], np.int32)
    for gamma, lam in ((1.0, 1.0), (0.9999, 1.0), (1.0, 0.999)):
        check_egae(1, r, v, sb, se, np.array([1], np.uint8), None, gamma, lam)


def test_egae_unaligned_arrays_and_no_returns():
    """Arrays that start off a 16-byte boundary take the plain-load path; returns may be omitted."""
    from paper_2506_15050_b200 import binding as b
    rng = np.random.default_rng(10)
    N, B = 3 * 2048 + 500, 3
    r = rng.standard_normal(N).astype(np.float32)
    v = rng.standard_normal(N).astype(np.float32)
    sb, se = np.array([0, 2500, 5000], np.int32), np.array([2400, 4999, N], np.int32)
    tr = np.array([1, 0, 1], np.uint8)
    ra, rr = oracle.egae(r, v, sb, se, tr, None, f32(1.0), f32(0.95))
    adv, ret, st = run_egae(B, r, v, sb, se, tr, None, 1.0, 0.95, want_returns=False)
    assert st == 0 and ret is None and adv_close(adv, ra, sb, se, ADV_RTOL) <= 1.0
    for off_in, off_out in ((1, 0), (0, 1), (3, 2)):
        rbuf, vbuf = torch.zeros(N + 4, device=DEV), torch.zeros(N + 4, device=DEV)
        rbuf[off_in:off_in + N] = dev(r, torch.float32)
        vbuf[off_in:off_in + N] = dev(v, torch.float32)
        abuf = torch.full((N + 4,), float("nan"), device=DEV)
        gbuf = torch.full((N + 4,), float("nan"), device=DEV)
        status = torch.full((1,), -1, dtype=torch.int32, device=DEV)
        ws = b.workspace(b.OP_EGAE, N, B, 0, 0, DEV)
        b.tppo_egae(rbuf[off_in:off_in + N], vbuf[off_in:off_in + N], dev(sb, torch.int32),
                    dev(se, torch.int32), dev(tr, torch.uint8), None, 1.0, 0.95,
                    abuf[off_out:off_out + N], gbuf[off_out:off_out + N], status, ws)
        torch.cuda.synchronize()
        assert int(status) == 0
        assert adv_close(abuf[off_out:off_out + N].cpu().numpy(), ra, sb, se, ADV_RTOL) <= 1.0
        assert adv_close(gbuf[off_out:off_out + N].cpu().numpy(), rr, sb, se, ADV_RTOL) <= 1.0
        assert torch.isnan(abuf[:off_out]).all() and torch.isnan(abuf[off_out + N:]).all()


@pytest.mark.parametrize("lam", [0.9, 0.95, 1.0])
def test_egae_config4_reduced(lam):
    c = synth.config4(B=400)
    check_egae(c["B"], c["rewards"], c["values"], c["seg_begin"], c["seg_end"], c["truncated"],
               c["bootstrap"], 1.0, lam)


# ------------------------------------------------------------------------------------------------
# policy loss
# ------------------------------------------------------------------------------------------------
def grad_close(gpu, ref, coef_abs, bf16):
    """dlogits tolerance: one rounding of the result (2^-8 relative for bf16, generous for fp32) plus
    the propagated log-prob error, relative to the row's gradient factor."""
    rel = 2.0 ** -7 if bf16 else 1e-4
    tol = rel * np.abs(ref) + 1e-3 * coef_abs[:, None] + 1e-12
    err = np.abs(gpu.astype(np.float64) - ref)
    return float(np.max(err / tol))


def check_policy(logits_t, targets, rows, aux_idx, old_logp, adv, el, eh, denom=0.0, mode=2, hint=0,
                 inplace=False, min_compared=0.9):
    is_bf16 = logits_t.dtype == torch.bfloat16
    host = synth.bf16_bits(logits_t) if is_bf16 else logits_t.cpu().numpy()
    R, V = host.shape
    ref = oracle.policy_loss(host, targets, rows, aux_idx, old_logp, adv, f32(el), f32(eh), f32(denom))
    out = run_policy(logits_t.clone() if inplace else logits_t, targets, rows, aux_idx, old_logp, adv,
                     el, eh, denom, mode, hint, inplace=inplace)
    n = R if rows is None else len(rows)
    assert out["status"] == 0 and out["n"] == n
    np.testing.assert_allclose(out["logp"][:n], ref["logp"], rtol=0, atol=LOGP_ATOL)
    np.testing.assert_allclose(out["token_loss"][:n], ref["token_loss"], rtol=0,
                               atol=LOGP_ATOL * max(1.0, float(np.max(np.abs(adv))) * 2))
    assert abs(out["loss"] - ref["loss"]) <= LOGP_ATOL * max(1.0, float(np.max(np.abs(adv))))
    # Clip decisions are taken in fp32 on the GPU and in float64 by the oracle: a row whose ratio lies
    # within 1e-3 of a clip edge may fall on either side.  Only those rows are left out of the gradient
    # comparison (and they bound the difference of the clip counts); every other row is compared.
    a_idx = aux_idx if aux_idx is not None else (rows if rows is not None else np.arange(R))
    rho = np.exp(ref["logp"] - np.asarray(old_logp, np.float64)[a_idx])
    near_row = (np.abs(rho - (1 - f32(el))) < 1e-3) | (np.abs(rho - (1 + f32(eh))) < 1e-3)
    near = int(near_row.sum())
    keep = np.where(~near_row)[0]
    assert len(keep) >= min_compared * n, "too many rows near a clip edge: the check would be hollow"
    assert abs(out["clip_lo"] - ref["clip_lo"]) <= near and abs(out["clip_hi"] - ref["clip_hi"]) <= near
    if mode != 0:
        g = out["dlogits"].float().cpu().numpy()
        d = f32(denom) if denom > 0 else max(n, 1)
        coef = np.abs(np.asarray(adv, np.float64)[a_idx] * rho / d)
        if mode == 2:
            assert g.shape == (max(n, 1), V)
            gsel = g[:n]
        else:
            sel = np.arange(R) if rows is None else np.asarray(rows)
            gsel = g[sel][:, :V]
            unsel = np.setdiff1d(np.arange(R), sel)
            assert np.all(g[unsel][:, :V] == 0)          # rows that are not selected: exact zeros
        assert grad_close(gsel[keep], ref["dlogits"][keep], coef[keep], is_bf16) <= 1.0
        A = np.asarray(adv, np.float64)[a_idx]
        clipped = np.clip(rho, 1 - f32(el), 1 + f32(eh)) * A < rho * A
        inactive = np.where((clipped | (A == 0)) & ~near_row)[0]
        if len(inactive):
            assert np.all(gsel[inactive] == 0)            # clipped rows: exact zeros
    return out, ref


def policy_inputs(rng, R, V, dtype, scale, n_aux=None):
    x = (scale * rng.standard_normal((R, V))).astype(np.float32)
    xt = torch.from_numpy(x).to(dtype).to(DEV)
    host = synth.bf16_bits(xt) if dtype == torch.bfloat16 else x
    y = rng.integers(0, V, R).astype(np.int32)
    y[0], y[-1] = 0, V - 1
    lp = oracle.logprob(host, y)
    n_aux = R if n_aux is None else n_aux
    return xt, y, lp


def test_policy_config1_fp32():
    c = synth.config1()
    xt = torch.from_numpy(c["logits"]).to(DEV)
    pol, _ = oracle.select_tokens(c["seq_begin"], c["prompt_len"], c["prev_len"], c["new_len"], c["truncated"])
    adv, _ = oracle.egae(c["rewards"], c["values"], c["seg_begin"], c["seg_end"], c["truncated"], None, 1.0, f32(0.95))
    old = (oracle.logprob(c["logits"], c["targets"]) + c["old_logp_noise"]).astype(np.float32)
    for mode in (0, 1, 2):
        out, ref = check_policy(xt, c["targets"], pol, None, old, adv.astype(np.float32), 0.2, 0.2, mode=mode)
    assert out["n"] == 170
    check_policy(xt, c["targets"], pol, None, old, adv.astype(np.float32), 0.2, 0.2, mode=1, inplace=True)


@pytest.mark.parametrize("hint", [1, 2])
@pytest.mark.parametrize("mode", [0, 1, 2])
def test_policy_bf16_qwen_vocab(hint, mode):
    """V = 152064 with few rows: several rows per cluster, every cluster rank, both kernels."""
    rng = np.random.default_rng(10 + mode)
    R, V = 330, 152064
    xt, y, lp = policy_inputs(rng, R, V, torch.bfloat16, 2.0)
    rows = np.sort(rng.choice(R, 301, replace=False)).astype(np.int32)
    y[rows[1]] = 38016          # first element of the second slice of a 4-CTA cluster
    y[rows[2]] = 38015
    lp = oracle.logprob(synth.bf16_bits(xt), y)
    old = (lp + 0.15 * rng.standard_normal(R)).astype(np.float32)       # some ratios leave the clip range
    adv = rng.standard_normal(R).astype(np.float32)
    out, ref = check_policy(xt, y, rows, None, old, adv, 0.2, 0.28, mode=mode, hint=hint)
    assert ref["clip_lo"] > 0 and ref["clip_hi"] > 0


@pytest.mark.parametrize("variant,V", [(2, 65536), (4, 152064), (8, 152064), (4 | (1 << 4), 152064),
                                       (4 | (2 << 4), 152064), (8 | (3 << 4), 100000), (4 | 128, 152064),
                                       (4 | 128 | (1 << 4), 152064), (8 | 128 | (2 << 4), 152064),
                                       (2 | 128, 50000)])
def test_policy_cluster_variants_inplace(variant, V):
    """Cluster sizes 2 / 4 / 8, capped stage counts and the bulk-store output path (bit 7) are tuning
    variants of one kernel and give the same result."""
    rng = np.random.default_rng(20)
    R = 200
    xt, y, lp = policy_inputs(rng, R, V, torch.bfloat16, 2.0)
    old = (lp + 0.05 * rng.standard_normal(R)).astype(np.float32)
    adv = rng.standard_normal(R).astype(np.float32)
    check_policy(xt, y, None, None, old, adv, 0.2, 0.2, mode=1, hint=2 | (variant << 8), inplace=True)


@pytest.mark.parametrize("V,ld,dtype,hint", [(1001, 1001, torch.bfloat16, 0), (1001, 1008, torch.float32, 0),
                                             (4096, 4096, torch.bfloat16, 2), (32000, 32768, torch.bfloat16, 2),
                                             (32000, 32768, torch.bfloat16, 1), (50264, 50264, torch.bfloat16, 0),
                                             (1000, 1000, torch.float32, 1)])
def test_policy_shapes(V, ld, dtype, hint):
    rng = np.random.default_rng(30)
    R = 70
    x = (2 * rng.standard_normal((R, ld))).astype(np.float32)
    full = torch.from_numpy(x).to(dtype).to(DEV)
    xt = full[:, :V]
    host = (synth.bf16_bits(full) if dtype == torch.bfloat16 else x)[:, :V]
    y = rng.integers(0, V, R).astype(np.int32)
    y[0], y[1] = 0, V - 1
    rows = np.sort(rng.choice(R, 50, replace=False)).astype(np.int32)
    aux = rng.permutation(90)[:50].astype(np.int32)
    lp = oracle.logprob(host, y, rows)
    old = np.zeros(90, np.float32)
    adv = np.zeros(90, np.float32)
    old[aux] = lp + 0.1 * rng.standard_normal(50)
    adv[aux] = rng.standard_normal(50)
    for mode in (1, 2):
        is_bf16 = dtype == torch.bfloat16
        ref = oracle.policy_loss(host, y, rows, aux, old, adv, f32(0.2), f32(0.2), f32(64.0))
        out = run_policy(xt, y, rows, aux, old, adv, 0.2, 0.2, 64.0, mode, hint, V=V)
        assert out["status"] == 0 and out["n"] == 50
        np.testing.assert_allclose(out["logp"][:50], ref["logp"], atol=LOGP_ATOL)
        assert abs(out["loss"] - ref["loss"]) <= LOGP_ATOL
        g = out["dlogits"].float().cpu().numpy()
        rho = np.exp(ref["logp"] - old[aux])
        coef = np.abs(adv[aux] * rho / 64.0)
        gsel = g[:50] if mode == 2 else g[rows][:, :V]
        keep = ~((np.abs(rho - 0.8) < 1e-3) | (np.abs(rho - 1.2) < 1e-3))     # rows off the clip edges
        assert keep.sum() >= 45
        assert grad_close(gsel[keep], ref["dlogits"][keep], coef[keep], is_bf16) <= 1.0


BF16_MAX = 3.3895313892515355e38      # largest finite bf16


def test_policy_overflow_safety_and_onehot_row():
    """Logits at the largest finite bf16 magnitude: exp(x - max) is formed from the difference, so
    nothing overflows on the way.  Rows: all +max (uniform), one +max among -max (one-hot, logp 0),
    all -max (uniform), a wide ramp, and -inf entries (masked vocabulary) beside ordinary ones."""
    V = 8192
    x = np.zeros((6, V), np.float32)
    x[0, :] = BF16_MAX
    x[1, :] = -BF16_MAX
    x[1, 5] = BF16_MAX
    x[2, :] = -BF16_MAX
    x[3, :] = np.linspace(-80, 80, V)
    x[4, :] = np.linspace(-3, 3, V)
    x[4, 100:4000] = -np.inf
    x[5, :] = 1.0e4
    x[5, 6:] = -3.0e4
    xt = torch.from_numpy(x).to(torch.bfloat16).to(DEV)
    assert float(xt[0, 0]) == BF16_MAX and float(xt[2, 0]) == -BF16_MAX
    y = np.array([7, 5, 0, V - 1, 50, 3], np.int32)
    host = synth.bf16_bits(xt)
    lp = oracle.logprob(host, y)
    assert abs(lp[0] + np.log(V)) < 1e-9 and abs(lp[1]) < 1e-9 and abs(lp[2] + np.log(V)) < 1e-9
    old = lp.astype(np.float32)
    adv = np.array([1.0, -1.0, 0.5, 2.0, -0.7, 1.5], np.float32)
    for hint in (1, 2):
        out, ref = check_policy(xt, y, None, None, old, adv, 0.2, 0.2, mode=2, hint=hint)
        g = out["dlogits"].float().cpu().numpy()
        assert np.all(np.isfinite(g)) and np.all(g[4, 100:4000] == 0)


@pytest.mark.parametrize("hint", [1, 2])
def test_policy_nonfinite_rows_are_skipped_and_reported(hint):
    """A row with a NaN or +inf logit, or with nothing but -inf, has no log-softmax: it contributes
    nothing (loss term 0, zero gradient row), raises the status bit, and leaves the other rows alone."""
    from paper_2506_15050_b200 import binding as b
    rng = np.random.default_rng(77)
    R, V = 9, 8192
    x = (2 * rng.standard_normal((R, V))).astype(np.float32)
    x[1, 4000] = np.nan
    x[3, 17] = np.inf
    x[6, :] = -np.inf
    xt = torch.from_numpy(x).to(torch.bfloat16).to(DEV)
    y = rng.integers(0, V, R).astype(np.int32)
    good = np.array([0, 2, 4, 5, 7, 8], np.int32)
    host = synth.bf16_bits(xt)
    lp = np.zeros(R)
    lp[good] = oracle.logprob(host, y, good)
    old = (lp + 0.05 * rng.standard_normal(R)).astype(np.float32)
    adv = rng.standard_normal(R).astype(np.float32)
    out = run_policy(xt, y, None, None, old, adv, 0.2, 0.2, 0.0, 2, hint)
    assert out["status"] == b.DEV_NONFINITE and out["n"] == R
    ref = oracle.policy_loss(host, y, good, None, old, adv, f32(0.2), f32(0.2), float(R))
    g = out["dlogits"].float().cpu().numpy()
    assert np.all(np.isfinite(g)) and np.isfinite(out["loss"])
    bad = np.setdiff1d(np.arange(R), good)
    assert np.all(g[bad] == 0) and np.all(out["logp"][bad] == 0) and np.all(out["token_loss"][bad] == 0)
    np.testing.assert_allclose(out["logp"][good], ref["logp"], rtol=0, atol=LOGP_ATOL)
    assert abs(out["loss"] - ref["loss"]) <= LOGP_ATOL
    rho = np.exp(ref["logp"] - old[good])
    coef = np.abs(adv[good] * rho / R)
    assert grad_close(g[good], ref["dlogits"], coef, True) <= 1.0


@pytest.mark.parametrize("hint", [1, 2])
def test_policy_zero_selected_and_device_count(hint):
    rng = np.random.default_rng(40)
    R, V = 40, 8192
    xt, y, lp = policy_inputs(rng, R, V, torch.bfloat16, 2.0)
    old = lp.astype(np.float32)
    adv = rng.standard_normal(R).astype(np.float32)
    rows = np.arange(0, R, 2).astype(np.int32)
    out = run_policy(xt, y, rows, None, old, adv, 0.2, 0.2, 0.0, 1, hint, n_sel=0)
    assert out["n"] == 0 and out["loss"] == 0.0 and out["status"] == 0
    assert np.all(out["dlogits"].float().cpu().numpy() == 0)     # FULL mode: every row zero-filled
    # device-side count smaller than the list capacity
    out = run_policy(xt, y, rows, None, old, adv, 0.2, 0.2, 0.0, 1, hint, n_sel=7)
    ref = oracle.policy_loss(synth.bf16_bits(xt), y, rows[:7], None, old, adv, f32(0.2), f32(0.2))
    assert out["n"] == 7 and abs(out["loss"] - ref["loss"]) < LOGP_ATOL
    g = out["dlogits"].float().cpu().numpy()
    assert np.all(g[np.setdiff1d(np.arange(R), rows[:7])] == 0)
    # bad target / bad row are reported and skipped
    y2 = y.copy()
    y2[rows[2]] = V
    rows2 = rows.copy()
    rows2[4] = R + 5
    out = run_policy(xt, y2, rows2, None, old, adv, 0.2, 0.2, 0.0, 2, hint)
    assert out["status"] == (1 | 4)
    keep = np.array([k for k in range(len(rows)) if k not in (2, 4)])
    ref = oracle.policy_loss(synth.bf16_bits(xt), y, rows[keep], None, old, adv, f32(0.2), f32(0.2), f32(len(rows)))
    assert abs(out["loss"] - ref["loss"]) < LOGP_ATOL
    g = out["dlogits"].float().cpu().numpy()
    assert np.all(g[2] == 0) and np.all(g[4] == 0) and np.all(np.isfinite(g))


def test_policy_run_to_run_identical():
    rng = np.random.default_rng(41)
    R, V = 300, 152064
    xt, y, lp = policy_inputs(rng, R, V, torch.bfloat16, 2.0)
    old = (lp + 0.05 * rng.standard_normal(R)).astype(np.float32)
    adv = rng.standard_normal(R).astype(np.float32)
    a = run_policy(xt, y, None, None, old, adv, 0.2, 0.2, 0.0, 2, 0)
    b = run_policy(xt, y, None, None, old, adv, 0.2, 0.2, 0.0, 2, 0)
    assert a["loss"] == b["loss"] and np.array_equal(a["logp"], b["logp"])
    assert torch.equal(a["dlogits"], b["dlogits"])


def test_policy_rejects_bad_arguments():
    from paper_2506_15050_b200 import binding as b
    xt = torch.zeros((4, 64), dtype=torch.bfloat16, device=DEV)
    y = np.zeros(4, np.int32)
    z = np.zeros(4, np.float32)
    with pytest.raises(b.TppoError) as e:
        run_policy(xt, y, None, None, z, z, -0.1, 0.2)
    assert e.value.status == 1
    with pytest.raises(b.TppoError) as e:
        run_policy(xt, y, None, None, z, z, 0.2, 0.2, hint=2)       # V too small for the cluster kernel
    assert e.value.status == 3
    ws = torch.empty(16, dtype=torch.uint8, device=DEV)
    with pytest.raises(b.TppoError) as e:
        b.tppo_policy_loss_fwd_bwd(xt, dev(y), None, None, 4, None, dev(z), dev(z), 0.2, 0.2, 0.0, None, None,
                                   torch.zeros(1, device=DEV), torch.zeros(4, dtype=torch.int32, device=DEV),
                                   None, 0, ws)
    assert e.value.status == 2


# ------------------------------------------------------------------------------------------------
# value loss
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("xl,xh", [(0.5, 0.6), (0.05, 0.02)])
def test_value_loss(xl, xh):
    rng = np.random.default_rng(50)
    N = 70000
    v = rng.standard_normal(N).astype(np.float32)
    vo = (v + 0.3 * rng.standard_normal(N)).astype(np.float32)
    R = rng.choice([-1.0, 1.0], N).astype(np.float32)
    idx = np.sort(rng.choice(N, 41234, replace=False)).astype(np.int32)
    loss, dv, n, st = run_value(v, vo, R, idx, xl, xh)
    rl, rdv = oracle.value_loss(v, vo, R, idx, f32(xl), f32(xh))
    assert n == len(idx) and st == 0
    assert abs(loss - rl) <= 1e-5 * max(1.0, abs(rl))
    # the clip bound is rounded in fp32 on the GPU: tokens within an ulp of a bound may switch branch
    edge = (np.abs(v - (vo - f32(xl))) < 1e-6) | (np.abs(v - (vo + f32(xh))) < 1e-6)
    np.testing.assert_allclose(dv[~edge], rdv[~edge], rtol=1e-5, atol=1e-9)
    loss2, dv2, _, _ = run_value(v, vo, R, idx, xl, xh)
    assert loss2 == loss and np.array_equal(dv, dv2)
    loss3, dv3, n3, _ = run_value(v, vo, R, idx, xl, xh, denom=1000.0, n_sel=100)
    rl3, rdv3 = oracle.value_loss(v, vo, R, idx[:100], f32(xl), f32(xh), 1000.0)
    assert n3 == 100 and abs(loss3 - rl3) <= 1e-6
    np.testing.assert_allclose(dv3[~edge], rdv3[~edge], rtol=1e-5, atol=1e-9)
    loss4, dv4, n4, _ = run_value(v, vo, R, idx, xl, xh, n_sel=0)
    assert loss4 == 0 and n4 == 0 and np.all(dv4 == 0)
    bad = idx.copy()
    bad[5] = N + 3
    _, dv5, _, st5 = run_value(v, vo, R, bad, xl, xh)
    assert st5 == 4 and np.all(np.isfinite(dv5))


def test_value_loss_nonfinite_tokens_and_list_forms():
    from paper_2506_15050_b200 import binding as b
    rng = np.random.default_rng(52)
    N = 30000
    v = rng.standard_normal(N).astype(np.float32)
    vo = (v + 0.3 * rng.standard_normal(N)).astype(np.float32)
    R = rng.choice([-1.0, 1.0], N).astype(np.float32)
    idx = np.sort(rng.choice(N, 12000, replace=False)).astype(np.int32)
    bad_tok = idx[[5, 4000, 11999]]
    v2, vo2, R2 = v.copy(), vo.copy(), R.copy()
    v2[bad_tok[0]], vo2[bad_tok[1]], R2[bad_tok[2]] = np.nan, np.inf, -np.inf
    off = np.setdiff1d(np.arange(N), idx)
    v2[off[7]] = np.nan                                     # not a value token: ignored
    keep = np.setdiff1d(idx, bad_tok).astype(np.int32)
    for want_grad in (True, False):
        loss, dv, n, st = run_value(v2, vo2, R2, idx, 0.5, 0.6, want_grad=want_grad)
        rl, rdv = oracle.value_loss(v, vo, R, keep, f32(0.5), f32(0.6), denom=float(len(idx)))
        assert st == b.DEV_NONFINITE and n == len(idx) and abs(loss - rl) <= 1e-5 * max(1.0, abs(rl))
        if want_grad:
            assert np.all(np.isfinite(dv)) and np.all(dv[bad_tok] == 0) and np.all(dv[off] == 0)
            np.testing.assert_allclose(dv[keep], rdv[keep], rtol=1e-5, atol=1e-9)
    # the list may come in any order (distinct entries)
    perm = rng.permutation(idx).astype(np.int32)
    rl, rdv = oracle.value_loss(v, vo, R, idx, f32(0.5), f32(0.6))
    for want_grad in (True, False):
        loss_p, dv_p, _, st_p = run_value(v, vo, R, perm, 0.5, 0.6, want_grad=want_grad)
        assert st_p == 0 and abs(loss_p - rl) <= 1e-5 * max(1.0, abs(rl))
        if want_grad:
            np.testing.assert_allclose(dv_p, rdv, rtol=1e-5, atol=1e-9)
    # no list: the first n positions; unaligned arrays take the element-wise path
    loss_i, dv_i, n_i, st_i = run_value(v, vo, R, None, 0.5, 0.6, n_sel=777)
    rl_i, rdv_i = oracle.value_loss(v, vo, R, np.arange(777, dtype=np.int32), f32(0.5), f32(0.6))
    assert st_i == 0 and n_i == 777 and abs(loss_i - rl_i) <= 1e-5
    np.testing.assert_allclose(dv_i, rdv_i, rtol=1e-5, atol=1e-9)


def test_value_loss_unaligned_arrays_and_tile_edges():
    """Dense and sparse lists over several thousand positions, the whole array selected, and arrays
    that start off a 16-byte boundary."""
    from paper_2506_15050_b200 import binding as b
    rng = np.random.default_rng(53)
    T = 4032
    N = 5 * T + 17
    v = rng.standard_normal(N).astype(np.float32)
    vo = (v + 0.3 * rng.standard_normal(N)).astype(np.float32)
    R = rng.standard_normal(N).astype(np.float32)
    edges = np.concatenate([[k * T - 1, k * T, k * T + 1] for k in range(1, 6)])
    idx = np.unique(np.concatenate([[0, N - 1], edges[edges < N], rng.choice(N, 900, replace=False)])).astype(np.int32)
    for sel in (idx, idx[idx < 2 * T], np.arange(N, dtype=np.int32), np.arange(T, 2 * T, dtype=np.int32)):
        loss, dv, n, st = run_value(v, vo, R, sel, 0.5, 0.6)
        rl, rdv = oracle.value_loss(v, vo, R, sel, f32(0.5), f32(0.6))
        assert st == 0 and n == len(sel) and abs(loss - rl) <= 1e-5 * max(1.0, abs(rl))
        np.testing.assert_allclose(dv, rdv, rtol=1e-5, atol=1e-9)
    # unaligned views
    buf = [torch.zeros(N + 4, device=DEV) for _ in range(4)]
    for off in (1, 3):
        for t_, h in zip(buf[:3], (v, vo, R)):
            t_[off:off + N] = dev(h, torch.float32)
        buf[3].fill_(float("nan"))
        loss_t = torch.zeros(1, device=DEV)
        stats = torch.zeros(2, dtype=torch.int32, device=DEV)
        ws = b.workspace(b.OP_VALUE_LOSS, N, 0, len(idx), 0, DEV)
        b.tppo_value_loss(buf[0][off:off + N], buf[1][off:off + N], buf[2][off:off + N], dev(idx, torch.int32),
                          None, len(idx), 0.5, 0.6, 0.0, loss_t, buf[3][off:off + N], stats, ws)
        torch.cuda.synchronize()
        rl, rdv = oracle.value_loss(v, vo, R, idx, f32(0.5), f32(0.6))
        assert int(stats[1]) == 0 and abs(float(loss_t) - rl) <= 1e-5 * max(1.0, abs(rl))
        np.testing.assert_allclose(buf[3][off:off + N].cpu().numpy(), rdv, rtol=1e-5, atol=1e-9)
        assert torch.isnan(buf[3][:off]).all() and torch.isnan(buf[3][off + N:]).all()


def test_value_loss_config1():
    c = synth.config1()
    _, ret = oracle.egae(c["rewards"], c["values"], c["seg_begin"], c["seg_end"], c["truncated"], None, 1.0, f32(0.95))
    _, val = oracle.select_tokens(c["seq_begin"], c["prompt_len"], c["prev_len"], c["new_len"], c["truncated"])
    loss, dv, n, st = run_value(c["values"], c["old_values"], ret.astype(np.float32), val, 0.5, 0.6)
    rl, rdv = oracle.value_loss(c["values"], c["old_values"], ret.astype(np.float32), val, f32(0.5), f32(0.6))
    assert n == 42 and abs(loss - rl) < 1e-6
    np.testing.assert_allclose(dv, rdv, rtol=1e-5, atol=1e-9)


# ------------------------------------------------------------------------------------------------
# many tiny sequences: more sequence starts per tile than the kernels keep in shared memory, so the
# paths that search the global arrays run
# ------------------------------------------------------------------------------------------------
def test_select_and_egae_many_tiny_sequences():
    rng = np.random.default_rng(12)
    B = 6000
    prompt = rng.integers(0, 3, B)
    prev = rng.integers(0, 3, B) * rng.integers(0, 2, B)
    new = rng.integers(0, 6, B)
    trunc = rng.integers(0, 2, B).astype(np.uint8)
    sb, seg_b, seg_e = synth.pack(prompt, prev, new)
    N = int(sb[-1])
    assert B / max(N // 4096, 1) > 400           # several hundred sequences per 4096-position tile
    c = dict(seq_begin=sb, prompt_len=prompt, prev_len=prev, new_len=new, truncated=trunc)
    pm = rng.integers(0, 2, N).astype(np.uint8)
    vm = rng.integers(0, 2, N).astype(np.uint8)
    check_select(c, tail_drop=1)
    check_select(c, 2, pm, vm)
    r = rng.standard_normal(N).astype(np.float32)
    v = rng.standard_normal(N).astype(np.float32)
    boot = rng.standard_normal(B).astype(np.float32)
    check_egae(B, r, v, seg_b, seg_e, trunc, boot, 0.99, 0.95)
    check_egae(B, r, v, seg_b, seg_e, trunc, None, 1.0, 1.0)


# more sequences than the clearing kernels stage in shared memory (12288 segments for the scan,
# 24575 sequence starts for the selection): their window searches then read the global arrays
def test_select_and_egae_more_sequences_than_the_clearing_kernels_stage():
    rng = np.random.default_rng(21)
    B = 26000
    prompt = rng.integers(0, 4, B)
    prev = rng.integers(0, 5, B) * rng.integers(0, 2, B)
    new = rng.integers(0, 24, B)
    trunc = rng.integers(0, 2, B).astype(np.uint8)
    sb, seg_b, seg_e = synth.pack(prompt, prev, new)
    N = int(sb[-1])
    assert N > 8 * 8192                          # several tiles of either kernel
    c = dict(seq_begin=sb, prompt_len=prompt, prev_len=prev, new_len=new, truncated=trunc)
    pm = rng.integers(0, 2, N).astype(np.uint8)
    vm = rng.integers(0, 2, N).astype(np.uint8)
    check_select(c, tail_drop=2)
    check_select(c, 1, pm, vm)
    r = rng.standard_normal(N).astype(np.float32)
    v = rng.standard_normal(N).astype(np.float32)
    boot = rng.standard_normal(B).astype(np.float32)
    check_egae(B, r, v, seg_b, seg_e, trunc, boot, 0.99, 0.95)
    check_egae(B, r, v, seg_b, seg_e, trunc, None, 1.0, 0.9)
