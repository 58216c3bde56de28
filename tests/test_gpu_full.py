"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration that
bench.py times: every integer output bit-exact, every advantage / return / log-prob / loss checked,
gradients checked on sampled rows against the oracle (which computes them one row at a time)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_15050_b200 import synth
from gpu_util import DEV, adv_close, dev, run_egae, run_select, run_value

pytestmark = pytest.mark.gpu
f32 = lambda x: float(np.float32(x))
LOGP_ATOL = 2e-3


def test_config4_full_egae_and_compaction():
    c = synth.config4()
    assert c["B"] == 4096 and c["N"] > 15_000_000
    for lam in c["lams"]:
        adv, ret, st = run_egae(c["B"], c["rewards"], c["values"], c["seg_begin"], c["seg_end"],
                                c["truncated"], c["bootstrap"], 1.0, lam)
        ra, rr = oracle.egae(c["rewards"], c["values"], c["seg_begin"], c["seg_end"], c["truncated"],
                             c["bootstrap"], 1.0, f32(lam))
        assert st == 0
        assert adv_close(adv, ra, c["seg_begin"], c["seg_end"], 1e-5) <= 1.0
        assert adv_close(ret, rr, c["seg_begin"], c["seg_end"], 1e-5) <= 1.0
    for td in c["tail_drops"]:
        pol, val, cn = run_select(c, td, c["extra_policy_mask"], c["extra_value_mask"])
        rp, rv = oracle.select_tokens(c["seq_begin"], c["prompt_len"], c["prev_len"], c["new_len"],
                                      c["truncated"], td, c["extra_policy_mask"], c["extra_value_mask"])
        assert cn[2] == 0 and np.array_equal(pol, rp) and np.array_equal(val, rv)
    pol, val, cn = run_select(c, 16)
    rp, rv = oracle.select_tokens(c["seq_begin"], c["prompt_len"], c["prev_len"], c["new_len"],
                                  c["truncated"], 16)
    assert np.array_equal(pol, rp) and np.array_equal(val, rv)
    assert cn[0] == int(np.sum(np.maximum(0, c["new_len"].astype(np.int64) - 16 * c["truncated"])))


def policy_full(c, logits, rows, aux, old_logp, adv, n_sel_t, mode, inplace=False, hint=0):
    from paper_2506_15050_b200 import binding as b
    R, V = logits.shape
    n_max = R if rows is None else len(rows)
    t = lambda a, dt: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(dt).to(DEV)
    logp = torch.full((n_max,), float("nan"), device=DEV)
    tl = torch.full((n_max,), float("nan"), device=DEV)
    loss = torch.zeros(1, device=DEV)
    stats = torch.zeros(4, dtype=torch.int32, device=DEV)
    if mode == b.DLOGITS_FULL:
        dl = logits if inplace else torch.empty_like(logits)
    else:
        dl = torch.empty((n_max, V), dtype=logits.dtype, device=DEV)
    ws = b.workspace(b.OP_POLICY_LOSS, R, 0, n_max, V, DEV)
    b.tppo_policy_loss_fwd_bwd(logits, t(c["targets"], torch.int32), t(rows, torch.int32), n_sel_t, n_max,
                               t(aux, torch.int32), t(old_logp, torch.float32), t(adv, torch.float32),
                               c["eps_low"], c["eps_high"], 0.0, logp, tl, loss, stats, dl, mode, ws,
                               kernel_hint=hint)
    torch.cuda.synchronize()
    return logp.cpu().numpy(), tl.cpu().numpy(), float(loss), stats.cpu().numpy(), dl


def check_sampled_gradient(dl_rows_gpu, host_logits, c, rows_s, aux_s, old_logp, adv, denom):
    ref = oracle.policy_loss(host_logits, c["targets"], rows_s, aux_s, old_logp, adv,
                             f32(c["eps_low"]), f32(c["eps_high"]), float(denom))
    g = dl_rows_gpu.float().cpu().numpy()
    a_idx = aux_s if aux_s is not None else rows_s
    rho = np.exp(ref["logp"] - old_logp[a_idx].astype(np.float64))
    coef = np.abs(adv[a_idx].astype(np.float64) * rho / denom)
    near = (np.abs(rho - (1 - f32(c["eps_low"]))) < 1e-3) | (np.abs(rho - (1 + f32(c["eps_high"]))) < 1e-3)
    tol = 2.0 ** -7 * np.abs(ref["dlogits"]) + 1e-3 * coef[:, None] + 1e-12
    err = np.abs(g - ref["dlogits"]) / tol
    assert float(err[~near].max()) <= 1.0
    np.testing.assert_allclose(g[~near].sum(axis=1), 0, atol=2e-2 * coef[~near].max())
    return ref


@pytest.mark.parametrize("mode", [1, 2])
def test_config2_full(mode):
    """[8192, 152064] bf16, 4096 selected rows given by the device-side selection (row list +
    device count); FULL (zero-filled) and COMPACT gradients."""
    c = synth.config2(DEV)
    assert c["logits"].shape == (8192, 152064)
    N, B = c["N"], c["B"]
    adv, ret, st = run_egae(B, c["rewards"], c["values"], c["seg_begin"], c["seg_end"], c["truncated"],
                            None, c["gamma"], c["lam"])
    ra, _ = oracle.egae(c["rewards"], c["values"], c["seg_begin"], c["seg_end"], c["truncated"], None,
                        f32(c["gamma"]), f32(c["lam"]))
    assert adv_close(adv, ra, c["seg_begin"], c["seg_end"], 1e-5) <= 1.0
    pol, val, cn = run_select(c)
    rp, rv = oracle.select_tokens(c["seq_begin"], c["prompt_len"], c["prev_len"], c["new_len"], c["truncated"])
    assert np.array_equal(pol, rp) and np.array_equal(val, rv) and len(rp) == 4096
    host = synth.bf16_bits(c["logits"])
    adv32 = ra.astype(np.float32)
    lp_all = oracle.logprob(host, c["targets"], rp)
    old = np.zeros(N, np.float32)
    old[rp] = lp_all + c["old_logp_noise"][rp]
    # capacity N, count on the device, as the selection kernel leaves them
    rows_cap = np.zeros(N, np.int32)
    rows_cap[:len(rp)] = rp
    n_sel = torch.tensor([len(rp)], dtype=torch.int32, device=DEV)
    logp, tl, loss, stats, dl = policy_full(c, c["logits"], rows_cap, None, old, adv32, n_sel, mode)
    ref = oracle.policy_loss(host, c["targets"], rp, None, old, adv32, f32(c["eps_low"]), f32(c["eps_high"]),
                             want_dlogits=False)
    assert stats[0] == 4096 and stats[3] == 0
    np.testing.assert_allclose(logp[:4096], ref["logp"], rtol=0, atol=LOGP_ATOL)
    np.testing.assert_allclose(tl[:4096], ref["token_loss"], rtol=0, atol=LOGP_ATOL * 4)
    assert abs(loss - ref["loss"]) <= LOGP_ATOL
    assert abs(int(stats[1]) - ref["clip_lo"]) <= 2 and abs(int(stats[2]) - ref["clip_hi"]) <= 2
    rng = np.random.default_rng(0)
    pick = np.sort(rng.choice(4096, 192, replace=False))
    pick[0], pick[-1] = 0, 4095
    g_rows = dl[torch.from_numpy(rp[pick]).long().to(DEV)] if mode == 1 else dl[torch.from_numpy(pick).long().to(DEV)]
    check_sampled_gradient(g_rows, host, c, rp[pick], None, old, adv32, 4096)
    if mode == 1:
        unsel = np.setdiff1d(np.arange(N), rp)
        assert float(dl[torch.from_numpy(unsel).long().to(DEV)].float().abs().max()) == 0.0


@pytest.mark.parametrize("inplace", [False, True])
def test_config3_full(inplace):
    """The headline configuration: EGAE and selection over the 512-response batch, then the
    [16384, 152064] bf16 micro-batch with identity rows, aux_idx = selected positions and the
    device-side count -- compact gradient into a second buffer (as timed), and in place."""
    from paper_2506_15050_b200 import binding as b
    c = synth.config3(DEV)
    N, B, n = c["N"], c["B"], c["n_tokens"]
    assert n == 16384 and c["logits"].shape == (16384, 152064)
    adv, ret, st = run_egae(B, c["rewards"], c["values"], c["seg_begin"], c["seg_end"], c["truncated"],
                            None, c["gamma"], c["lam"])
    ra, rr = oracle.egae(c["rewards"], c["values"], c["seg_begin"], c["seg_end"], c["truncated"], None,
                         f32(c["gamma"]), f32(c["lam"]))
    assert st == 0 and adv_close(adv, ra, c["seg_begin"], c["seg_end"], 1e-5) <= 1.0
    assert adv_close(ret, rr, c["seg_begin"], c["seg_end"], 1e-5) <= 1.0
    pol, val, cn = run_select(c, 0, c["extra_policy_mask"], c["extra_value_mask"])
    rp, rv = oracle.select_tokens(c["seq_begin"], c["prompt_len"], c["prev_len"], c["new_len"],
                                  c["truncated"], 0, c["extra_policy_mask"], c["extra_value_mask"])
    assert np.array_equal(pol, rp) and np.array_equal(val, rv)
    assert len(rp) == 16384 and len(rv) == 16384 and not np.array_equal(rp, rv)   # independent filters
    # value loss on the 16384 value tokens
    loss_v, dv, nv, stv = run_value(c["values"], c["old_values"], rr.astype(np.float32), rv, c["xi_low"], c["xi_high"])
    rl, rdv = oracle.value_loss(c["values"], c["old_values"], rr.astype(np.float32), rv, f32(c["xi_low"]), f32(c["xi_high"]))
    assert nv == 16384 and abs(loss_v - rl) <= 1e-5 * max(1, abs(rl))
    edge = (np.abs(c["values"] - (c["old_values"] - f32(c["xi_low"]))) < 1e-6) | \
           (np.abs(c["values"] - (c["old_values"] + f32(c["xi_high"]))) < 1e-6)
    np.testing.assert_allclose(dv[~edge], rdv[~edge], rtol=1e-5, atol=1e-10)
    # policy loss
    host = synth.bf16_bits(c["logits"])
    adv32 = ra.astype(np.float32)
    lp_all = oracle.logprob(host, c["targets"])
    old = np.zeros(N, np.float32)
    old[rp] = lp_all + c["old_logp_noise"][rp]
    n_sel = torch.tensor([n], dtype=torch.int32, device=DEV)
    logits = c["logits"].clone() if inplace else c["logits"]
    logp, tl, loss, stats, dl = policy_full(c, logits, None, rp, old, adv32, n_sel,
                                            b.DLOGITS_FULL if inplace else b.DLOGITS_COMPACT, inplace=inplace)
    ref = oracle.policy_loss(host, c["targets"], None, rp, old, adv32, f32(c["eps_low"]), f32(c["eps_high"]),
                             want_dlogits=False)
    assert stats[0] == n and stats[3] == 0
    np.testing.assert_allclose(logp, ref["logp"], rtol=0, atol=LOGP_ATOL)
    np.testing.assert_allclose(tl, ref["token_loss"], rtol=0, atol=LOGP_ATOL * 4)
    assert abs(loss - ref["loss"]) <= LOGP_ATOL
    assert abs(int(stats[1]) - ref["clip_lo"]) <= 3 and abs(int(stats[2]) - ref["clip_hi"]) <= 3
    rng = np.random.default_rng(1)
    pick = np.sort(rng.choice(n, 192, replace=False)).astype(np.int32)
    pick[0], pick[-1] = 0, n - 1
    check_sampled_gradient(dl[torch.from_numpy(pick).long().to(DEV)], host, c, pick, rp[pick], old, adv32, n)
    # every gradient row sums to ~0 and is finite (property that holds at any size)
    sums = dl.float().sum(dim=1)
    assert bool(torch.isfinite(sums).all()) and float(sums.abs().max()) < 1e-3


def test_step_sequence_back_to_back_matches_single_calls():
    """The four calls of a training step issued back to back, several steps in a row, in the launch
    configuration the benchmark times (config 3's batch, the cluster-resident policy kernel directly
    followed by the next step's EGAE scan): every step must reproduce the results of the first one
    and the advantages must match the oracle."""
    import os
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench
    st = bench.Step(torch.device(DEV), rows=2048)
    st.run()
    torch.cuda.synchronize()
    first = (st.adv.clone(), st.ret.clone(), st.pol.clone(), float(st.loss), float(st.vloss))
    for _ in range(4):
        st.run()
        st.egae()                      # and once more straight after the value loss
    torch.cuda.synchronize()
    assert int(st.status) == 0 and int(st.stats[3]) == 0
    assert torch.equal(st.adv, first[0]) and torch.equal(st.ret, first[1]) and torch.equal(st.pol, first[2])
    assert float(st.loss) == first[3] and float(st.vloss) == first[4]
    c = st.c
    ra, rr = oracle.egae(c["rewards"], c["values"], c["seg_begin"], c["seg_end"], c["truncated"], None,
                         np.float32(c["gamma"]), np.float32(c["lam"]))
    assert adv_close(st.adv.cpu().numpy(), ra, c["seg_begin"], c["seg_end"], 1e-5) <= 1.0
    assert adv_close(st.ret.cpu().numpy(), rr, c["seg_begin"], c["seg_end"], 1e-5) <= 1.0
