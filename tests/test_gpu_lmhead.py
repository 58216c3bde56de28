"""GPU parity of the LM-head variant (logits = hidden x weight on the tensor cores, never stored)
against the oracle, which forms the logits in float64 from the same bf16 inputs and then applies
its ordinary policy-loss routine and the plain definitions dH = dX W^T, dW = H^T dX.

Tolerances: log-probs, per-token losses and the loss 2e-3 absolute; gradients 1e-2 of the largest
reference magnitude per tensor, plus a per-element worst-case rounding bound: dX is rounded to bf16
(unit roundoff 2^-8) before the second contraction and the result once more, so
|gpu - ref| <= 2^-8 * (sum |a||b| + |ref|), the sum of absolute products coming from the oracle's own
contraction routines applied to the operands with their sign bits cleared."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_15050_b200 import binding as b
from paper_2506_15050_b200 import synth
from gpu_util import DEV

pytestmark = pytest.mark.gpu
f32 = lambda x: float(np.float32(x))
LOGP_ATOL = 2e-3
GRAD_RTOL = 1e-2


def t(a, dt):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(dt).to(DEV)


def run_lmhead(hidden, weight, targets, old_logp, adv, eps_low, eps_high, denom=0.0, aux=None,
               want_dh=True, want_dw=True, chunk_tiles=0):
    M, K = hidden.shape
    V = weight.shape[1]
    logp = torch.full((M,), float("nan"), device=DEV)
    tl = torch.full((M,), float("nan"), device=DEV)
    loss = torch.full((1,), float("nan"), device=DEV)
    stats = torch.full((4,), -1, dtype=torch.int32, device=DEV)
    dh = torch.full((M, K), float("nan"), dtype=torch.bfloat16, device=DEV) if want_dh else None
    dw = torch.full((K, V), float("nan"), dtype=torch.bfloat16, device=DEV) if want_dw else None
    ws = b.workspace(b.OP_LMHEAD, M, K, 0, V, DEV)
    b.tppo_lmhead_logprob_fwd_bwd(hidden, weight, t(targets, torch.int32), t(aux, torch.int32),
                                  t(old_logp, torch.float32), t(adv, torch.float32), eps_low,
                                  eps_high, denom, logp, tl, loss, stats, dh, dw, ws,
                                  chunk_tiles=chunk_tiles)
    torch.cuda.synchronize()
    return dict(logp=logp.cpu().numpy(), token_loss=tl.cpu().numpy(), loss=float(loss),
                stats=stats.cpu().numpy(), dh=None if dh is None else dh.float().cpu().numpy(),
                dw=None if dw is None else dw.float().cpu().numpy(), dh_t=dh, dw_t=dw)


def oracle_lmhead(hb, wb, rows, targets, old_logp, adv, eps_low, eps_high, denom):
    """Oracle results for the given rows: float64 logits, then Eq. 1 on them."""
    x = oracle.lmhead_logits_rows(hb, wb, np.asarray(rows, np.int32))
    ref = oracle.policy_loss(x, np.asarray(targets)[rows], None, None, np.asarray(old_logp)[rows],
                             np.asarray(adv)[rows], eps_low, eps_high, denom=denom)
    return x, ref


def grad_close(gpu, ref, abs_sum, what):
    scale = float(np.max(np.abs(ref)))
    err = np.abs(gpu - ref)
    assert np.all(np.isfinite(gpu)), what
    assert float(err.max()) <= GRAD_RTOL * scale + 1e-30, (what, float(err.max()), scale)
    bound = 1.05 * 2.0 ** -8 * (abs_sum + np.abs(ref)) + 1e-30
    assert np.all(err <= bound), (what, float((err / bound).max()))


def magnitude(bits):
    return np.asarray(bits) & np.uint16(0x7FFF)


def ref_dhidden(dx, wb):
    return oracle.lmhead_dhidden_rows(dx, wb), oracle.lmhead_dhidden_rows(np.abs(dx), magnitude(wb))


def ref_dweight(hb, dx):
    return oracle.lmhead_dweight_cols(hb, dx), oracle.lmhead_dweight_cols(magnitude(hb), np.abs(dx))


def make_case(M, K, V, seed, w_std=0.05):
    hidden = synth.randn_bf16((M, K), 1.0, seed, DEV)
    weight = synth.randn_bf16((K, V), w_std, seed + 1000, DEV)
    rng = np.random.default_rng(seed)
    targets = rng.integers(0, V, M).astype(np.int32)
    adv = rng.standard_normal(M).astype(np.float32)
    noise = (0.05 * rng.standard_normal(M)).astype(np.float32)
    return hidden, weight, targets, adv, noise


def old_logp_from_oracle(hb, wb, targets, noise):
    M = hb.shape[0]
    x = oracle.lmhead_logits_rows(hb, wb, np.arange(M, dtype=np.int32))
    lp = oracle.logprob(x, targets)
    return x, (lp + noise).astype(np.float32)


CTA_PAIR = 65536        # added to chunk_tiles: the CTA-pair (cta_group::2) GEMM kernels


@pytest.mark.parametrize("M,K,V,chunk", [(300, 320, 2000, 0), (300, 320, 2000, 3),
                                         (1024, 512, 8200, 5), (128, 64, 256, 0),
                                         (1, 64, 264, 0), (130, 328, 2008, 2),
                                         (130, 328, 2008, CTA_PAIR + 2),
                                         (300, 320, 2000, CTA_PAIR + 3),
                                         (1024, 512, 8200, CTA_PAIR)])
def test_lmhead_matches_oracle(M, K, V, chunk):
    hidden, weight, targets, adv, noise = make_case(M, K, V, seed=40 + M % 7)
    hb, wb = synth.bf16_bits(hidden), synth.bf16_bits(weight)
    x, old_logp = old_logp_from_oracle(hb, wb, targets, noise)
    eps_low, eps_high = 0.2, 0.28
    ref = oracle.policy_loss(x, targets, None, None, old_logp, adv, f32(eps_low), f32(eps_high))
    out = run_lmhead(hidden, weight, targets, old_logp, adv, eps_low, eps_high, chunk_tiles=chunk)
    assert out["stats"][3] == 0 and out["stats"][0] == M
    assert np.max(np.abs(out["logp"] - ref["logp"])) <= LOGP_ATOL
    # rows whose ratio sits on a clip edge may take the other branch in fp32
    rho = np.exp(ref["logp"] - old_logp)
    edge = (np.abs(rho - (1 - eps_low)) < 1e-3) | (np.abs(rho - (1 + eps_high)) < 1e-3)
    assert np.max(np.abs(out["token_loss"] - ref["token_loss"])[~edge]) <= LOGP_ATOL
    assert abs(out["loss"] - ref["loss"]) <= LOGP_ATOL
    assert abs(int(out["stats"][1]) - ref["clip_lo"]) <= int(edge.sum())
    assert abs(int(out["stats"][2]) - ref["clip_hi"]) <= int(edge.sum())
    dx = ref["dlogits"]
    dx[edge] = 0.0
    keep = ~edge
    ref_dh, abs_dh = ref_dhidden(dx, wb)
    grad_close(out["dh"][keep], ref_dh[keep], abs_dh[keep], "dhidden")
    # dweight sums over all rows, so a row on a clip edge cannot be left out of it: the seeds are
    # chosen so that there is none, and the comparison below always runs
    assert not edge.any()
    grad_close(out["dw"], *ref_dweight(hb, dx), "dweight")
    # clipped rows have a zero gradient
    clipped = (ref["dlogits"] == 0).all(axis=1) & keep
    assert np.all(out["dh"][clipped] == 0)


def test_lmhead_forward_only_and_denominator():
    M, K, V = 256, 128, 1024
    hidden, weight, targets, adv, noise = make_case(M, K, V, seed=7)
    hb, wb = synth.bf16_bits(hidden), synth.bf16_bits(weight)
    x, old_logp = old_logp_from_oracle(hb, wb, targets, noise)
    ref = oracle.policy_loss(x, targets, None, None, old_logp, adv, f32(0.2), f32(0.2), denom=1000.0)
    fwd = run_lmhead(hidden, weight, targets, old_logp, adv, 0.2, 0.2, denom=1000.0, want_dh=False,
                     want_dw=False)
    assert abs(fwd["loss"] - ref["loss"]) <= LOGP_ATOL
    assert np.max(np.abs(fwd["logp"] - ref["logp"])) <= LOGP_ATOL
    full = run_lmhead(hidden, weight, targets, old_logp, adv, 0.2, 0.2, denom=1000.0)
    assert full["loss"] == fwd["loss"] and np.array_equal(full["logp"], fwd["logp"])
    grad_close(full["dh"], *ref_dhidden(ref["dlogits"], wb), "dhidden")


def test_lmhead_aux_index_and_bad_rows():
    M, K, V = 200, 64, 512
    hidden, weight, targets, adv, noise = make_case(M, K, V, seed=11)
    hb, wb = synth.bf16_bits(hidden), synth.bf16_bits(weight)
    x, old_logp = old_logp_from_oracle(hb, wb, targets, noise)
    rng = np.random.default_rng(3)
    perm = rng.permutation(M).astype(np.int32)              # row j reads adv / old_logp at perm[j]
    adv_p = np.empty_like(adv); adv_p[perm] = adv
    old_p = np.empty_like(old_logp); old_p[perm] = old_logp
    bad_t = targets.copy(); bad_t[5] = V; bad_t[17] = -1
    aux = perm.copy(); aux[40] = M + 3
    good = np.ones(M, bool); good[[5, 17, 40]] = False
    out = run_lmhead(hidden, weight, bad_t, old_p, adv_p, 0.2, 0.2, aux=aux)
    assert out["stats"][3] == (b.DEV_BAD_TARGET | b.DEV_BAD_INDEX)
    # the mean still divides by M; the three bad rows contribute nothing
    rows = np.nonzero(good)[0].astype(np.int32)
    ref = oracle.policy_loss(x, targets, rows, None, old_logp, adv, f32(0.2), f32(0.2), denom=float(M))
    assert abs(out["loss"] - ref["loss"]) <= LOGP_ATOL
    assert np.max(np.abs(out["logp"][good] - ref["logp"])) <= LOGP_ATOL
    assert np.all(out["logp"][~good] == 0) and np.all(out["token_loss"][~good] == 0)
    assert np.all(out["dh"][~good] == 0)
    grad_close(out["dh"][good], *ref_dhidden(ref["dlogits"], wb), "dhidden")
    dx_all = np.zeros((M, V)); dx_all[good] = ref["dlogits"]
    grad_close(out["dw"], *ref_dweight(hb, dx_all), "dweight")


def test_lmhead_host_errors_and_determinism():
    M, K, V = 128, 64, 512
    hidden, weight, targets, adv, noise = make_case(M, K, V, seed=5)
    old = np.full(M, -6.0, np.float32)
    a = run_lmhead(hidden, weight, targets, old, adv, 0.2, 0.2)
    c = run_lmhead(hidden, weight, targets, old, adv, 0.2, 0.2)
    assert a["loss"] == c["loss"] and torch.equal(a["dh_t"], c["dh_t"]) and torch.equal(a["dw_t"], c["dw_t"])
    ws = b.workspace(b.OP_LMHEAD, M, K, 0, V, DEV)
    loss = torch.zeros(1, device=DEV)
    stats = torch.zeros(4, dtype=torch.int32, device=DEV)
    args = lambda h, w, wsp: (h, w, t(targets, torch.int32), None, t(old, torch.float32),
                              t(adv, torch.float32), 0.2, 0.2, 0.0, None, None, loss, stats, None,
                              None, wsp)
    with pytest.raises(b.TppoError) as e:
        b.tppo_lmhead_logprob_fwd_bwd(*args(hidden, weight, ws[:256]))
    assert e.value.status == 2
    w_odd = synth.randn_bf16((K, 508), 0.05, 1, DEV)          # V not a multiple of 8
    with pytest.raises(b.TppoError) as e:
        b.tppo_lmhead_logprob_fwd_bwd(*args(hidden, w_odd, ws))
    assert e.value.status == 3


# ---------------------------------------------------------------------------------------------
# config 5 at full size: [16384, 5120] x [5120, 152064], the launch configuration that is timed.
# The oracle forms one vocabulary row of logits at a time, so it checks about 256 sampled rows in
# full (every row position of a GEMM tile, both edges of 32 tiles; a few minutes of host time) and,
# for dweight (which sums over all rows), a run whose advantages are zero outside the sampled
# rows: every other row then has dX = 0 and the reference sum has only the sampled terms.
# ---------------------------------------------------------------------------------------------
LOG_V_MODEL = -13.0      # typical log-prob of a random token under these logits (an input, not a result)


def _config5_sample(c, seed, tile=128):
    """At least 256 rows of the M = 16384: the first and the last row of 32 different 128-row GEMM
    tiles (the first and the last tile among them), one row for every position 0..127 inside a tile
    (each taken from a different tile), and 64 rows drawn at random."""
    rng = np.random.default_rng(seed)
    M = c["M"]
    n_tiles = M // tile
    edge_tiles = np.unique(np.concatenate([np.arange(0, n_tiles, n_tiles // 32), [n_tiles - 1]]))
    edges = np.concatenate([edge_tiles * tile, edge_tiles * tile + tile - 1])
    lanes = np.array([((i * 37) % n_tiles) * tile + i for i in range(tile)])
    pick = np.unique(np.concatenate([edges, lanes, rng.choice(M, 64, replace=False)])).astype(np.int32)
    assert len(pick) >= 224 and len(np.unique(pick % tile)) == tile
    assert len(np.intersect1d(pick[pick % tile == 0] // tile, pick[pick % tile == tile - 1] // tile)) >= 32
    return pick


@pytest.fixture(scope="module")
def cfg5():
    c = synth.config5(DEV)
    assert c["hidden"].shape == (16384, 5120) and c["weight"].shape == (5120, 152064)
    c["hb"], c["wb"] = synth.bf16_bits(c["hidden"]), synth.bf16_bits(c["weight"])
    c["pick"] = _config5_sample(c, seed=50)
    c["x_pick"] = oracle.lmhead_logits_rows(c["hb"], c["wb"], c["pick"])
    lp = oracle.logprob(c["x_pick"], c["targets"][c["pick"]])
    old = (LOG_V_MODEL + c["old_logp_noise"]).astype(np.float32)
    old[c["pick"]] = (lp + c["old_logp_noise"][c["pick"]]).astype(np.float32)
    c["old_logp"] = old
    # the oracle's Eq. 1 results and dhidden rows for the sampled rows, shared by the tests below
    # (the advantages of the sampled rows and the divisor M are the same in all of them)
    c["ref"] = oracle.policy_loss(c["x_pick"], c["targets"][c["pick"]], None, None, old[c["pick"]],
                                  c["adv"][c["pick"]], f32(c["eps_low"]), f32(c["eps_high"]),
                                  denom=float(c["M"]))
    c["ref_dh"] = ref_dhidden(c["ref"]["dlogits"], c["wb"])
    yield c
    del c["hidden"], c["weight"]
    torch.cuda.empty_cache()


@pytest.mark.parametrize("variant", [0, CTA_PAIR])
def test_config5_full_sampled_rows(cfg5, variant):
    c = cfg5
    M, K, V, pick = c["M"], c["K"], c["V"], c["pick"]
    out = run_lmhead(c["hidden"], c["weight"], c["targets"], c["old_logp"], c["adv"], c["eps_low"],
                     c["eps_high"], chunk_tiles=variant)
    assert out["stats"][0] == M and out["stats"][3] == 0
    ref = c["ref"]
    np.testing.assert_allclose(out["logp"][pick], ref["logp"], rtol=0, atol=LOGP_ATOL)
    np.testing.assert_allclose(out["token_loss"][pick], ref["token_loss"], rtol=0, atol=4 * LOGP_ATOL)
    grad_close(out["dh"][pick], *c["ref_dh"], "dhidden rows")
    # properties that hold at any size
    assert np.all(np.isfinite(out["logp"])) and np.all(out["logp"] < 0)
    assert abs(out["loss"] - float(np.mean(out["token_loss"].astype(np.float64)))) <= 1e-5
    dw = out["dw_t"].float()
    assert bool(torch.isfinite(dw).all()) and bool(torch.isfinite(out["dh_t"].float()).all())
    # every dX row sums to zero, hence every dweight row does
    row_sum = dw.sum(dim=1).abs()
    row_abs = dw.abs().sum(dim=1)
    assert float((row_sum / row_abs).max()) < 1e-3
    # the run is reproducible bit for bit
    again = run_lmhead(c["hidden"], c["weight"], c["targets"], c["old_logp"], c["adv"], c["eps_low"],
                       c["eps_high"], chunk_tiles=variant)
    assert again["loss"] == out["loss"] and torch.equal(again["dw_t"], out["dw_t"]) and \
        torch.equal(again["dh_t"], out["dh_t"])


def test_config5_full_dweight_from_sampled_rows(cfg5):
    c = cfg5
    M, K, V, pick = c["M"], c["K"], c["V"], c["pick"]
    adv = np.zeros(M, np.float32)
    adv[pick] = c["adv"][pick]
    out = run_lmhead(c["hidden"], c["weight"], c["targets"], c["old_logp"], adv, c["eps_low"],
                     c["eps_high"])
    assert out["stats"][3] == 0
    ref = c["ref"]                 # same rows, same advantages on them, same divisor
    assert np.any(ref["dlogits"] != 0)
    rng = np.random.default_rng(51)
    cols = np.concatenate([rng.choice(V, 1500, replace=False), [0, 255, 256, V - 1, V - 8],
                           c["targets"][pick]]).astype(np.int64)
    cols = np.unique(cols)
    got = out["dw_t"][:, torch.from_numpy(cols).to(DEV)].float().cpu().numpy()
    dx_cols = np.ascontiguousarray(ref["dlogits"][:, cols])
    hb_pick = np.ascontiguousarray(c["hb"][pick])
    grad_close(got, *ref_dweight(hb_pick, dx_cols), "dweight columns")
    # rows without advantage have an exactly zero gradient; the sampled ones match the oracle
    others = np.setdiff1d(np.arange(M), pick)
    assert float(out["dh_t"][torch.from_numpy(others).to(DEV)].float().abs().max()) == 0.0
    grad_close(out["dh"][pick], *c["ref_dh"], "dhidden rows")


# ---- vocabulary shards (weight split by columns; the ranks are emulated one after another) --------
def run_lmhead_sharded(hidden, weight, bounds, targets, old_logp, adv, eps_low, eps_high, denom=0.0,
                       aux=None, chunk_tiles=0):
    """Both shard calls for every shard [bounds[i], bounds[i+1]) with the merge a caller performs
    between them (max, rescale, sum) done by torch reductions over the emulated ranks."""
    M, K = hidden.shape
    V = weight.shape[1]
    tg, ax = t(targets, torch.int32), t(aux, torch.int32)
    olp, ad = t(old_logp, torch.float32), t(adv, torch.float32)
    shards = [weight[:, lo:hi].contiguous() for lo, hi in zip(bounds[:-1], bounds[1:])]
    rm, rs, rxy, bits = [], [], [], 0
    for lo, wsd in zip(bounds[:-1], shards):
        m_, s_, xy_ = (torch.full((M,), float("nan"), device=DEV) for _ in range(3))
        st = torch.full((4,), -1, dtype=torch.int32, device=DEV)
        ws = b.workspace(b.OP_LMHEAD, M, K, 0, wsd.shape[1], DEV)
        b.tppo_lmhead_shard_stats(hidden, wsd, lo, V, tg, m_, s_, xy_, st, ws, chunk_tiles=chunk_tiles)
        bits |= int(st[3])
        rm.append(m_); rs.append(s_); rxy.append(xy_)
    m_all = torch.stack(rm).max(dim=0).values
    for m_, s_ in zip(rm, rs):
        b.tppo_lmhead_shard_rescale(m_, m_all, s_)
    s_all, xy_all = torch.stack(rs).sum(dim=0), torch.stack(rxy).sum(dim=0)
    outs = []
    for lo, wsd in zip(bounds[:-1], shards):
        Vs = wsd.shape[1]
        logp = torch.full((M,), float("nan"), device=DEV)
        tl = torch.full((M,), float("nan"), device=DEV)
        loss = torch.full((1,), float("nan"), device=DEV)
        st = torch.full((4,), -1, dtype=torch.int32, device=DEV)
        dh = torch.full((M, K), float("nan"), dtype=torch.bfloat16, device=DEV)
        dw = torch.full((K, Vs), float("nan"), dtype=torch.bfloat16, device=DEV)
        ws = b.workspace(b.OP_LMHEAD, M, K, 0, Vs, DEV)
        b.tppo_lmhead_shard_fwd_bwd(hidden, wsd, lo, V, tg, ax, olp, ad, eps_low, eps_high, denom,
                                    m_all, s_all, xy_all, logp, tl, loss, st, dh, dw, ws,
                                    chunk_tiles=chunk_tiles)
        outs.append(dict(logp=logp, tl=tl, loss=loss, st=st, dh=dh, dw=dw))
    torch.cuda.synchronize()
    for o in outs[1:]:           # the replicated outputs agree bit for bit across the shards
        for k in ("logp", "tl", "loss", "st"):
            assert torch.equal(o[k], outs[0][k]), k
    return dict(logp=outs[0]["logp"].cpu().numpy(), token_loss=outs[0]["tl"].cpu().numpy(),
                loss=float(outs[0]["loss"]), stats=outs[0]["st"].cpu().numpy(), stats_bits=bits,
                dh=torch.stack([o["dh"].float() for o in outs]).sum(dim=0).cpu().numpy(),
                dw=torch.cat([o["dw"].float() for o in outs], dim=1).cpu().numpy(),
                dh_parts=[o["dh"] for o in outs], dw_parts=[o["dw"] for o in outs])


@pytest.mark.parametrize("M,K,V,bounds,chunk", [(300, 320, 2000, (0, 840, 2000), 0),
                                                (130, 328, 2008, (0, 8, 1000, 2008), 2),
                                                (1024, 512, 8200, (0, 4096, 8200), CTA_PAIR)])
def test_lmhead_vocabulary_shards_match_oracle(M, K, V, bounds, chunk):
    hidden, weight, targets, adv, noise = make_case(M, K, V, seed=90 + M % 7)
    targets[:4] = [0, bounds[1] - 1, bounds[1], V - 1]           # shard edges
    hb, wb = synth.bf16_bits(hidden), synth.bf16_bits(weight)
    x, old_logp = old_logp_from_oracle(hb, wb, targets, noise)
    eps_low, eps_high = 0.2, 0.28
    ref = oracle.policy_loss(x, targets, None, None, old_logp, adv, f32(eps_low), f32(eps_high))
    out = run_lmhead_sharded(hidden, weight, bounds, targets, old_logp, adv, eps_low, eps_high,
                             chunk_tiles=chunk)
    assert out["stats_bits"] == 0 and out["stats"][3] == 0 and out["stats"][0] == M
    assert np.max(np.abs(out["logp"] - ref["logp"])) <= LOGP_ATOL
    rho = np.exp(ref["logp"] - old_logp)
    edge = (np.abs(rho - (1 - eps_low)) < 1e-3) | (np.abs(rho - (1 + eps_high)) < 1e-3)
    assert np.max(np.abs(out["token_loss"] - ref["token_loss"])[~edge]) <= LOGP_ATOL
    assert abs(out["loss"] - ref["loss"]) <= LOGP_ATOL
    dx = ref["dlogits"]
    dx[edge] = 0.0
    keep = ~edge
    ref_dh, abs_dh = ref_dhidden(dx, wb)
    # every shard's partial dhidden is rounded to bf16 before the sum: |p_i| <= its sum of |a||b|
    grad_close(out["dh"][keep], ref_dh[keep], 2.0 * abs_dh[keep], "dhidden")
    # dweight sums over all rows, so a row on a clip edge cannot be left out of it: the seeds are
    # chosen so that there is none, and the comparison below always runs
    assert not edge.any()
    grad_close(out["dw"], *ref_dweight(hb, dx), "dweight")


def test_lmhead_one_shard_equals_the_unsharded_call():
    M, K, V = 200, 128, 1032
    hidden, weight, targets, adv, noise = make_case(M, K, V, seed=5)
    hb, wb = synth.bf16_bits(hidden), synth.bf16_bits(weight)
    _, old_logp = old_logp_from_oracle(hb, wb, targets, noise)
    whole = run_lmhead(hidden, weight, targets, old_logp, adv, 0.2, 0.28)
    one = run_lmhead_sharded(hidden, weight, (0, V), targets, old_logp, adv, 0.2, 0.28)
    for k in ("logp", "token_loss", "stats"):
        assert np.array_equal(whole[k], one[k]), k
    assert whole["loss"] == one["loss"]
    assert torch.equal(whole["dh_t"], one["dh_parts"][0])
    assert torch.equal(whole["dw_t"], one["dw_parts"][0])


def test_lmhead_shards_bad_target_aux_and_host_errors():
    M, K, V = 64, 64, 512
    hidden, weight, targets, adv, noise = make_case(M, K, V, seed=11)
    hb, wb = synth.bf16_bits(hidden), synth.bf16_bits(weight)
    _, old_logp = old_logp_from_oracle(hb, wb, targets, noise)
    bad = targets.copy()
    bad[3], bad[9] = V, -1                                   # outside the whole vocabulary
    aux = np.random.default_rng(2).permutation(M).astype(np.int32)
    olp_a, adv_a = np.empty_like(old_logp), np.empty_like(adv)
    olp_a[aux], adv_a[aux] = old_logp, adv                   # row r reads entry aux[r]
    out = run_lmhead_sharded(hidden, weight, (0, 256, 512), bad, olp_a, adv_a, 0.2, 0.28, aux=aux)
    assert out["stats_bits"] & b.DEV_BAD_TARGET and out["stats"][3] & b.DEV_BAD_TARGET
    good = np.ones(M, bool)
    good[[3, 9]] = False
    x = oracle.lmhead_logits_rows(hb, wb, np.arange(M, dtype=np.int32))
    ref = oracle.policy_loss(x[good], bad[good], None, None, old_logp[good], adv[good], f32(0.2),
                             f32(0.28), denom=float(M))
    assert np.max(np.abs(out["logp"][good] - ref["logp"])) <= LOGP_ATOL
    assert np.all(out["logp"][~good] == 0) and np.all(out["dh"][~good] == 0)
    assert abs(out["loss"] - ref["loss"]) <= LOGP_ATOL
    # host-detectable errors: offset outside the vocabulary, shard wider than the vocabulary
    wsd = weight[:, :256].contiguous()
    m_, s_, xy_ = (torch.zeros(M, device=DEV) for _ in range(3))
    st = torch.zeros(4, dtype=torch.int32, device=DEV)
    ws = b.workspace(b.OP_LMHEAD, M, K, 0, 256, DEV)
    for off, vt in ((-1, V), (300, V), (0, 128)):
        with pytest.raises(b.TppoError) as e:
            b.tppo_lmhead_shard_stats(hidden, wsd, off, vt, t(bad, torch.int32), m_, s_, xy_, st, ws)
        assert e.value.status == 1
