"""The several-GPU path on CPU: two gloo ranks, each with its own slice of a batch split by
sequence.  The per-rank arithmetic is done by the oracle here (there is no GPU); what is under test
is the host logic of `paper_2506_15050_b200.shard` -- the partition, the re-based packed slices,
the global token counts passed as `denom`, and the reduction of the partial losses -- which must
reproduce the unsharded result."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2506_15050_b200 import shard, synth

f32 = lambda x: float(np.float32(x))


def _batch():
    c = synth.config1()
    lp = oracle.logprob(c["logits"], c["targets"])
    c["old_logp"] = (lp + c["old_logp_noise"]).astype(np.float32)
    return c


def _run_path(c, denom_pol=0.0, denom_val=0.0):
    """EGAE -> selection -> policy loss -> value loss on one packed batch, with the oracle."""
    adv, ret = oracle.egae(c["rewards"], c["values"], c["seg_begin"], c["seg_end"], c["truncated"],
                           None, f32(c["gamma"]), f32(c["lam"]))
    pol, val = oracle.select_tokens(c["seq_begin"], c["prompt_len"], c["prev_len"], c["new_len"],
                                    c["truncated"])
    p = oracle.policy_loss(c["logits"], c["targets"], pol, None, c["old_logp"], adv.astype(np.float32),
                           f32(c["eps_low"]), f32(c["eps_high"]), denom=denom_pol, want_dlogits=False)
    vl, _ = oracle.value_loss(c["values"], c["old_values"], ret.astype(np.float32), val,
                              f32(c["xi_low"]), f32(c["xi_high"]), denom=denom_val, want_grad=False)
    return adv, pol, val, p["loss"], vl


def _worker(rank, world, port, out_path):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        c = _batch()
        c["old_logp_noise"] = c["old_logp"]                 # carried through the per-token slicing
        tokens = np.diff(c["seq_begin"].astype(np.int64))
        lo, hi = shard.partition_sequences(tokens, world)[rank]
        s = shard.shard_batch(c, lo, hi)
        s["old_logp"] = s["old_logp_noise"]
        # pass 1: counts only (denominators are needed before the losses)
        pol, val = oracle.select_tokens(s["seq_begin"], s["prompt_len"], s["prev_len"], s["new_len"],
                                        s["truncated"])
        n_pol, n_val = shard.global_token_counts(len(pol), len(val))
        adv, pol, val, pl, vl = _run_path(s, float(n_pol), float(n_val))
        pl, vl = shard.reduce_losses(pl, vl)
        gathered = [None] * world
        dist.all_gather_object(gathered, dict(off=s["token_offset"], adv=adv, pol=pol, val=val))
        if rank == 0:
            np.savez(out_path, n_pol=n_pol, n_val=n_val, pl=pl, vl=vl,
                     adv=np.concatenate([g["adv"] for g in gathered]),
                     pol=np.concatenate([g["pol"] + g["off"] for g in gathered]),
                     val=np.concatenate([g["val"] + g["off"] for g in gathered]))
    finally:
        dist.destroy_process_group()


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.timeout(180)
def test_two_ranks_reproduce_the_unsharded_batch(tmp_path):
    out = str(tmp_path / "sharded.npz")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    got = np.load(out)
    c = _batch()
    adv, pol, val, pl, vl = _run_path(c)
    assert int(got["n_pol"]) == len(pol) and int(got["n_val"]) == len(val)
    assert np.array_equal(got["pol"], pol) and np.array_equal(got["val"], val)
    np.testing.assert_array_equal(got["adv"], adv)          # per-sequence work: identical
    assert abs(float(got["pl"]) - pl) <= 1e-12 * max(1.0, abs(pl))
    assert abs(float(got["vl"]) - vl) <= 1e-12 * max(1.0, abs(vl))


def test_partition_covers_every_sequence_once_and_balances():
    rng = np.random.default_rng(0)
    for world in (1, 2, 3, 8):
        for B in (0, 1, 5, 64):
            t = rng.integers(1, 5000, B)
            parts = shard.partition_sequences(t, world)
            assert len(parts) == world and parts[0][0] == 0 and parts[-1][1] == B
            assert all(a[1] == b[0] for a, b in zip(parts, parts[1:]))
            assert all(lo <= hi for lo, hi in parts)
            if B >= 8 * world:
                loads = np.array([t[lo:hi].sum() for lo, hi in parts])
                assert loads.max() - loads.min() <= 2 * t.max()


def test_shard_batch_rebases_offsets():
    c = _batch()
    s = shard.shard_batch(c, 1, 3)
    assert s["B"] == 2 and s["seq_begin"][0] == 0 and s["N"] == int(c["seq_begin"][3] - c["seq_begin"][1])
    off = s["token_offset"]
    assert np.array_equal(s["values"], c["values"][off:off + s["N"]])
    assert np.array_equal(s["seg_end"] + off, c["seg_end"][1:3])
    assert np.array_equal(s["truncated"], c["truncated"][1:3])


# ---- vocabulary-parallel LM-head: the exchange between the two shard calls -----------------------
def _vocab_worker(rank, world, port, out_path):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        c = _batch()
        x = c["logits"].astype(np.float64)
        V = x.shape[1]
        lo, hi = (0, 40) if rank == 0 else (40, V)          # unequal shards
        xs = x[:, lo:hi]
        m = xs.max(axis=1)
        s = np.exp(xs - m[:, None]).sum(axis=1)
        y = c["targets"].astype(np.int64)
        inside = (y >= lo) & (y < hi)
        xy = np.where(inside, x[np.arange(len(y)), np.clip(y, lo, hi - 1)], 0.0)

        def rescale(row_max, row_max_all, row_sumexp):
            row_sumexp.mul_(torch.exp(row_max - row_max_all))

        tm, ts, txy = (torch.from_numpy(a.copy()) for a in (m, s, xy))
        shard.combine_row_stats(tm, ts, txy, rescale)
        logp = txy - tm - torch.log(ts)
        gathered = [None] * world
        dist.all_gather_object(gathered, logp.numpy())
        if rank == 0:
            np.savez(out_path, a=gathered[0], b=gathered[1])
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(180)
def test_two_vocabulary_shards_merge_to_the_whole_log_softmax(tmp_path):
    out = str(tmp_path / "vocab.npz")
    mp.spawn(_vocab_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    got = np.load(out)
    c = _batch()
    ref = oracle.logprob(c["logits"], c["targets"])
    np.testing.assert_array_equal(got["a"], got["b"])        # every rank ends with the same values
    np.testing.assert_allclose(got["a"], ref, rtol=0, atol=1e-12)


def test_combine_row_stats_is_the_identity_on_one_rank():
    m, s, xy = torch.tensor([1.0, 2.0]), torch.tensor([3.0, 4.0]), torch.tensor([0.5, 0.0])
    out = shard.combine_row_stats(m, s, xy, rescale=None)
    assert out[0] is m and out[1] is s and out[2] is xy


# ---- vocabulary-parallel LM-head: the whole step (statistics, exchange, gradients, dhidden sum) --------
def _lm_case():
    rng = np.random.default_rng(17)
    M, K, V = 24, 16, 88
    h = torch.from_numpy(rng.standard_normal((M, K)).astype(np.float32)).to(torch.bfloat16)
    w = torch.from_numpy((0.3 * rng.standard_normal((K, V))).astype(np.float32)).to(torch.bfloat16)
    hb = h.view(torch.int16).numpy().view(np.uint16)
    wb = w.view(torch.int16).numpy().view(np.uint16)
    y = rng.integers(0, V, M).astype(np.int32)
    y[:3] = [0, 47, 48]                                      # both sides of the shard boundary
    adv = rng.standard_normal(M).astype(np.float32)
    x = oracle.lmhead_logits_rows(hb, wb, np.arange(M, dtype=np.int32))
    old = (oracle.logprob(x, y) + 0.2 * rng.standard_normal(M)).astype(np.float32)   # some ratios clip
    return dict(M=M, K=K, V=V, hb=hb, wb=wb, y=y, adv=adv, old=old, x=x)


def _lm_worker(rank, world, port, out_path):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        c = _lm_case()
        M, V = c["M"], c["V"]
        lo, hi = shard.vocab_shard_bounds(V, world)[rank]
        assert (lo, hi) == ((0, 48) if rank == 0 else (48, 88))
        wb_s = np.ascontiguousarray(c["wb"][:, lo:hi])
        xs = oracle.lmhead_logits_rows(c["hb"], wb_s, np.arange(M, dtype=np.int32))   # this rank's logits
        inside = (c["y"] >= lo) & (c["y"] < hi)
        col = np.clip(c["y"] - lo, 0, hi - lo - 1)
        out = {}

        def stats_fn():
            m = xs.max(axis=1)
            return (torch.from_numpy(m.copy()), torch.from_numpy(np.exp(xs - m[:, None]).sum(axis=1)),
                    torch.from_numpy(np.where(inside, xs[np.arange(M), col], 0.0)))

        def rescale_fn(row_max, row_max_all, row_sumexp):
            row_sumexp.mul_(torch.exp(row_max - row_max_all))

        def grads_fn(row_max, row_sumexp, row_xy):
            m, s_, xy = row_max.numpy(), row_sumexp.numpy(), row_xy.numpy()
            logp = xy - m - np.log(s_)
            # Eq. 1 by the oracle on the two-class reduction {target, everything else}: a row of two
            # logits whose softmax gives the target exactly the probability exp(logp)
            two = np.stack([logp, np.log1p(-np.exp(logp))], axis=1)
            r = oracle.policy_loss(two, np.zeros(M, np.int32), None, None, c["old"], c["adv"],
                                   f32(0.2), f32(0.28))
            p_y = np.exp(logp)
            coef = r["dlogits"][:, 0] / (p_y - 1.0)          # dlogits = coef * (softmax - onehot)
            dx = coef[:, None] * np.exp(xs - m[:, None] - np.log(s_)[:, None])
            dx[inside, col[inside]] -= coef[inside]
            out["loss"], out["logp"] = r["loss"], logp
            out["dw"] = oracle.lmhead_dweight_cols(c["hb"], dx)
            return torch.from_numpy(oracle.lmhead_dhidden_rows(dx, wb_s))

        dh = shard.vocab_parallel_step(stats_fn, rescale_fn, grads_fn)
        gathered = [None] * world
        dist.all_gather_object(gathered, dict(dw=out["dw"], dh=dh.numpy(), loss=out["loss"], logp=out["logp"]))
        if rank == 0:
            np.savez(out_path, dw=np.concatenate([g["dw"] for g in gathered], axis=1),
                     dh0=gathered[0]["dh"], dh1=gathered[1]["dh"], loss0=gathered[0]["loss"],
                     loss1=gathered[1]["loss"], logp=gathered[0]["logp"])
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(180)
def test_two_vocabulary_shards_reproduce_the_unsharded_lm_head_step(tmp_path):
    """Each of two gloo ranks holds one column shard of the weight; the merged loss, dhidden and
    dweight must equal the oracle's unsharded LM-head results."""
    out = str(tmp_path / "lm.npz")
    mp.spawn(_lm_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    got = np.load(out)
    c = _lm_case()
    ref = oracle.policy_loss(c["x"], c["y"], None, None, c["old"], c["adv"], f32(0.2), f32(0.28))
    assert ref["clip_lo"] + ref["clip_hi"] > 0               # the clipped branch is exercised
    np.testing.assert_allclose(got["logp"], ref["logp"], rtol=0, atol=1e-12)
    assert abs(float(got["loss0"]) - ref["loss"]) <= 1e-12 and float(got["loss0"]) == float(got["loss1"])
    ref_dh = oracle.lmhead_dhidden_rows(ref["dlogits"], c["wb"])
    ref_dw = oracle.lmhead_dweight_cols(c["hb"], ref["dlogits"])
    np.testing.assert_array_equal(got["dh0"], got["dh1"])    # the all-reduce leaves every rank with the sum
    np.testing.assert_allclose(got["dh0"], ref_dh, rtol=0, atol=1e-12 * max(1.0, np.abs(ref_dh).max()))
    np.testing.assert_allclose(got["dw"], ref_dw, rtol=0, atol=1e-12 * max(1.0, np.abs(ref_dw).max()))


def test_vocab_shard_bounds_cover_the_vocabulary():
    for V in (88, 152064, 1000, 8):
        for world in (1, 2, 3, 8):
            b = shard.vocab_shard_bounds(V, world)
            assert len(b) == world and b[0][0] == 0 and b[-1][1] == V
            assert all(x[1] == y[0] for x, y in zip(b, b[1:])) and all(lo <= hi for lo, hi in b)
            assert all(lo % 8 == 0 for lo, _ in b)
