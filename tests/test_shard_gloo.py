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
