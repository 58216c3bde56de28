"""GPU parity of tppo_advance_batch (successive batching between steps) against the oracle:
every output integer bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_15050_b200 import binding as b
from paper_2506_15050_b200 import synth
from gpu_util import DEV

pytestmark = pytest.mark.gpu


def t(a, dt):
    return torch.from_numpy(np.ascontiguousarray(a)).to(dt).to(DEV)


def run_advance(c, tokens, qb, qt, capacity=None):
    B = len(c["prompt_len"])
    cap = int(len(tokens) + len(qt)) if capacity is None else capacity
    npl = torch.full((max(B, 1),), -5, dtype=torch.int32, device=DEV)
    npv = torch.full((max(B, 1),), -5, dtype=torch.int32, device=DEV)
    nsb = torch.full((B + 1,), -5, dtype=torch.int32, device=DEV)
    ntk = torch.full((max(cap, 1),), -7, dtype=torch.int32, device=DEV)
    fs = torch.full((max(B, 1),), -9, dtype=torch.int32, device=DEV)
    src = torch.full((max(B, 1),), -5, dtype=torch.int32, device=DEV)
    counts = torch.full((4,), -1, dtype=torch.int32, device=DEV)
    b.tppo_advance_batch(t(c["seq_begin"], torch.int32), t(c["prompt_len"], torch.int32),
                         t(c["prev_len"], torch.int32), t(c["new_len"], torch.int32),
                         t(c["truncated"], torch.uint8), t(tokens, torch.int32), t(qb, torch.int32),
                         t(qt, torch.int32), npl[:B], npv[:B], nsb, ntk[:cap], fs[:B], src[:B], counts)
    torch.cuda.synchronize()
    cn = counts.cpu().numpy()
    return dict(next_prompt_len=npl[:B].cpu().numpy(), next_prev_len=npv[:B].cpu().numpy(),
                next_seq_begin=nsb.cpu().numpy(), next_tokens=ntk.cpu().numpy(),
                free_slots=fs.cpu().numpy()[:cn[0]], slot_source=src[:B].cpu().numpy(), counts=cn)


def check(c, tokens, qb, qt, capacity=None):
    got = run_advance(c, tokens, qb, qt, capacity)
    ref = oracle.advance_batch(c["seq_begin"], c["prompt_len"], c["prev_len"], c["new_len"],
                               c["truncated"], tokens, qb, qt, capacity)
    cap = int(len(tokens) + len(qt)) if capacity is None else capacity
    assert got["counts"][0] == ref["n_free"] and got["counts"][1] == ref["n_refilled"]
    assert got["counts"][2] == ref["total"]
    assert got["counts"][3] == (b.DEV_OVERFLOW if ref["total"] > cap else 0)
    for k in ("next_prompt_len", "next_prev_len", "next_seq_begin", "free_slots", "slot_source"):
        assert np.array_equal(got[k], ref[k]), k
    n = min(ref["total"], cap)
    assert np.array_equal(got["next_tokens"][:n], ref["next_tokens"][:n])
    assert np.all(got["next_tokens"][n:] == -7)            # nothing written past the context
    return got


def make_queue(rng, n, lo=1, hi=600):
    lens = rng.integers(lo, hi, n)
    qb = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    return qb, rng.integers(0, 150000, int(qb[-1])).astype(np.int32)


def ragged(rng, B, zero_frac=0.0):
    prompt = rng.integers(1, 700, B).astype(np.int32)
    prev = (rng.integers(0, 2, B) * rng.integers(0, 5000, B)).astype(np.int32)
    new = rng.integers(1, 3000, B).astype(np.int32)
    if zero_frac:
        z = rng.random(B) < zero_frac
        prompt[z], prev[z], new[z] = 0, 0, 0
    trunc = (rng.random(B) < 0.5).astype(np.uint8)
    sb, _, _ = synth.pack(prompt, prev, new)
    return dict(prompt_len=prompt, prev_len=prev, new_len=new, truncated=trunc, seq_begin=sb)


def test_advance_config1():
    c = synth.config1()
    got = check(c, np.arange(c["N"], dtype=np.int32), np.array([0, 3, 5], np.int32),
                np.array([11, 12, 13, 21, 22], np.int32))
    assert got["free_slots"].tolist() == [0, 2] and got["slot_source"].tolist() == [0, -1, 1, -1]


@pytest.mark.parametrize("B,seed,zero", [(1, 0, 0.0), (37, 1, 0.0), (1500, 2, 0.0), (4100, 3, 0.3)])
def test_advance_random_ragged(B, seed, zero):
    rng = np.random.default_rng(seed)
    c = ragged(rng, B, zero)
    N = int(c["seq_begin"][-1])
    tokens = rng.integers(0, 150000, N).astype(np.int32)
    n_fin = int((c["truncated"] == 0).sum())
    for m in (n_fin, max(n_fin - 2, 0), n_fin + 3, 0):
        qb, qt = make_queue(rng, m)
        check(c, tokens, qb, qt)
    qb, qt = make_queue(rng, n_fin)
    check(c, tokens, qb, qt, capacity=max(1, N // 3))      # output buffer too small: flagged


def test_advance_all_finished_all_unfinished_and_rerun():
    rng = np.random.default_rng(7)
    c = ragged(rng, 200)
    N = int(c["seq_begin"][-1])
    tokens = rng.integers(0, 1000, N).astype(np.int32)
    qb, qt = make_queue(rng, 200)
    for flag in (0, 1):
        c2 = dict(c, truncated=np.full(200, flag, np.uint8))
        check(c2, tokens, qb, qt)
    a = run_advance(c, tokens, qb, qt)
    d = run_advance(c, tokens, qb, qt)
    assert all(np.array_equal(a[k], d[k]) for k in a)


def test_advance_config4_scale():
    """The scale of config 4: 4096 slots, 17.5 M tokens, half of them finished."""
    c4 = synth.config4()
    rng = np.random.default_rng(8)
    tokens = rng.integers(0, 152064, c4["N"]).astype(np.int32)
    qb, qt = make_queue(rng, int((c4["truncated"] == 0).sum()), 16, 2048)
    check(c4, tokens, qb, qt)
