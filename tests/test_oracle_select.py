"""Pins for the oracle's token filter (Section 3.2)."""
import itertools

import numpy as np

import oracle
from paper_2506_15050_b200 import synth


def set_builder(prompt, prev, new, trunc, tail_drop, pm=None, vm=None):
    """The filter rule written as set comprehensions over (sequence, offset) pairs.  tail_drop is
    one count for every unfinished sequence, or a list with one count per sequence."""
    starts = np.concatenate([[0], np.cumsum(np.array(prompt) + np.array(prev) + np.array(new))])
    drop = [tail_drop] * len(prompt) if np.isscalar(tail_drop) else list(tail_drop)
    pol = {int(starts[i]) + o
           for i in range(len(prompt))
           for o in range(prompt[i] + prev[i] + new[i])
           if prompt[i] + prev[i] <= o < prompt[i] + prev[i] + new[i] - (max(drop[i], 0) if trunc[i] else 0)}
    val = {int(starts[i]) + o
           for i in range(len(prompt))
           for o in range(prompt[i] + prev[i] + new[i])
           if not trunc[i] and o >= prompt[i]}
    if pm is not None:
        pol = {p for p in pol if pm[p]}
    if vm is not None:
        val = {p for p in val if vm[p]}
    return sorted(pol), sorted(val)


def run(prompt, prev, new, trunc, tail_drop, pm=None, vm=None):
    sb, _, _ = synth.pack(prompt, prev, new)
    if np.isscalar(tail_drop):
        return oracle.select_tokens(sb, prompt, prev, new, trunc, tail_drop, pm, vm)
    # a per-sequence array overrides the scalar, whatever the scalar is
    return oracle.select_tokens(sb, prompt, prev, new, trunc, 99, pm, vm, tail_drop_seq=tail_drop)


def test_exhaustive_enumeration_small():
    lens = range(0, 4)
    n = 0
    for B in (1, 2):
        for combo in itertools.product(itertools.product(lens, lens, lens, (0, 1)), repeat=B):
            prompt = [c[0] for c in combo]
            prev = [c[1] for c in combo]
            new = [c[2] for c in combo]
            trunc = [c[3] for c in combo]
            for td in (0, 1, 2, 5):
                pol, val = run(prompt, prev, new, trunc, td)
                rp, rv = set_builder(prompt, prev, new, trunc, td)
                assert pol.tolist() == rp and val.tolist() == rv
                n += 1
    assert n > 60000


def test_exhaustive_three_sequences_with_masks():
    rng = np.random.default_rng(0)
    lens = range(0, 3)
    for combo in itertools.product(itertools.product(lens, lens, lens, (0, 1)), repeat=3):
        prompt = [c[0] for c in combo]
        prev = [c[1] for c in combo]
        new = [c[2] for c in combo]
        trunc = [c[3] for c in combo]
        N = sum(prompt) + sum(prev) + sum(new)
        pm = rng.integers(0, 2, max(N, 1)).astype(np.uint8)
        vm = rng.integers(0, 2, max(N, 1)).astype(np.uint8)
        pol, val = run(prompt, prev, new, trunc, 1, pm, vm)
        rp, rv = set_builder(prompt, prev, new, trunc, 1, pm, vm)
        assert pol.tolist() == rp and val.tolist() == rv


def test_exhaustive_enumeration_per_sequence_tail_drop():
    """Every pair of sequences with lengths <= 3 and every pair of per-sequence counts in
    {-1, 0, 1, 2, 4} (more than a sequence has, and a negative one, included)."""
    lens = range(0, 4)
    drops = (-1, 0, 1, 2, 4)
    n = 0
    for combo in itertools.product(itertools.product(lens, (0, 2), lens, (0, 1)), repeat=2):
        prompt = [c[0] for c in combo]
        prev = [c[1] for c in combo]
        new = [c[2] for c in combo]
        trunc = [c[3] for c in combo]
        for td in itertools.product(drops, repeat=2):
            pol, val = run(prompt, prev, new, trunc, list(td))
            rp, rv = set_builder(prompt, prev, new, trunc, list(td))
            assert pol.tolist() == rp and val.tolist() == rv
            n += 1
    assert n > 25000


def test_per_sequence_tail_drop_counts_and_scalar_equivalence():
    rng = np.random.default_rng(4)
    B = 60
    prompt = rng.integers(0, 30, B)
    prev = rng.integers(0, 30, B) * rng.integers(0, 2, B)
    new = rng.integers(0, 40, B)
    trunc = rng.integers(0, 2, B)
    td = rng.integers(0, 50, B)
    pol, val = run(prompt, prev, new, trunc, td)
    assert len(pol) == int(np.sum(np.maximum(0, new - trunc * td)))          # closed form
    assert len(val) == int(np.sum((1 - trunc) * (prev + new)))               # value tokens unaffected
    same = run(prompt, prev, new, trunc, np.full(B, 7))
    scalar = run(prompt, prev, new, trunc, 7)
    assert np.array_equal(same[0], scalar[0]) and np.array_equal(same[1], scalar[1])
    # only the tail goes: what is left of a sequence's policy tokens is a prefix of its new tokens
    sb, seg_b, _ = synth.pack(prompt, prev, new)
    seq_of = np.searchsorted(sb, pol, side="right") - 1
    for i in range(B):
        mine = pol[seq_of == i]
        first_new = seg_b[i] + prev[i]
        assert np.array_equal(mine, np.arange(first_new, first_new + len(mine)))


def test_closed_form_counts_and_disjointness():
    rng = np.random.default_rng(3)
    B = 50
    prompt = rng.integers(0, 30, B)
    prev = rng.integers(0, 30, B) * rng.integers(0, 2, B)
    new = rng.integers(0, 40, B)
    trunc = rng.integers(0, 2, B)
    for td in (0, 7):
        pol, val = run(prompt, prev, new, trunc, td)
        assert len(pol) == int(np.sum(np.maximum(0, new - trunc * td)))
        assert len(val) == int(np.sum((1 - trunc) * (prev + new)))
        sb, seg_b, seg_e = synth.pack(prompt, prev, new)
        seq_of = np.searchsorted(sb, val, side="right") - 1
        assert not np.any(trunc[seq_of])            # no value token in an unfinished sequence
        seq_of = np.searchsorted(sb, pol, side="right") - 1
        assert np.all(pol >= seg_b[seq_of] + prev[seq_of])   # never a prompt / earlier-window token
        assert np.all(np.diff(pol) > 0) and np.all(np.diff(val) > 0)


def test_config1_counts():
    c = synth.config1()
    pol, val = oracle.select_tokens(c["seq_begin"], c["prompt_len"], c["prev_len"], c["new_len"],
                                    c["truncated"])
    assert len(pol) == 170 and len(val) == 42
