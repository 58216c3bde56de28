"""Pins for the oracle's successive-batching step (Section 3.2, batching figure; the batch
collection step of Algorithm 1):
an independent list-based restatement, exhaustive enumeration on tiny batches, and invariants."""
import itertools

import numpy as np

import oracle
from paper_2506_15050_b200 import synth


def by_lists(prompt, prev, new, trunc, tokens, queue):
    """The same rule with Python lists of token lists (no offsets, no packing)."""
    starts = np.concatenate([[0], np.cumsum(np.array(prompt) + np.array(prev) + np.array(new))]).astype(int)
    seqs = [list(tokens[starts[i]:starts[i + 1]]) for i in range(len(prompt))]
    waiting = list(queue)
    out, src, free = [], [], []
    for i, s in enumerate(seqs):
        if trunc[i]:
            out.append((prompt[i], prev[i] + new[i], s)); src.append(-1)
        else:
            free.append(i)
            k = len(free) - 1
            if k < len(queue):
                out.append((len(waiting[k]), 0, list(waiting[k]))); src.append(k)
            else:
                out.append((0, 0, [])); src.append(-2)
    return out, src, free


def run(prompt, prev, new, trunc, tokens, queue, capacity=None):
    sb, _, _ = synth.pack(prompt, prev, new)
    qb = np.concatenate([[0], np.cumsum([len(q) for q in queue])]).astype(np.int32)
    qt = np.array([t for q in queue for t in q], np.int32)
    return oracle.advance_batch(sb, prompt, prev, new, trunc, tokens, qb, qt, capacity)


def check(prompt, prev, new, trunc, queue, rng):
    N = int(np.sum(prompt) + np.sum(prev) + np.sum(new))
    tokens = rng.integers(0, 1000, N).astype(np.int32)
    got = run(prompt, prev, new, trunc, tokens, queue)
    ref, src, free = by_lists(prompt, prev, new, trunc, tokens, queue)
    assert got["free_slots"].tolist() == free and got["slot_source"].tolist() == src
    assert got["next_prompt_len"].tolist() == [r[0] for r in ref]
    assert got["next_prev_len"].tolist() == [r[1] for r in ref]
    flat = [t for r in ref for t in r[2]]
    assert got["next_tokens"].tolist() == flat and got["total"] == len(flat)
    lens = [len(r[2]) for r in ref]
    assert got["next_seq_begin"].tolist() == np.concatenate([[0], np.cumsum(lens)]).astype(int).tolist()
    assert got["n_free"] == len(free) and got["n_refilled"] == min(len(free), len(queue))


def test_exhaustive_small_batches():
    rng = np.random.default_rng(0)
    lens = (0, 1, 3)
    n = 0
    for B in (1, 2, 3):
        for combo in itertools.product(itertools.product(lens, (0, 2), lens, (0, 1)), repeat=B):
            prompt, prev, new, trunc = (np.array([c[j] for c in combo], np.int32) for j in range(4))
            for queue in ([], [[5, 6]], [[7], [], [8, 9, 10]]):
                check(prompt, prev, new, trunc.astype(np.uint8), queue, rng)
                n += 1
    assert n > 15000


def test_invariants_on_a_ragged_batch():
    rng = np.random.default_rng(1)
    B = 300
    prompt = rng.integers(1, 50, B).astype(np.int32)
    prev = (rng.integers(0, 3, B) * rng.integers(0, 400, B)).astype(np.int32)
    new = rng.integers(1, 200, B).astype(np.int32)
    trunc = (rng.random(B) < 0.5).astype(np.uint8)
    queue = [list(rng.integers(0, 1000, rng.integers(1, 60))) for _ in range(int((1 - trunc).sum()) - 3)]
    check(prompt, prev, new, trunc, queue, rng)
    N = int((prompt + prev + new).sum())
    tokens = np.arange(N, dtype=np.int32)            # token id = its old position
    got = run(prompt, prev, new, trunc, tokens, queue)
    sb, _, _ = synth.pack(prompt, prev, new)
    kept = np.concatenate([np.arange(sb[i], sb[i + 1]) for i in range(B) if trunc[i]])
    from_old = got["next_tokens"][np.concatenate(
        [np.arange(got["next_seq_begin"][i], got["next_seq_begin"][i + 1]) for i in range(B) if trunc[i]])]
    assert np.array_equal(from_old, kept)            # every kept token survives, in order
    assert got["total"] == len(kept) + sum(len(q) for q in queue)
    assert np.all(got["next_prev_len"][trunc == 1] == (prev + new)[trunc == 1])
    assert np.all(got["next_prev_len"][trunc == 0] == 0)
    assert (got["slot_source"] == -2).sum() == 3     # queue ran out three slots early


def test_config1_and_capacity_limit():
    c = synth.config1()
    tokens = np.arange(c["N"], dtype=np.int32)
    queue = [[1, 2, 3], [4, 5]]
    got = run(c["prompt_len"], c["prev_len"], c["new_len"], c["truncated"], tokens, queue)
    assert got["free_slots"].tolist() == [0, 2] and got["slot_source"].tolist() == [0, -1, 1, -1]
    assert got["next_prompt_len"].tolist() == [3, 16, 2, 16] and got["next_prev_len"].tolist() == [0, 64, 0, 64]
    assert got["total"] == 3 + 80 + 2 + 80
    small = run(c["prompt_len"], c["prev_len"], c["new_len"], c["truncated"], tokens, queue, capacity=50)
    assert small["total"] == 165 and np.array_equal(small["next_tokens"], got["next_tokens"][:50])
