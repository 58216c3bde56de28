"""Seeded synthetic workloads shaped like T-PPO's long-CoT training batches.

This module only draws random inputs and lays sequences out in packed form.  It contains none
of the method's arithmetic (no advantage, filter, softmax or loss computation), so both the
CUDA path and the CPU oracle may be fed from it.  Small arrays come from numpy's PCG64
(bit-reproducible on any host); the large logit / hidden / weight tensors come from torch's
generator on the device they are asked for, and whoever needs them elsewhere copies them.

Packed layout: sequence i occupies positions [seq_begin[i], seq_begin[i+1]) as
``prompt | tokens generated in earlier windows | tokens generated in this window``.
Its response segment (the tokens that carry a value and a reward) is everything after the
prompt.  ``truncated[i]`` is 1 when generation stopped at the window limit without an end
condition (Section 3.2 of the paper).
"""
from __future__ import annotations

import numpy as np
import torch

V_QWEN = 152064


def pack(prompt_len, prev_len, new_len):
    """cu-seqlens style offsets plus the response segment of every sequence."""
    prompt_len = np.asarray(prompt_len, np.int32)
    prev_len = np.asarray(prev_len, np.int32)
    new_len = np.asarray(new_len, np.int32)
    tot = prompt_len.astype(np.int64) + prev_len + new_len
    seq_begin = np.zeros(len(tot) + 1, np.int64)
    np.cumsum(tot, out=seq_begin[1:])
    assert seq_begin[-1] < 2**31
    seq_begin = seq_begin.astype(np.int32)
    seg_begin = (seq_begin[:-1] + prompt_len).astype(np.int32)
    seg_end = seq_begin[1:].astype(np.int32).copy()
    return seq_begin, seg_begin, seg_end


def _terminal_rewards(rng, N, seg_end, truncated):
    """+1 / -1 (fair coin) on the last token of every finished response, 0 elsewhere."""
    r = np.zeros(N, np.float32)
    for e, t in zip(seg_end, truncated):
        coin = rng.integers(0, 2)
        if not t and e > 0:
            r[e - 1] = 1.0 if coin else -1.0
    return r


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """Bit patterns of a bf16 tensor as a uint16 numpy array (host copy, no arithmetic)."""
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def randn_bf16(shape, std, seed, device, chunk_rows=2048):
    """bf16 N(0, std) tensor filled chunk by chunk so that the fp32 temporary stays small."""
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    rows = shape[0]
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        tmp = torch.randn((r1 - r0,) + tuple(shape[1:]), generator=g, device=device,
                          dtype=torch.float32)
        out[r0:r1] = (tmp * std).to(torch.bfloat16)
    return out


# ---------------------------------------------------------------------------------------------
# config 1: tiny CPU-seconds case
# ---------------------------------------------------------------------------------------------
def config1(seed: int = 0):
    rng = np.random.default_rng(seed)
    B, V = 4, 1000
    prompt = np.full(B, 16, np.int32)
    prev = np.zeros(B, np.int32)
    new = np.array([37, 64, 5, 64], np.int32)
    truncated = np.array([0, 1, 0, 1], np.uint8)
    seq_begin, seg_begin, seg_end = pack(prompt, prev, new)
    N = int(seq_begin[-1])
    logits = rng.standard_normal((N, V)).astype(np.float32)
    targets = rng.integers(0, V, N).astype(np.int32)
    values = (0.5 * rng.standard_normal(N)).astype(np.float32)
    old_values = (values + 0.2 * rng.standard_normal(N)).astype(np.float32)
    rewards = _terminal_rewards(rng, N, seg_end, truncated)
    old_logp_noise = (0.05 * rng.standard_normal(N)).astype(np.float32)
    return dict(name="cfg1", B=B, N=N, V=V, W=64, prompt_len=prompt, prev_len=prev, new_len=new,
                truncated=truncated, seq_begin=seq_begin, seg_begin=seg_begin, seg_end=seg_end,
                logits=logits, targets=targets, values=values, old_values=old_values,
                rewards=rewards, old_logp_noise=old_logp_noise, bootstrap=None,
                gamma=1.0, lam=0.95, eps_low=0.2, eps_high=0.2, xi_low=0.5, xi_high=0.6,
                tail_drop=0)


# ---------------------------------------------------------------------------------------------
# config 2: Qwen2.5-7B-shaped micro-batch, 8 packed sequences, 8192 rows
# ---------------------------------------------------------------------------------------------
def config2_meta(seed: int = 1, n_rows: int = 8192, B: int = 8, prompt: int = 512):
    rng = np.random.default_rng(seed)
    W = 1024
    raw = np.minimum(W, np.rint(rng.lognormal(np.log(900.0), 0.51, B))).astype(np.int64)
    truncated = (raw >= W).astype(np.uint8)
    if truncated.sum() == 0:
        truncated[int(np.argmax(raw))] = 1
    budget = n_rows - B * prompt
    new = np.floor(raw * (budget / raw.sum())).astype(np.int64)
    new[-1] += budget - new.sum()
    prompt_len = np.full(B, prompt, np.int32)
    prev = np.zeros(B, np.int32)
    seq_begin, seg_begin, seg_end = pack(prompt_len, prev, new)
    N = int(seq_begin[-1])
    assert N == n_rows
    values = (0.5 * rng.standard_normal(N)).astype(np.float32)
    old_values = (values + 0.2 * rng.standard_normal(N)).astype(np.float32)
    rewards = _terminal_rewards(rng, N, seg_end, truncated)
    noise = (0.05 * rng.standard_normal(N)).astype(np.float32)
    return dict(name="cfg2", B=B, N=N, W=W, prompt_len=prompt_len, prev_len=prev,
                new_len=new.astype(np.int32), truncated=truncated, seq_begin=seq_begin,
                seg_begin=seg_begin, seg_end=seg_end, values=values, old_values=old_values,
                rewards=rewards, old_logp_noise=noise, bootstrap=None, rng=rng,
                gamma=1.0, lam=0.95, eps_low=0.2, eps_high=0.2, xi_low=0.5, xi_high=0.6,
                tail_drop=0)


def config2(device, V: int = V_QWEN, seed: int = 1, n_rows: int = 8192, B: int = 8,
            prompt: int = 512):
    c = config2_meta(seed, n_rows, B, prompt)
    rng = c.pop("rng")
    c["V"] = V
    c["targets"] = rng.integers(0, V, c["N"]).astype(np.int32)
    c["logits"] = randn_bf16((c["N"], V), 2.0, seed, device)
    return c


# ---------------------------------------------------------------------------------------------
# config 3: Qwen2.5-32B-shaped long-CoT step (full batch) and its loss micro-batch
# ---------------------------------------------------------------------------------------------
def config3_batch(seed: int = 2, B: int = 512, prompt: int = 256, W: int = 8192,
                  median: float = 3000.0):
    rng = np.random.default_rng(seed)
    new = np.minimum(W, np.maximum(1, np.rint(rng.lognormal(np.log(median), 1.0, B))))
    new = new.astype(np.int64)
    at_cap = new >= W
    truncated = (at_cap | (rng.random(B) < 0.41)).astype(np.uint8)
    carried = rng.random(B) < 0.25
    prev = np.where(carried, rng.integers(1, W + 1, B), 0).astype(np.int64)
    prompt_len = np.full(B, prompt, np.int32)
    seq_begin, seg_begin, seg_end = pack(prompt_len, prev, new)
    N = int(seq_begin[-1])
    values = (0.5 * rng.standard_normal(N)).astype(np.float32)
    old_values = (values + 0.2 * rng.standard_normal(N)).astype(np.float32)
    rewards = _terminal_rewards(rng, N, seg_end, truncated)
    noise = (0.05 * rng.standard_normal(N)).astype(np.float32)
    return dict(name="cfg3", B=B, N=N, W=W, prompt_len=prompt_len, prev_len=prev.astype(np.int32),
                new_len=new.astype(np.int32), truncated=truncated, seq_begin=seq_begin,
                seg_begin=seg_begin, seg_end=seg_end, values=values, old_values=old_values,
                rewards=rewards, old_logp_noise=noise, bootstrap=None, rng=rng,
                gamma=1.0, lam=0.95, eps_low=0.2, eps_high=0.2, xi_low=0.5, xi_high=0.6,
                tail_drop=0)


def config3_microbatch_masks(c, n_tokens: int = 16384, n_resp: int = 32):
    """Independent policy / value byte masks that keep exactly n_tokens tokens each, drawn from
    the first n_resp responses that can supply them (policy: this-window tokens of any of them;
    value: all generated tokens of the finished ones)."""
    rng = c["rng"]
    N, B = c["N"], c["B"]
    sb, pl, pv, nl, tr = (c["seq_begin"], c["prompt_len"], c["prev_len"], c["new_len"],
                          c["truncated"])
    pol_pos, val_pos = [], []
    taken = 0
    for i in range(B):
        if taken >= n_resp:
            break
        taken += 1
        new0 = int(sb[i]) + int(pl[i]) + int(pv[i])
        pol_pos.append(np.arange(new0, new0 + int(nl[i]), dtype=np.int64))
        if not tr[i]:
            val_pos.append(np.arange(int(sb[i]) + int(pl[i]), int(sb[i + 1]), dtype=np.int64))
    pol_pos = np.concatenate(pol_pos)
    val_pos = np.concatenate(val_pos) if val_pos else np.zeros(0, np.int64)
    n_pol = min(n_tokens, len(pol_pos))
    n_val = min(n_tokens, len(val_pos))
    pm = np.zeros(N, np.uint8)
    vm = np.zeros(N, np.uint8)
    pm[rng.choice(pol_pos, n_pol, replace=False)] = 1
    vm[rng.choice(val_pos, n_val, replace=False)] = 1
    return pm, vm


def config3(device, V: int = V_QWEN, seed: int = 2, n_tokens: int = 16384, B: int = 512,
            W: int = 8192, median: float = 3000.0, n_resp: int = 32, with_logits: bool = True):
    c = config3_batch(seed, B=B, W=W, median=median)
    pm, vm = config3_microbatch_masks(c, n_tokens, n_resp)
    rng = c.pop("rng")
    c["extra_policy_mask"], c["extra_value_mask"] = pm, vm
    c["V"] = V
    c["n_tokens"] = int(pm.sum())
    # logits row j scores the j-th selected policy token (ascending position order)
    c["targets"] = rng.integers(0, V, c["n_tokens"]).astype(np.int32)
    if with_logits:
        c["logits"] = randn_bf16((c["n_tokens"], V), 2.0, seed, device)
    return c


# ---------------------------------------------------------------------------------------------
# config 4: EGAE + compaction scaling sweep
# ---------------------------------------------------------------------------------------------
def config4(seed: int = 3, B: int = 4096, lo: int = 16, hi: int = 32768):
    rng = np.random.default_rng(seed)
    lens = np.rint(np.exp(rng.uniform(np.log(lo), np.log(hi), B))).astype(np.int64)
    zeros = np.zeros(B, np.int32)
    seq_begin, seg_begin, seg_end = pack(zeros, zeros, lens)
    N = int(seq_begin[-1])
    truncated = (rng.random(B) < 0.5).astype(np.uint8)
    bootstrap = (0.5 * rng.standard_normal(B)).astype(np.float32)
    values = (0.5 * rng.standard_normal(N, dtype=np.float32)).astype(np.float32)
    rewards = _terminal_rewards(rng, N, seg_end, truncated)
    mask = (rng.random(N, dtype=np.float32) < 0.5).astype(np.uint8)
    return dict(name="cfg4", B=B, N=N, prompt_len=zeros, prev_len=zeros.copy(),
                new_len=lens.astype(np.int32), truncated=truncated, seq_begin=seq_begin,
                seg_begin=seg_begin, seg_end=seg_end, values=values, rewards=rewards,
                bootstrap=bootstrap, extra_policy_mask=mask, extra_value_mask=mask[::-1].copy(),
                gamma=1.0, lams=(0.9, 0.95, 1.0), tail_drops=(0, 16))


# ---------------------------------------------------------------------------------------------
# config 5: fused LM-head variant (hidden x vocabulary contraction)
# ---------------------------------------------------------------------------------------------
def config5(device, M: int = 16384, K: int = 5120, V: int = V_QWEN, seed: int = 4):
    rng = np.random.default_rng(seed)
    hidden = randn_bf16((M, K), 1.0, seed, device)
    weight = randn_bf16((K, V), 0.02, seed + 1000, device)
    targets = rng.integers(0, V, M).astype(np.int32)
    adv = rng.standard_normal(M).astype(np.float32)
    noise = (0.05 * rng.standard_normal(M)).astype(np.float32)
    return dict(name="cfg5", M=M, K=K, V=V, hidden=hidden, weight=weight, targets=targets,
                adv=adv, old_logp_noise=noise, eps_low=0.2, eps_high=0.2)
