"""GPU parity of the forward-only statistics sweep (tppo_policy_logprob_stats: old-policy log-probs,
softmax entropy, mean entropy, mean old_logp - logp) against the oracle.  Tolerances: log-probs and
entropies 2e-3 absolute (bf16 logits, fp32 accumulation), the two means likewise."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_15050_b200 import binding as b
from paper_2506_15050_b200 import synth
from gpu_util import DEV, dev

pytestmark = pytest.mark.gpu
ATOL = 2e-3


def run_stats(logits_t, targets, rows, aux, old_logp, n_sel=None, want_entropy=True, V=None):
    R = logits_t.shape[0]
    V = logits_t.shape[1] if V is None else V
    n_max = R if rows is None else len(rows)
    logp = torch.full((max(n_max, 1),), float("nan"), device=DEV)
    ent = torch.full((max(n_max, 1),), float("nan"), device=DEV) if want_entropy else None
    means = torch.full((2,), float("nan"), device=DEV)
    stats = torch.full((4,), -1, dtype=torch.int32, device=DEV)
    ns = None if n_sel is None else torch.tensor([n_sel], dtype=torch.int32, device=DEV)
    ws = b.workspace(b.OP_POLICY_LOSS, R, 0, n_max, V, DEV)
    ws.fill_(0xAB)
    b.tppo_policy_logprob_stats(logits_t, dev(targets, torch.int32), dev(rows, torch.int32), ns, n_max,
                                dev(aux, torch.int32), dev(old_logp, torch.float32), logp, ent, means,
                                stats, ws, V=V)
    torch.cuda.synchronize()
    return (logp.cpu().numpy(), None if ent is None else ent.cpu().numpy(), means.cpu().numpy(),
            stats.cpu().numpy())


@pytest.mark.parametrize("V,ld,dtype", [(152064, 152064, torch.bfloat16), (1001, 1008, torch.bfloat16),
                                        (1001, 1001, torch.float32), (32000, 32768, torch.float32),
                                        (50264, 50264, torch.bfloat16)])
def test_stats_match_oracle(V, ld, dtype):
    rng = np.random.default_rng(V)
    R = 40
    x = (2.5 * rng.standard_normal((R, ld))).astype(np.float32)
    full = torch.from_numpy(x).to(dtype).to(DEV)
    xt = full[:, :V]
    host = (synth.bf16_bits(full) if dtype == torch.bfloat16 else x)[:, :V]
    y = rng.integers(0, V, R).astype(np.int32)
    y[0], y[1] = 0, V - 1
    rows = np.sort(rng.choice(R, 29, replace=False)).astype(np.int32)
    aux = rng.permutation(64)[:29].astype(np.int32)
    old = rng.standard_normal(64).astype(np.float32) - 9.0
    ref = oracle.logprob_stats(host, y, rows, aux, old)
    logp, ent, means, st = run_stats(xt, y, rows, aux, old, V=V)
    assert st[0] == 29 and st[3] == 0
    np.testing.assert_allclose(logp[:29], ref["logp"], rtol=0, atol=ATOL)
    np.testing.assert_allclose(ent[:29], ref["entropy"], rtol=0, atol=ATOL)
    assert abs(means[0] - ref["mean_entropy"]) <= ATOL and abs(means[1] - ref["mean_kl"]) <= ATOL
    # identity rows, no old log-probs, no per-row entropy, a device-side count
    ref2 = oracle.logprob_stats(host, y, np.arange(17, dtype=np.int32))
    logp2, ent2, means2, st2 = run_stats(xt, y, None, None, None, n_sel=17, want_entropy=False, V=V)
    assert st2[0] == 17 and st2[3] == 0 and ent2 is None and means2[1] == 0.0
    np.testing.assert_allclose(logp2[:17], ref2["logp"], rtol=0, atol=ATOL)
    assert abs(means2[0] - ref2["mean_entropy"]) <= ATOL
    # run-to-run identical
    again = run_stats(xt, y, rows, aux, old, V=V)
    assert np.array_equal(again[0], logp) and np.array_equal(again[1], ent) and np.array_equal(again[2], means)


def test_stats_closed_forms_and_skipped_rows():
    V = 8192
    x = np.zeros((7, V), np.float32)
    x[0, :] = 3.25                              # uniform: entropy log V
    x[1, :] = -np.inf
    x[1, 77] = 1.0                              # one-hot: entropy 0, log-prob 0
    x[2, :] = -np.inf
    x[2, [5, 4000]] = -2.0                      # two equal entries: log 2
    x[3, :] = np.linspace(-30, 30, V)
    x[4, 9] = np.nan                            # no softmax: skipped, reported
    x[5, :] = -np.inf                           # likewise
    x[6, :] = 3.3895313892515355e38             # the largest finite bf16 everywhere: uniform
    xt = torch.from_numpy(x).to(torch.bfloat16).to(DEV)
    y = np.array([1, 77, 5, V - 1, 0, 0, 3], np.int32)
    y_bad = y.copy()
    logp, ent, means, st = run_stats(xt, y, None, None, None)
    assert st[0] == 7 and st[3] == b.DEV_NONFINITE
    good = np.array([0, 1, 2, 3, 6], np.int32)
    ref = oracle.logprob_stats(synth.bf16_bits(xt), y, good)
    np.testing.assert_allclose(ent[good], ref["entropy"], rtol=0, atol=ATOL)
    np.testing.assert_allclose(logp[good], ref["logp"], rtol=0, atol=ATOL)
    np.testing.assert_allclose(ent[[0, 1, 2, 6]], [np.log(V), 0.0, np.log(2.0), np.log(V)], atol=ATOL)
    assert np.all(logp[[4, 5]] == 0) and np.all(ent[[4, 5]] == 0)
    assert abs(means[0] - ref["entropy"].sum() / 7) <= ATOL        # skipped rows add nothing, n divides
    y_bad[3] = V                                 # a target outside the vocabulary: skipped, reported
    logp, ent, means, st = run_stats(xt, y_bad, None, None, None)
    assert st[3] == (b.DEV_NONFINITE | b.DEV_BAD_TARGET) and logp[3] == 0 and ent[3] == 0


def test_stats_config3_rows():
    """Rows of the headline shape: [512, 152064] bf16 of config 3's logits, old log-probs through the
    selected-position index map."""
    c = synth.config3(DEV, n_tokens=512)
    n = c["n_tokens"]
    host = synth.bf16_bits(c["logits"])
    pol, _ = oracle.select_tokens(c["seq_begin"], c["prompt_len"], c["prev_len"], c["new_len"],
                                  c["truncated"], 0, c["extra_policy_mask"], c["extra_value_mask"])
    old = np.zeros(c["N"], np.float32)
    old[pol] = oracle.logprob(host, c["targets"]) + c["old_logp_noise"][pol]
    ref = oracle.logprob_stats(host, c["targets"], None, pol, old)
    logp, ent, means, st = run_stats(c["logits"], c["targets"], None, pol, old)
    assert st[0] == n and st[3] == 0
    np.testing.assert_allclose(logp, ref["logp"], rtol=0, atol=ATOL)
    np.testing.assert_allclose(ent, ref["entropy"], rtol=0, atol=ATOL)
    assert abs(means[0] - ref["mean_entropy"]) <= ATOL and abs(means[1] - ref["mean_kl"]) <= 1e-4
