"""Writes tests/golden/cfg1_oracle.txt: what the float64 oracle computes on the tiny config
(4 responses, V=1000, seed 0).  Calls only oracle/ and the seeded input generator; no value in
the file comes from the CUDA path.  Run:  python tests/golden/make_cfg1_golden.py
"""
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402
from paper_2506_15050_b200 import synth  # noqa: E402


def compute():
    c = synth.config1()
    adv, ret = oracle.egae(c["rewards"], c["values"], c["seg_begin"], c["seg_end"],
                           c["truncated"], None, c["gamma"], c["lam"])
    pol, val = oracle.select_tokens(c["seq_begin"], c["prompt_len"], c["prev_len"],
                                    c["new_len"], c["truncated"], c["tail_drop"])
    logp_all = oracle.logprob(c["logits"], c["targets"])
    old_logp = (logp_all + c["old_logp_noise"]).astype(np.float32)
    out = oracle.policy_loss(c["logits"], c["targets"], pol, None, old_logp,
                             adv.astype(np.float32), c["eps_low"], c["eps_high"])
    vloss, dv = oracle.value_loss(c["values"], c["old_values"], ret.astype(np.float32), val,
                                  c["xi_low"], c["xi_high"])
    return {
        "n_policy": len(pol), "n_value": len(val),
        "policy_idx_sum": int(pol.astype(np.int64).sum()),
        "value_idx_sum": int(val.astype(np.int64).sum()),
        "adv_sum": float(adv.sum()), "adv_abs_sum": float(np.abs(adv).sum()),
        "ret_sum": float(ret.sum()),
        "adv_first_policy_token": float(adv[pol[0]]),
        "logp_sum": float(out["logp"].sum()),
        "policy_loss": out["loss"], "clip_lo": out["clip_lo"], "clip_hi": out["clip_hi"],
        "dlogits_abs_sum": float(np.abs(out["dlogits"]).sum()),
        "value_loss": vloss, "dvalues_abs_sum": float(np.abs(dv).sum()),
    }


if __name__ == "__main__":
    with open(os.path.join(HERE, "cfg1_oracle.txt"), "w") as f:
        f.write("# written by tests/golden/make_cfg1_golden.py from oracle/ only (config 1, seed 0)\n")
        for k, v in compute().items():
            f.write(f"{k} {v!r}\n")
