"""The calls of one step captured into a CUDA graph (programmatic dependent launches and all) and
replayed: every output equals the eager run's bit for bit, and the replay is repeatable."""
import numpy as np
import pytest
import torch

from paper_2506_15050_b200 import synth
from gpu_util import DEV, dev

pytestmark = pytest.mark.gpu


def test_step_captured_in_a_cuda_graph_matches_eager_calls():
    from paper_2506_15050_b200 import binding as b
    c = synth.config4(seed=11, B=96, lo=16, hi=9000)
    N, B = c["N"], c["B"]
    r, v = dev(c["rewards"], torch.float32), dev(c["values"], torch.float32)
    sb, se = dev(c["seg_begin"], torch.int32), dev(c["seg_end"], torch.int32)
    tr, boot = dev(c["truncated"], torch.uint8), dev(c["bootstrap"], torch.float32)
    seqb = dev(c["seq_begin"], torch.int32)
    pl, pv, nl = (dev(c[k], torch.int32) for k in ("prompt_len", "prev_len", "new_len"))
    pm, vm = dev(c["extra_policy_mask"], torch.uint8), dev(c["extra_value_mask"], torch.uint8)
    old_v = v + 0.25
    V = 4096
    n_rows = 2304          # enough rows for the policy call's side launch
    logits = synth.randn_bf16((n_rows, V), 2.0, 5, DEV)
    targets = torch.randint(0, V, (n_rows,), device=DEV, dtype=torch.int32)
    old_logp = torch.full((N,), -8.0, device=DEV)

    def buffers():
        return dict(adv=torch.full((N,), 7.0, device=DEV), ret=torch.full((N,), 7.0, device=DEV),
                    status=torch.full((1,), -1, dtype=torch.int32, device=DEV),
                    pol=torch.full((N,), -7, dtype=torch.int32, device=DEV),
                    val=torch.full((N,), -7, dtype=torch.int32, device=DEV),
                    counts=torch.full((4,), -1, dtype=torch.int32, device=DEV),
                    vloss=torch.zeros(1, device=DEV), dv=torch.full((N,), 7.0, device=DEV),
                    vst=torch.full((2,), -1, dtype=torch.int32, device=DEV),
                    ploss=torch.zeros(1, device=DEV), logp=torch.zeros(n_rows, device=DEV),
                    tloss=torch.zeros(n_rows, device=DEV),
                    dlogits=torch.zeros_like(logits), pst=torch.full((4,), -1, dtype=torch.int32, device=DEV),
                    ws1=b.workspace(b.OP_EGAE, N, B, 0, 0, DEV), ws2=b.workspace(b.OP_SELECT_TOKENS, N, B, 0, 0, DEV),
                    ws3=b.workspace(b.OP_VALUE_LOSS, N, 0, N, 0, DEV),
                    ws4=b.workspace(b.OP_POLICY_LOSS, n_rows, 0, n_rows, V, DEV))

    def step(o):
        b.tppo_egae(r, v, sb, se, tr, boot, 1.0, 0.95, o["adv"], o["ret"], o["status"], o["ws1"])
        b.tppo_select_tokens(seqb, pl, pv, nl, tr, 0, pm, vm, N, o["pol"], o["val"], o["counts"], o["ws2"])
        b.tppo_value_loss(v, old_v, o["ret"], o["val"], o["counts"][1:2], N, 0.5, 0.6, 0.0, o["vloss"],
                          o["dv"], o["vst"], o["ws3"])
        # the first n_rows policy tokens stand for the micro-batch whose logits are at hand
        b.tppo_policy_loss_fwd_bwd(logits, targets, None, None, n_rows, o["pol"][:n_rows], old_logp, o["adv"],
                                   0.2, 0.28, 0.0, o["logp"], o["tloss"], o["ploss"], o["pst"], o["dlogits"],
                                   b.DLOGITS_COMPACT, o["ws4"])

    eager = buffers()
    step(eager)
    torch.cuda.synchronize()
    assert int(eager["status"]) == 0 and int(eager["counts"][2]) == 0 and int(eager["vst"][1]) == 0
    assert int(eager["counts"][0]) >= n_rows and int(eager["pst"][3]) == 0 and int(eager["pst"][0]) == n_rows

    o = buffers()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step(o)                      # first use of every workspace outside the capture
        torch.cuda.synchronize()
        for k in ("adv", "ret", "dv"):
            o[k].fill_(3.0)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            step(o)
    torch.cuda.synchronize()
    for rep in range(3):
        g.replay()
        torch.cuda.synchronize()
        for k in ("adv", "ret", "status", "pol", "val", "counts", "vloss", "dv", "vst", "ploss", "logp",
                  "tloss", "dlogits", "pst"):
            assert torch.equal(o[k], eager[k]), (k, rep)
