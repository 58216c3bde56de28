"""The allocation-free EGAE entry point (tppo_egae_static): for callers that cannot request device
memory -- e.g. a plug-in inside a runtime that has reserved the whole GPU for its own pool, where a
raw cudaMalloc fails -- and have no workspace to lend.  Its scratch is a fixed array inside the
library, shared by all calls, so the test runs it several times in a row (each call meets the
previous call's leftovers) and compares every result with the workspace-taking tppo_egae, bit for
bit (same kernel, same arithmetic, fixed-order reductions), and once with the oracle.  The device's
free memory is read before and after the calls to show that they allocate nothing.  This file is
collected last on purpose; it must pass alone in a fresh process and after all other tests."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import adv_close

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(seed, B, maxlen):
    rng = np.random.default_rng(seed)
    lens = rng.integers(1, maxlen, B)
    gaps = rng.integers(0, 30, B)
    sb = np.cumsum(gaps + np.concatenate([[0], lens[:-1]])).astype(np.int32)
    se = (sb + lens).astype(np.int32)
    N = int(se[-1]) + 5
    host = dict(r=rng.standard_normal(N).astype(np.float32), v=rng.standard_normal(N).astype(np.float32),
                sb=sb, se=se, tr=rng.integers(0, 2, B).astype(np.uint8),
                boot=rng.standard_normal(B).astype(np.float32))
    t = lambda a, dt: torch.from_numpy(a).to(dt).to(DEV)
    return dict(N=N, B=B, host=host, r=t(host["r"], torch.float32), v=t(host["v"], torch.float32),
                sb=t(sb, torch.int32), se=t(se, torch.int32), tr=t(host["tr"], torch.uint8),
                boot=t(host["boot"], torch.float32))


def _with_workspace(b, c, gamma, lam):
    adv, ret = torch.empty(c["N"], device=DEV), torch.empty(c["N"], device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    b.tppo_egae(c["r"], c["v"], c["sb"], c["se"], c["tr"], c["boot"], gamma, lam, adv, ret, st,
                b.workspace(b.OP_EGAE, c["N"], c["B"], 0, 0, DEV))
    torch.cuda.synchronize()
    return adv, ret, int(st)


def test_static_entry_matches_workspace_entry_twice_in_a_row():
    from paper_2506_15050_b200 import binding as b
    big = _case(1, 300, 9000)        # ~1.3 M tokens, several hundred tiles
    small = _case(2, 7, 600)         # a second, smaller call that reuses the dirty scratch
    for c, gamma, lam in ((big, 1.0, 0.95), (small, 0.99, 0.9), (big, 1.0, 1.0)):
        ref_adv, ref_ret, ref_st = _with_workspace(b, c, gamma, lam)
        # outputs exist before the bracket, so the bracket sees only what the call itself does
        adv = torch.full((c["N"],), float("nan"), device=DEV)
        ret = torch.full((c["N"],), float("nan"), device=DEV)
        st = torch.full((1,), -1, dtype=torch.int32, device=DEV)
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        torch_allocs0 = torch.cuda.memory_stats()["allocation.all.allocated"]     # count of requests
        b.tppo_egae_static(c["r"], c["v"], c["sb"], c["se"], c["tr"], c["boot"], gamma, lam, adv, ret, st)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        # neither the driver's pool nor torch's was asked for memory
        assert free1 == free0 and torch.cuda.memory_stats()["allocation.all.allocated"] == torch_allocs0
        assert int(st) == 0 and ref_st == 0
        assert torch.equal(adv, ref_adv) and torch.equal(ret, ref_ret)
        h = c["host"]
        ra, rr = oracle.egae(h["r"], h["v"], h["sb"], h["se"], h["tr"], h["boot"],
                             float(np.float32(gamma)), float(np.float32(lam)))
        assert adv_close(adv.cpu().numpy(), ra, h["sb"], h["se"], 1e-5) <= 1.0
        assert adv_close(ret.cpu().numpy(), rr, h["sb"], h["se"], 1e-5) <= 1.0


def test_static_entry_rejects_sizes_beyond_its_capacity():
    from paper_2506_15050_b200 import binding as b
    n = b.EGAE_STATIC_MAX_TOKENS + 1
    x = torch.zeros(n, device=DEV)
    out = torch.zeros(n, device=DEV)
    one = torch.zeros(1, dtype=torch.int32, device=DEV)
    end = torch.full((1,), n, dtype=torch.int32, device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    with pytest.raises(b.TppoError) as e:
        b.tppo_egae_static(x, x, one, end, torch.zeros(1, dtype=torch.uint8, device=DEV), None, 1.0, 0.95,
                           out, None, st)
    assert e.value.status == 5 and "capacity" in str(e.value)
