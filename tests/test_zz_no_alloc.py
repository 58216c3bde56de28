"""The allocation-free EGAE entry point (tppo_egae_static): for callers that cannot request device
memory -- e.g. a plug-in inside a runtime that has reserved the whole GPU for its own pool, where a
raw cudaMalloc fails -- and have no workspace to lend.  Its scratch is a fixed array inside the
library, shared by all calls, so the test runs it twice in a row (the second call meets the first
call's leftovers) and compares both results with the workspace-taking tppo_egae.  This file is
collected last on purpose; it must pass alone in a fresh process and after all other tests."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(seed, B, maxlen):
    rng = np.random.default_rng(seed)
    lens = rng.integers(1, maxlen, B)
    gaps = rng.integers(0, 30, B)
    sb = np.cumsum(gaps + np.concatenate([[0], lens[:-1]])).astype(np.int32)
    se = (sb + lens).astype(np.int32)
    N = int(se[-1]) + 5
    t = lambda a, dt: torch.from_numpy(a).to(dt).to(DEV)
    return dict(N=N, B=B, r=t(rng.standard_normal(N).astype(np.float32), torch.float32),
                v=t(rng.standard_normal(N).astype(np.float32), torch.float32),
                sb=t(sb, torch.int32), se=t(se, torch.int32),
                tr=t(rng.integers(0, 2, B).astype(np.uint8), torch.uint8),
                boot=t(rng.standard_normal(B).astype(np.float32), torch.float32))


def _with_workspace(b, c, gamma, lam):
    adv, ret = torch.empty(c["N"], device=DEV), torch.empty(c["N"], device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    b.tppo_egae(c["r"], c["v"], c["sb"], c["se"], c["tr"], c["boot"], gamma, lam, adv, ret, st,
                b.workspace(b.OP_EGAE, c["N"], c["B"], 0, 0, DEV))
    torch.cuda.synchronize()
    return adv, ret, int(st)


def _static(b, c, gamma, lam):
    adv = torch.full((c["N"],), float("nan"), device=DEV)
    ret = torch.full((c["N"],), float("nan"), device=DEV)
    st = torch.full((1,), -1, dtype=torch.int32, device=DEV)
    b.tppo_egae_static(c["r"], c["v"], c["sb"], c["se"], c["tr"], c["boot"], gamma, lam, adv, ret, st)
    torch.cuda.synchronize()
    return adv, ret, int(st)


def test_static_entry_matches_workspace_entry_twice_in_a_row():
    from paper_2506_15050_b200 import binding as b
    big = _case(1, 300, 9000)        # ~1.3 M tokens, several hundred tiles
    small = _case(2, 7, 600)         # a second, smaller call that reuses the dirty scratch
    for c, gamma, lam in ((big, 1.0, 0.95), (small, 0.99, 0.9), (big, 1.0, 1.0)):
        ref_adv, ref_ret, ref_st = _with_workspace(b, c, gamma, lam)
        adv, ret, st = _static(b, c, gamma, lam)
        assert st == 0 and ref_st == 0
        # same kernel, same arithmetic: the advantage tolerance of the other tests (1e-5) is met exactly
        scale = max(1.0, float(ref_adv.abs().max()))
        assert float((adv - ref_adv).abs().max()) <= 1e-5 * scale
        assert float((ret - ref_ret).abs().max()) <= 1e-5 * max(1.0, float(ref_ret.abs().max()))


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
