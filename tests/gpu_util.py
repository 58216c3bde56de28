"""Helpers for the GPU parity tests: thin callers of the C ABI (through the binding) that take and
return host numpy arrays.  No arithmetic of the method happens here."""
import numpy as np
import torch

DEV = "cuda:0"


def dev(a, dtype=None):
    if a is None:
        return None
    if isinstance(a, torch.Tensor):
        return a.to(DEV)
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.to(DEV)


def run_egae(B, rewards, values, seg_begin, seg_end, truncated, bootstrap, gamma, lam,
             want_returns=True):
    from paper_2506_15050_b200 import binding as b
    N = len(rewards)
    r, v = dev(rewards, torch.float32), dev(values, torch.float32)
    sb, se, tr = dev(seg_begin, torch.int32), dev(seg_end, torch.int32), dev(truncated, torch.uint8)
    bs = dev(bootstrap, torch.float32)
    adv = torch.full((max(N, 1),), float("nan"), device=DEV)
    ret = torch.full((max(N, 1),), float("nan"), device=DEV) if want_returns else None
    status = torch.full((1,), -1, dtype=torch.int32, device=DEV)
    ws = b.workspace(b.OP_EGAE, N, B, 0, 0, DEV)
    ws.fill_(0xAB)
    b.tppo_egae(r[:N], v[:N], sb, se, tr, bs, gamma, lam, adv[:N], None if ret is None else ret[:N],
                status, ws)
    torch.cuda.synchronize()
    return adv[:N].cpu().numpy(), (None if ret is None else ret[:N].cpu().numpy()), int(status.item())


def run_select(c, tail_drop=0, pm=None, vm=None, N=None, tail_drop_seq=None, strict=True):
    from paper_2506_15050_b200 import binding as b
    N = int(c["seq_begin"][-1]) if N is None else N
    sb = dev(c["seq_begin"], torch.int32)
    pl, pv, nl = (dev(c[k], torch.int32) for k in ("prompt_len", "prev_len", "new_len"))
    tr = dev(c["truncated"], torch.uint8)
    pol = torch.full((max(N, 1),), -7, dtype=torch.int32, device=DEV)
    val = torch.full((max(N, 1),), -7, dtype=torch.int32, device=DEV)
    counts = torch.full((4,), -1, dtype=torch.int32, device=DEV)
    ws = b.workspace(b.OP_SELECT_TOKENS, N, len(c["prompt_len"]), 0, 0, DEV)
    ws.fill_(0xAB)
    b.tppo_select_tokens(sb, pl, pv, nl, tr, tail_drop, dev(pm, torch.uint8), dev(vm, torch.uint8),
                         N, pol, val, counts, ws, tail_drop_seq=dev(tail_drop_seq, torch.int32))
    torch.cuda.synchronize()
    cn = counts.cpu().numpy()
    pol, val = pol.cpu().numpy(), val.cpu().numpy()
    if not strict:       # a call that is expected to give up: whatever was written, anywhere in the lists
        return pol[pol != -7], val[val != -7], cn
    assert np.all(pol[cn[0]:] == -7) and np.all(val[cn[1]:] == -7)   # nothing past the counts
    return pol[:cn[0]], val[:cn[1]], cn


def run_policy(logits_t, targets, rows, aux_idx, old_logp, adv, eps_low, eps_high, denom=0.0,
               mode=2, hint=0, n_sel=None, n_max=None, inplace=False, V=None):
    """logits_t: torch tensor on DEV (bf16 or fp32), possibly a strided view.  Returns a dict of
    host arrays; dlogits as float32 numpy (compact [n_max,V] or full [R,V])."""
    from paper_2506_15050_b200 import binding as b
    R = logits_t.shape[0]
    V = logits_t.shape[1] if V is None else V
    t = dev(targets, torch.int32)
    rw = dev(rows, torch.int32)
    ax = dev(aux_idx, torch.int32)
    ol, ad = dev(old_logp, torch.float32), dev(adv, torch.float32)
    if n_max is None:
        n_max = R if rows is None else len(rows)
    ns = None if n_sel is None else torch.tensor([n_sel], dtype=torch.int32, device=DEV)
    logp = torch.full((max(n_max, 1),), float("nan"), device=DEV)
    tl = torch.full((max(n_max, 1),), float("nan"), device=DEV)
    loss = torch.full((1,), float("nan"), device=DEV)
    stats = torch.full((4,), -1, dtype=torch.int32, device=DEV)
    if mode == b.DLOGITS_NONE:
        dl = None
    elif mode == b.DLOGITS_FULL:
        if inplace:
            dl = logits_t
        else:   # FULL mode shares the logits' row stride
            dl = torch.full((R, logits_t.stride(0)), float("nan"), dtype=logits_t.dtype, device=DEV)[:, :logits_t.shape[1]]
    else:
        dl = torch.full((max(n_max, 1), V), float("nan"), dtype=logits_t.dtype, device=DEV)
    ws = b.workspace(b.OP_POLICY_LOSS, R, 0, n_max, V, DEV)
    ws.fill_(0xAB)
    b.tppo_policy_loss_fwd_bwd(logits_t, t, rw, ns, n_max, ax, ol, ad, eps_low, eps_high, denom,
                               logp, tl, loss, stats, dl, mode, ws, kernel_hint=hint, V=V)
    torch.cuda.synchronize()
    st = stats.cpu().numpy()
    return dict(logp=logp.cpu().numpy(), token_loss=tl.cpu().numpy(), loss=float(loss.item()),
                n=int(st[0]), clip_lo=int(st[1]), clip_hi=int(st[2]), status=int(st[3]),
                dlogits=None if dl is None else dl, )


def run_value(values, old_values, returns, value_idx, xi_low, xi_high, denom=0.0, n_sel=None,
              want_grad=True):
    from paper_2506_15050_b200 import binding as b
    N = len(values)
    v, vo, R = (dev(x, torch.float32) for x in (values, old_values, returns))
    ix = dev(value_idx, torch.int32)
    n_max = N if value_idx is None else len(value_idx)
    ns = None if n_sel is None else torch.tensor([n_sel], dtype=torch.int32, device=DEV)
    loss = torch.full((1,), float("nan"), device=DEV)
    dv = torch.full((max(N, 1),), float("nan"), device=DEV) if want_grad else None
    stats = torch.full((2,), -1, dtype=torch.int32, device=DEV)
    ws = b.workspace(b.OP_VALUE_LOSS, N, 0, n_max, 0, DEV)
    ws.fill_(0xAB)
    b.tppo_value_loss(v, vo, R, ix, ns, n_max, xi_low, xi_high, denom, loss,
                      None if dv is None else dv[:N], stats, ws)
    torch.cuda.synchronize()
    st = stats.cpu().numpy()
    return float(loss.item()), (None if dv is None else dv[:N].cpu().numpy()), int(st[0]), int(st[1])


def adv_close(gpu, ref, seg_begin, seg_end, rtol=1e-5):
    """Largest |gpu - ref| / tol over the segments, tol = rtol * max(|ref|, 1) element by element:
    the relative bound for fp32 advantages and returns, with a floor of 1 only where the exact
    value is 0 or tiny (the last token of a cut response with gamma = 1 has advantage exactly 0).
    Positions outside every segment must be exactly 0."""
    worst = 0.0
    inside = np.zeros(len(ref), bool)
    for b, e in zip(seg_begin, seg_end):
        if e <= b:
            continue
        inside[b:e] = True
        err = np.abs(gpu[b:e].astype(np.float64) - ref[b:e])
        worst = max(worst, float(np.max(err / (rtol * np.maximum(np.abs(ref[b:e]), 1.0)))))
    assert np.all(gpu[~inside] == 0.0)
    return worst


def worst_relative_error(gpu, ref, floor=1.0):
    """Largest |gpu - ref| / |ref| over the elements with |ref| >= floor (reported by the tests)."""
    big = np.abs(ref) >= floor
    if not big.any():
        return 0.0
    return float(np.max(np.abs(gpu[big].astype(np.float64) - ref[big]) / np.abs(ref[big])))
