"""float64 CPU oracle for the T-PPO token-selective update path (ctypes view of tppo_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the benchmark's
CPU-baseline leg.  The product package never imports this module and this module never
imports the product package.  All arithmetic lives in tppo_oracle.c; this file only marshals
numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tppo_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile tppo_oracle.c with gcc (OpenMP over independent rows / segments)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
               "-ffp-contract=off", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_LIB)
        _lib.oracle_num_threads.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _arr(a, dtype):
    if a is None:
        return None
    return np.ascontiguousarray(np.asarray(a), dtype=dtype)


def _logits_view(logits):
    """Return (array, dtype_code, ld).  uint16 arrays are bf16 bit patterns."""
    a = np.asarray(logits)
    assert a.ndim == 2 and a.strides[1] == a.itemsize
    if a.dtype == np.uint16:
        code = 0
    elif a.dtype == np.float32:
        code = 1
    elif a.dtype == np.float64:
        code = 2
    else:
        raise TypeError("logits must be uint16 (bf16 bits), float32 or float64")
    return a, code, a.strides[0] // a.itemsize


def egae(rewards, values, seg_begin, seg_end, truncated, bootstrap, gamma, lam,
         want_returns=True):
    r = _arr(rewards, np.float32)
    v = _arr(values, np.float32)
    sb = _arr(seg_begin, np.int32)
    se = _arr(seg_end, np.int32)
    tr = _arr(truncated, np.uint8)
    bs = _arr(bootstrap, np.float32)
    N, B = r.shape[0], sb.shape[0]
    adv = np.empty(N, np.float64)
    ret = np.empty(N, np.float64) if want_returns else None
    lib().oracle_egae(_p(r), _p(v), _p(sb), _p(se), _p(tr), _p(bs), C.c_int32(B),
                      C.c_int64(N), C.c_double(gamma), C.c_double(lam), _p(adv), _p(ret))
    return adv, ret


def select_tokens(seq_begin, prompt_len, prev_len, new_len, truncated, tail_drop=0,
                  extra_policy_mask=None, extra_value_mask=None, N=None, tail_drop_seq=None):
    sb = _arr(seq_begin, np.int32)
    pl = _arr(prompt_len, np.int32)
    pv = _arr(prev_len, np.int32)
    nl = _arr(new_len, np.int32)
    tr = _arr(truncated, np.uint8)
    B = pl.shape[0]
    if N is None:
        N = int(sb[-1]) if B > 0 else 0
    em = _arr(extra_policy_mask, np.uint8)
    ev = _arr(extra_value_mask, np.uint8)
    pol = np.empty(max(N, 1), np.int32)
    val = np.empty(max(N, 1), np.int32)
    counts = np.zeros(2, np.int64)
    tds = _arr(tail_drop_seq, np.int32)
    assert tds is None or tds.shape[0] == B
    lib().oracle_select_tokens(_p(sb), _p(pl), _p(pv), _p(nl), _p(tr), C.c_int32(tail_drop),
                               _p(tds), _p(em), _p(ev), C.c_int32(B), C.c_int64(N),
                               _p(pol), _p(val), _p(counts))
    return pol[:counts[0]].copy(), val[:counts[1]].copy()


def logprob(logits, targets, rows=None):
    a, code, ld = _logits_view(logits)
    t = _arr(targets, np.int32)
    rw = _arr(rows, np.int32)
    n = a.shape[0] if rw is None else rw.shape[0]
    out = np.empty(n, np.float64)
    lib().oracle_logprob(_p(a), C.c_int(code), C.c_int32(a.shape[1]), C.c_int64(ld),
                         _p(t), _p(rw), C.c_int64(n), _p(out))
    return out


def logprob_stats(logits, targets, rows=None, aux_idx=None, old_logp=None):
    """Forward-only statistics: dict(logp[n], entropy[n], mean_entropy, mean_kl)."""
    a, code, ld = _logits_view(logits)
    t = _arr(targets, np.int32)
    rw = _arr(rows, np.int32)
    ax = _arr(aux_idx, np.int32)
    ol = _arr(old_logp, np.float32)
    n = a.shape[0] if rw is None else rw.shape[0]
    logp, ent = np.empty(n, np.float64), np.empty(n, np.float64)
    means = np.zeros(2, np.float64)
    lib().oracle_logprob_stats(_p(a), C.c_int(code), C.c_int32(a.shape[1]), C.c_int64(ld), _p(t),
                               _p(rw), _p(ax), C.c_int64(n), _p(ol), _p(logp), _p(ent), _p(means))
    return dict(logp=logp, entropy=ent, mean_entropy=float(means[0]), mean_kl=float(means[1]))


def policy_loss(logits, targets, rows, aux_idx, old_logp, adv, eps_low, eps_high,
                denom=0.0, want_dlogits=True):
    """Returns dict(logp, token_loss, loss, clip_lo, clip_hi, dlogits[n,V] or None)."""
    a, code, ld = _logits_view(logits)
    t = _arr(targets, np.int32)
    rw = _arr(rows, np.int32)
    ax = _arr(aux_idx, np.int32)
    ol = _arr(old_logp, np.float32)
    ad = _arr(adv, np.float32)
    n = a.shape[0] if rw is None else rw.shape[0]
    V = a.shape[1]
    logp = np.empty(n, np.float64)
    tl = np.empty(n, np.float64)
    loss = np.zeros(1, np.float64)
    cc = np.zeros(2, np.int64)
    dl = np.empty((n, V), np.float64) if want_dlogits else None
    lib().oracle_policy_loss(_p(a), C.c_int(code), C.c_int32(V), C.c_int64(ld), _p(t), _p(rw),
                             _p(ax), C.c_int64(n), _p(ol), _p(ad), C.c_double(eps_low),
                             C.c_double(eps_high), C.c_double(denom), _p(logp), _p(tl),
                             _p(loss), _p(cc), _p(dl))
    return dict(logp=logp, token_loss=tl, loss=float(loss[0]), clip_lo=int(cc[0]),
                clip_hi=int(cc[1]), dlogits=dl)


def value_loss(values, old_values, returns, value_idx, xi_low, xi_high, denom=0.0,
               want_grad=True):
    v = _arr(values, np.float32)
    vo = _arr(old_values, np.float32)
    R = _arr(returns, np.float32)
    ix = _arr(value_idx, np.int32)
    N, n = v.shape[0], ix.shape[0]
    loss = np.zeros(1, np.float64)
    dv = np.empty(N, np.float64) if want_grad else None
    lib().oracle_value_loss(_p(v), _p(vo), _p(R), _p(ix), C.c_int64(n), C.c_int64(N),
                            C.c_double(xi_low), C.c_double(xi_high), C.c_double(denom),
                            _p(loss), _p(dv))
    return float(loss[0]), dv


def lmhead_logits_rows(hidden_bits, weight_bits, rows):
    h = _arr(hidden_bits, np.uint16)
    w = _arr(weight_bits, np.uint16)
    rw = _arr(rows, np.int32)
    K, V = w.shape
    assert h.shape[1] == K
    x = np.empty((rw.shape[0], V), np.float64)
    lib().oracle_lmhead_logits_rows(_p(h), _p(w), C.c_int32(K), C.c_int32(V), _p(rw),
                                    C.c_int64(rw.shape[0]), _p(x))
    return x


def lmhead_dhidden_rows(dx, weight_bits):
    g = _arr(dx, np.float64)
    w = _arr(weight_bits, np.uint16)
    K, V = w.shape
    dh = np.empty((g.shape[0], K), np.float64)
    lib().oracle_lmhead_dhidden_rows(_p(g), _p(w), C.c_int32(K), C.c_int32(V),
                                     C.c_int64(g.shape[0]), _p(dh))
    return dh


def lmhead_dweight_cols(hidden_bits, dx_cols):
    h = _arr(hidden_bits, np.uint16)
    g = _arr(dx_cols, np.float64)
    M, K = h.shape
    assert g.shape[0] == M
    dw = np.empty((K, g.shape[1]), np.float64)
    lib().oracle_lmhead_dweight_cols(_p(h), _p(g), C.c_int64(M), C.c_int32(K),
                                     C.c_int64(g.shape[1]), _p(dw))
    return dw


def advance_batch(seq_begin, prompt_len, prev_len, new_len, truncated, tokens, queue_begin,
                  queue_tokens, capacity=None):
    """Successive batching between two steps.  Returns dict(next_prompt_len, next_prev_len,
    next_seq_begin, next_tokens[:total], free_slots[:n_free], slot_source, n_free, n_refilled, total)."""
    sb = _arr(seq_begin, np.int32)
    pl, pv, nl = _arr(prompt_len, np.int32), _arr(prev_len, np.int32), _arr(new_len, np.int32)
    tr = _arr(truncated, np.uint8)
    tk = _arr(tokens, np.int32)
    qb, qt = _arr(queue_begin, np.int32), _arr(queue_tokens, np.int32)
    B, M = pl.shape[0], qb.shape[0] - 1
    if capacity is None:
        capacity = int(tk.shape[0] + qt.shape[0])
    npl, npv = np.zeros(B, np.int32), np.zeros(B, np.int32)
    nsb = np.zeros(B + 1, np.int32)
    ntk = np.full(max(capacity, 1), -7, np.int32)
    fs, src = np.full(max(B, 1), -9, np.int32), np.zeros(max(B, 1), np.int32)
    counts = np.zeros(3, np.int64)
    lib().oracle_advance_batch(_p(sb), _p(pl), _p(pv), _p(nl), _p(tr), _p(tk), _p(qb), _p(qt),
                               C.c_int32(B), C.c_int32(M), _p(npl), _p(npv), _p(nsb), _p(ntk),
                               C.c_int64(capacity), _p(fs), _p(src), _p(counts))
    n_free, n_ref, total = (int(x) for x in counts)
    return dict(next_prompt_len=npl, next_prev_len=npv, next_seq_begin=nsb,
                next_tokens=ntk[:min(total, capacity)], free_slots=fs[:n_free], slot_source=src[:B],
                n_free=n_free, n_refilled=n_ref, total=total)
