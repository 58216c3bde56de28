"""ctypes binding of include/tppo.h: same entry-point names, argument marshalling only.

Every function takes torch CUDA tensors (or None), checks dtype / contiguity, hands raw device
pointers and the current torch stream to the C ABI and raises on a non-zero status.  Nothing is
computed here, and there is no fallback: if libtppo.so cannot be loaded the import fails.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# the in-tree build, or another build of the same sources named by TPPO_LIBRARY
LIB_PATH = os.environ.get("TPPO_LIBRARY") or os.path.join(_HERE, "libtppo.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2506_15050_b200.build` "
        "(there is no CPU fallback)")
_lib = C.CDLL(LIB_PATH)

OP_EGAE, OP_SELECT_TOKENS, OP_POLICY_LOSS, OP_VALUE_LOSS, OP_LMHEAD = range(5)
BF16, F32 = 0, 1
DLOGITS_NONE, DLOGITS_FULL, DLOGITS_COMPACT = 0, 1, 2
POLICY_AUTO, POLICY_TWO_PASS, POLICY_CLUSTER_SMEM = 0, 1, 2
DEV_BAD_TARGET, DEV_WAIT_TIMEOUT, DEV_BAD_INDEX, DEV_BAD_SEGMENT, DEV_OVERFLOW, DEV_NONFINITE = 1, 2, 4, 8, 16, 32

_vp, _i32, _i64, _f32, _sz = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_size_t

_lib.tppo_version.restype = C.c_int
_lib.tppo_status_string.restype = C.c_char_p
_lib.tppo_status_string.argtypes = [C.c_int]
_lib.tppo_workspace_bytes.restype = _sz
_lib.tppo_workspace_bytes.argtypes = [C.c_int, _i64, _i32, _i64, _i32]
_lib.tppo_egae.restype = C.c_int
_lib.tppo_egae.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _i32, _i64, _f32, _f32, _vp, _vp, _vp,
                           _vp, _sz, _vp]
_lib.tppo_egae_static.restype = C.c_int
_lib.tppo_egae_static.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _i32, _i64, _f32, _f32, _vp, _vp, _vp, _vp]
_lib.tppo_select_tokens.restype = C.c_int
_lib.tppo_select_tokens.argtypes = [_vp, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _vp, _i32, _i64, _vp, _vp,
                                    _vp, _vp, _sz, _vp]
_lib.tppo_test_hooks.restype = None
_lib.tppo_test_hooks.argtypes = [_i32, _i32]
_lib.tppo_policy_loss_fwd_bwd.restype = C.c_int
_lib.tppo_policy_loss_fwd_bwd.argtypes = [_vp, _i32, _i64, _i32, _i64, _vp, _vp, _vp, _i64, _vp,
                                          _vp, _vp, _i64, _f32, _f32, _f32, _vp, _vp, _vp, _vp,
                                          _vp, _i32, _i32, _vp, _sz, _vp]
_lib.tppo_policy_logprob_stats.restype = C.c_int
_lib.tppo_policy_logprob_stats.argtypes = [_vp, _i32, _i64, _i32, _i64, _vp, _vp, _vp, _i64, _vp, _vp, _i64,
                                           _vp, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.tppo_value_loss.restype = C.c_int
_lib.tppo_value_loss.argtypes = [_vp, _vp, _vp, _i64, _vp, _vp, _i64, _f32, _f32, _f32, _vp, _vp,
                                 _vp, _vp, _sz, _vp]
_lib.tppo_lmhead_logprob_fwd_bwd.restype = C.c_int
_lib.tppo_lmhead_logprob_fwd_bwd.argtypes = [_vp, _vp, _i64, _i32, _i32, _vp, _vp, _vp, _vp, _i64,
                                             _f32, _f32, _f32, _vp, _vp, _vp, _vp, _vp, _vp, _i32,
                                             _vp, _sz, _vp]
_lib.tppo_lmhead_shard_stats.restype = C.c_int
_lib.tppo_lmhead_shard_stats.argtypes = [_vp, _vp, _i64, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp,
                                         _vp, _i32, _vp, _sz, _vp]
_lib.tppo_lmhead_shard_rescale.restype = C.c_int
_lib.tppo_lmhead_shard_rescale.argtypes = [_vp, _vp, _vp, _i64, _vp]
_lib.tppo_lmhead_shard_fwd_bwd.restype = C.c_int
_lib.tppo_lmhead_shard_fwd_bwd.argtypes = [_vp, _vp, _i64, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp,
                                           _i64, _f32, _f32, _f32, _vp, _vp, _vp, _vp, _vp, _vp, _vp,
                                           _vp, _vp, _i32, _vp, _sz, _vp]
_lib.tppo_advance_batch.restype = C.c_int
_lib.tppo_advance_batch.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _i64, _vp, _vp, _i64, _i32, _i32,
                                    _vp, _vp, _vp, _vp, _i64, _vp, _vp, _vp, _vp]


class TppoError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        super().__init__(f"tppo status {status}: {_lib.tppo_status_string(status).decode()}")


def _check(status: int):
    if status != 0:
        raise TppoError(status)


def _ptr(t, dtype=None):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "tensors must be contiguous CUDA tensors"
    if dtype is not None:
        assert t.dtype == dtype, f"expected {dtype}, got {t.dtype}"
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def tppo_version() -> int:
    return int(_lib.tppo_version())


def tppo_workspace_bytes(op: int, N: int, B: int, n_max: int, V: int) -> int:
    return int(_lib.tppo_workspace_bytes(op, N, B, n_max, V))


def workspace(op: int, N: int, B: int, n_max: int, V: int, device) -> torch.Tensor:
    """A caller-owned scratch tensor of the size the op asks for (torch's allocator aligns it)."""
    nbytes = max(256, tppo_workspace_bytes(op, N, B, n_max, V))
    return torch.empty(nbytes, dtype=torch.uint8, device=device)


def tppo_egae(rewards, values, seg_begin, seg_end, truncated, bootstrap, gamma, lam,
              advantages, returns, status, ws):
    N, B = rewards.numel(), seg_begin.numel()
    _check(_lib.tppo_egae(_ptr(rewards, torch.float32), _ptr(values, torch.float32),
                          _ptr(seg_begin, torch.int32), _ptr(seg_end, torch.int32),
                          _ptr(truncated, torch.uint8), _ptr(bootstrap, torch.float32),
                          B, N, gamma, lam, _ptr(advantages, torch.float32),
                          _ptr(returns, torch.float32), _ptr(status, torch.int32),
                          _ptr(ws), ws.numel(), _stream()))


EGAE_STATIC_MAX_TOKENS = 4194304


def tppo_egae_static(rewards, values, seg_begin, seg_end, truncated, bootstrap, gamma, lam,
                     advantages, returns, status):
    """tppo_egae for callers that cannot allocate device memory and have no workspace to lend
    (e.g. a plug-in inside a runtime that owns the device's whole memory pool): the scan's scratch
    is a fixed array inside the library.  At most EGAE_STATIC_MAX_TOKENS tokens; calls on one device
    share that array, so calls that may overlap on the GPU must be ordered by the caller."""
    N, B = rewards.numel(), seg_begin.numel()
    _check(_lib.tppo_egae_static(_ptr(rewards, torch.float32), _ptr(values, torch.float32),
                                 _ptr(seg_begin, torch.int32), _ptr(seg_end, torch.int32),
                                 _ptr(truncated, torch.uint8), _ptr(bootstrap, torch.float32),
                                 B, N, gamma, lam, _ptr(advantages, torch.float32),
                                 _ptr(returns, torch.float32), _ptr(status, torch.int32), _stream()))


def tppo_test_hooks(lookback_polls: int = -1, no_publish: bool = False) -> None:
    """Test aid: shorten the look-back waits of tppo_egae / tppo_select_tokens and (optionally) stop
    tiles from publishing, so that the bounded waits run out; (-1, False) restores normal operation."""
    _lib.tppo_test_hooks(int(lookback_polls), 1 if no_publish else 0)


def tppo_select_tokens(seq_begin, prompt_len, prev_len, new_len, truncated, tail_drop,
                       extra_policy_mask, extra_value_mask, N, policy_idx, value_idx, counts, ws,
                       tail_drop_seq=None):
    B = prompt_len.numel()
    assert tail_drop_seq is None or tail_drop_seq.numel() == B
    _check(_lib.tppo_select_tokens(_ptr(seq_begin, torch.int32), _ptr(prompt_len, torch.int32),
                                   _ptr(prev_len, torch.int32), _ptr(new_len, torch.int32),
                                   _ptr(truncated, torch.uint8), tail_drop,
                                   _ptr(tail_drop_seq, torch.int32),
                                   _ptr(extra_policy_mask, torch.uint8),
                                   _ptr(extra_value_mask, torch.uint8), B, N,
                                   _ptr(policy_idx, torch.int32), _ptr(value_idx, torch.int32),
                                   _ptr(counts, torch.int32), _ptr(ws), ws.numel(), _stream()))


def tppo_policy_loss_fwd_bwd(logits, targets, rows, n_sel, n_max, aux_idx, old_logp, adv,
                             eps_low, eps_high, denom, logp, token_loss, loss, stats,
                             dlogits, dlogits_mode, ws, kernel_hint=POLICY_AUTO, V=None):
    assert logits.is_cuda and logits.dim() == 2 and logits.stride(1) == 1
    dt = {torch.bfloat16: BF16, torch.float32: F32}[logits.dtype]
    R, ld = logits.shape[0], logits.stride(0)
    V = logits.shape[1] if V is None else V
    if dlogits is not None:
        assert dlogits.dtype == logits.dtype and dlogits.is_cuda and dlogits.stride(-1) == 1
        if dlogits_mode == DLOGITS_FULL:
            assert dlogits.stride(0) == ld, "FULL mode: dlogits must have the logits' row stride"
        else:
            assert dlogits.is_contiguous(), "COMPACT mode: dlogits must be dense [n_max, V]"
    _check(_lib.tppo_policy_loss_fwd_bwd(
        logits.data_ptr(), dt, R, V, ld, _ptr(targets, torch.int32), _ptr(rows, torch.int32),
        _ptr(n_sel, torch.int32), n_max, _ptr(aux_idx, torch.int32),
        _ptr(old_logp, torch.float32), _ptr(adv, torch.float32), old_logp.numel(),
        eps_low, eps_high, denom, _ptr(logp, torch.float32), _ptr(token_loss, torch.float32),
        _ptr(loss, torch.float32), _ptr(stats, torch.int32),
        None if dlogits is None else dlogits.data_ptr(), dlogits_mode, kernel_hint,
        _ptr(ws), ws.numel(), _stream()))


def tppo_policy_logprob_stats(logits, targets, rows, n_sel, n_max, aux_idx, old_logp, logp, entropy,
                              means, stats, ws, V=None):
    assert logits.is_cuda and logits.dim() == 2 and logits.stride(1) == 1
    dt = {torch.bfloat16: BF16, torch.float32: F32}[logits.dtype]
    R, ld = logits.shape[0], logits.stride(0)
    V = logits.shape[1] if V is None else V
    _check(_lib.tppo_policy_logprob_stats(
        logits.data_ptr(), dt, R, V, ld, _ptr(targets, torch.int32), _ptr(rows, torch.int32),
        _ptr(n_sel, torch.int32), n_max, _ptr(aux_idx, torch.int32), _ptr(old_logp, torch.float32),
        0 if old_logp is None else old_logp.numel(), _ptr(logp, torch.float32),
        _ptr(entropy, torch.float32), _ptr(means, torch.float32), _ptr(stats, torch.int32),
        _ptr(ws), ws.numel(), _stream()))


def tppo_value_loss(values, old_values, returns, value_idx, n_sel, n_max, xi_low, xi_high, denom,
                    loss, dvalues, stats, ws):
    _check(_lib.tppo_value_loss(_ptr(values, torch.float32), _ptr(old_values, torch.float32),
                                _ptr(returns, torch.float32), values.numel(),
                                _ptr(value_idx, torch.int32), _ptr(n_sel, torch.int32), n_max,
                                xi_low, xi_high, denom, _ptr(loss, torch.float32),
                                _ptr(dvalues, torch.float32), _ptr(stats, torch.int32),
                                _ptr(ws), ws.numel(), _stream()))


def tppo_lmhead_logprob_fwd_bwd(hidden, weight, targets, aux_idx, old_logp, adv, eps_low,
                                eps_high, denom, logp, token_loss, loss, stats, dhidden, dweight,
                                ws, chunk_tiles=0):
    M, K = hidden.shape
    assert weight.shape[0] == K
    V = weight.shape[1]
    _check(_lib.tppo_lmhead_logprob_fwd_bwd(
        _ptr(hidden, torch.bfloat16), _ptr(weight, torch.bfloat16), M, K, V,
        _ptr(targets, torch.int32), _ptr(aux_idx, torch.int32), _ptr(old_logp, torch.float32),
        _ptr(adv, torch.float32), old_logp.numel(), eps_low, eps_high, denom,
        _ptr(logp, torch.float32), _ptr(token_loss, torch.float32), _ptr(loss, torch.float32),
        _ptr(stats, torch.int32), _ptr(dhidden, torch.bfloat16), _ptr(dweight, torch.bfloat16),
        chunk_tiles, _ptr(ws), ws.numel(), _stream()))


def tppo_lmhead_shard_stats(hidden, weight_shard, v_offset, V_total, targets, row_max, row_sumexp,
                            row_target_logit, stats, ws, chunk_tiles=0):
    M, K = hidden.shape
    assert weight_shard.shape[0] == K
    _check(_lib.tppo_lmhead_shard_stats(
        _ptr(hidden, torch.bfloat16), _ptr(weight_shard, torch.bfloat16), M, K,
        weight_shard.shape[1], v_offset, V_total, _ptr(targets, torch.int32),
        _ptr(row_max, torch.float32), _ptr(row_sumexp, torch.float32),
        _ptr(row_target_logit, torch.float32), _ptr(stats, torch.int32), chunk_tiles,
        _ptr(ws), ws.numel(), _stream()))


def tppo_lmhead_shard_rescale(row_max, row_max_all, row_sumexp):
    _check(_lib.tppo_lmhead_shard_rescale(
        _ptr(row_max, torch.float32), _ptr(row_max_all, torch.float32),
        _ptr(row_sumexp, torch.float32), row_max.numel(), _stream()))


def tppo_lmhead_shard_fwd_bwd(hidden, weight_shard, v_offset, V_total, targets, aux_idx, old_logp,
                              adv, eps_low, eps_high, denom, row_max, row_sumexp, row_target_logit,
                              logp, token_loss, loss, stats, dhidden_partial, dweight_shard, ws,
                              chunk_tiles=0):
    M, K = hidden.shape
    assert weight_shard.shape[0] == K
    _check(_lib.tppo_lmhead_shard_fwd_bwd(
        _ptr(hidden, torch.bfloat16), _ptr(weight_shard, torch.bfloat16), M, K,
        weight_shard.shape[1], v_offset, V_total, _ptr(targets, torch.int32),
        _ptr(aux_idx, torch.int32), _ptr(old_logp, torch.float32), _ptr(adv, torch.float32),
        old_logp.numel(), eps_low, eps_high, denom, _ptr(row_max, torch.float32),
        _ptr(row_sumexp, torch.float32), _ptr(row_target_logit, torch.float32),
        _ptr(logp, torch.float32), _ptr(token_loss, torch.float32), _ptr(loss, torch.float32),
        _ptr(stats, torch.int32), _ptr(dhidden_partial, torch.bfloat16),
        _ptr(dweight_shard, torch.bfloat16), chunk_tiles, _ptr(ws), ws.numel(), _stream()))


def tppo_advance_batch(seq_begin, prompt_len, prev_len, new_len, truncated, tokens, queue_begin,
                       queue_tokens, next_prompt_len, next_prev_len, next_seq_begin, next_tokens,
                       free_slots, slot_source, counts):
    B, M = prompt_len.numel(), queue_begin.numel() - 1
    _check(_lib.tppo_advance_batch(
        _ptr(seq_begin, torch.int32), _ptr(prompt_len, torch.int32), _ptr(prev_len, torch.int32),
        _ptr(new_len, torch.int32), _ptr(truncated, torch.uint8), _ptr(tokens, torch.int32),
        tokens.numel(), _ptr(queue_begin, torch.int32), _ptr(queue_tokens, torch.int32),
        queue_tokens.numel(), B, M, _ptr(next_prompt_len, torch.int32),
        _ptr(next_prev_len, torch.int32), _ptr(next_seq_begin, torch.int32),
        _ptr(next_tokens, torch.int32), next_tokens.numel(), _ptr(free_slots, torch.int32),
        _ptr(slot_source, torch.int32), _ptr(counts, torch.int32), _stream()))
