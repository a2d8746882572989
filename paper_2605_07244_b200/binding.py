"""ctypes binding of libmrl.so: same names as the C ABI, argument marshalling only.

Tensors are torch tensors used as device (or pinned host) memory; every step of the path runs
inside the library's CUDA kernels.  There is no fallback: a missing library raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from .build import LIB_PATH

OK = 0
F32, BF16 = 0, 1
ADV_MEAN_ONLY, ADV_GROUP_ZNORM, ADV_BATCH_ZNORM = 0, 1, 2
PICK_NONE, PICK_FIRST, PICK_SHORTEST, PICK_ALL, PICK_SEEDED = 0, 1, 2, 3, 4
AGG_TOKEN_MEAN, AGG_SEQ_MEAN_TOKEN_MEAN = 0, 1
RATIO_TOKEN, RATIO_SEQUENCE = 0, 1
KL_K1, KL_K2, KL_K3 = 0, 1, 2
FLAG_ACCUMULATE_LOSS, FLAG_SKIP_ZERO_ROWS, FLAG_ACCUMULATE_DW, FLAG_PAIR_TILES = 1, 2, 4, 8
WS_TOKEN_LOGPROBS, WS_POLICY_LOSS, WS_FUSED_LMHEAD, WS_THL_WORD_ALIGN = 0, 1, 2, 3
DEV_BAD_TOKEN_ID, DEV_TIMEOUT, DEV_BAD_WORD_MAP = 1, 2, 4

EXPORTS = ("mrl_group_advantages", "mrl_token_logprobs", "mrl_policy_loss_fwd_bwd",
           "mrl_fused_lmhead_loss_fwd_bwd", "mrl_workspace_bytes", "mrl_status_string", "mrl_version",
           "mrl_profile_dominant_kernel", "mrl_policy_loss_fwd_bwd_static", "mrl_thl_word_align_logprobs",
           "mrl_policy_loss_fwd_bwd_host", "mrl_host_pipeline_workspace_bytes", "mrl_profile_last_kernel")
STATIC_MAX_ROWS, STATIC_MAX_SEQS = 65536, 65536
ERR_STATIC_SCRATCH_TOO_SMALL = 8


class AdvParams(C.Structure):
    _fields_ = [("mode", C.c_int32), ("ddof", C.c_int32), ("eps", C.c_float),
                ("sgt_success_thr", C.c_float), ("sgt_negative_thr", C.c_float),
                ("sgt_pick", C.c_int32), ("seed", C.c_uint64)]


class LossParams(C.Structure):
    _fields_ = [("eps_lo", C.c_float), ("eps_hi", C.c_float), ("agg_mode", C.c_int32),
                ("flags", C.c_uint32), ("pg_denominator", C.c_double), ("seq_denominator", C.c_double),
                ("nll_coeff", C.c_float), ("ratio_level", C.c_int32), ("entropy", C.c_void_p),
                ("logp_ref", C.c_void_p), ("kl_coeff", C.c_float), ("kl_estimator", C.c_int32),
                ("kl_loss", C.c_void_p)]


class MrlError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


_lib = None


def lib() -> C.CDLL:
    """The loaded library; raises if it has not been built (there is no other code path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2605_07244_b200.build` "
                               "(or __graft_entry__.build()) first; there is no CPU fallback")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
        L.mrl_group_advantages.argtypes = [vp, vp, i32, i32, i32, i32, C.POINTER(AdvParams), vp, vp, vp, vp, vp, vp, vp]
        L.mrl_group_advantages.restype = C.c_int
        L.mrl_token_logprobs.argtypes = [vp, i32, i64, i32, i64, vp, vp, vp, vp, vp, vp, sz, vp]
        L.mrl_token_logprobs.restype = C.c_int
        L.mrl_policy_loss_fwd_bwd.argtypes = [vp, i32, i64, i32, i64, vp, vp, vp, i32, vp, vp, vp, vp,
                                              C.POINTER(LossParams), vp, i64, vp, vp, vp, vp, vp, sz, vp]
        L.mrl_policy_loss_fwd_bwd.restype = C.c_int
        L.mrl_policy_loss_fwd_bwd_static.argtypes = [vp, i32, i64, i32, i64, vp, vp, vp, i32, vp, vp, vp, vp,
                                                     C.POINTER(LossParams), vp, i64, vp, vp, vp, vp, vp]
        L.mrl_policy_loss_fwd_bwd_static.restype = C.c_int
        L.mrl_policy_loss_fwd_bwd_host.argtypes = [vp, i32, i64, i32, i64, vp, vp, vp, i32, vp, vp, vp, vp,
                                                   C.POINTER(LossParams), vp, i64, vp, vp, vp, vp, i64, vp, sz, vp]
        L.mrl_policy_loss_fwd_bwd_host.restype = C.c_int
        L.mrl_host_pipeline_workspace_bytes.argtypes = [i64, i64, i32, i32, i64]
        L.mrl_host_pipeline_workspace_bytes.restype = sz
        L.mrl_fused_lmhead_loss_fwd_bwd.argtypes = [vp, vp, i64, i32, i32, vp, vp, vp, i32, vp, vp, vp, vp,
                                                    C.POINTER(LossParams), vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.mrl_fused_lmhead_loss_fwd_bwd.restype = C.c_int
        L.mrl_thl_word_align_logprobs.argtypes = [vp, vp, vp, vp, vp, vp, i32, i64, i64, i64, C.c_float, vp, vp, vp, vp,
                                                  vp, sz, vp]
        L.mrl_thl_word_align_logprobs.restype = C.c_int
        L.mrl_workspace_bytes.argtypes = [i32, i64, i32, i32, i32, i32]
        L.mrl_workspace_bytes.restype = sz
        L.mrl_status_string.argtypes = [C.c_int]
        L.mrl_status_string.restype = C.c_char_p
        L.mrl_profile_dominant_kernel.argtypes = [C.POINTER(vp), C.POINTER(vp), i32]
        L.mrl_profile_dominant_kernel.restype = C.c_int
        L.mrl_profile_last_kernel.argtypes = []
        L.mrl_profile_last_kernel.restype = C.c_char_p
        L.mrl_version.argtypes = []
        L.mrl_version.restype = C.c_int
        _lib = L
    return _lib


def _p(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise MrlError(3, "dtype")


def _check(code: int, where: str):
    if code != OK:
        raise MrlError(code, where)


def status_string(code: int) -> str:
    return lib().mrl_status_string(code).decode()


def version() -> int:
    return lib().mrl_version()


def workspace_bytes(which: int, N: int, V: int, H: int = 0, dtype: int = BF16, S: int = 0) -> int:
    return int(lib().mrl_workspace_bytes(which, N, V, H, dtype, S))


def mrl_group_advantages(rewards, seq_len, learner: int, ap: AdvParams, adv_own=None, adv_pool=None,
                         rescue=None, pick=None, nll_seq_weight=None, n_gated=None, stream=None):
    P, M, G = rewards.shape
    _check(lib().mrl_group_advantages(_p(rewards), _p(seq_len), P, M, G, learner, C.byref(ap), _p(adv_own),
                                      _p(adv_pool), _p(rescue), _p(pick), _p(nll_seq_weight), _p(n_gated),
                                      _stream(stream)), "mrl_group_advantages")


def mrl_token_logprobs(logits, ids, mask, logp, lse=None, status=None, workspace=None, V=None, stream=None):
    N = logits.shape[0]
    V = logits.shape[1] if V is None else V
    ld = logits.stride(0) if N > 1 else max(logits.shape[1], V)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().mrl_token_logprobs(_p(logits), _dtype_code(logits), N, V, ld, _p(ids), _p(mask), _p(logp),
                                    _p(lse), _p(status), _p(workspace), ws_bytes, _stream(stream)),
           "mrl_token_logprobs")


def mrl_policy_loss_fwd_bwd(logits, ids, mask, cu_seqlens, adv_seq, logp_old, tok_weight, nll_weight,
                            lp: LossParams, dlogits, logp, loss, stats=None, status=None, workspace=None,
                            V=None, stream=None):
    N = logits.shape[0]
    V = logits.shape[1] if V is None else V
    S = cu_seqlens.numel() - 1
    ld = logits.stride(0) if N > 1 else max(logits.shape[1], V)
    ld_out = ld if dlogits is None else (dlogits.stride(0) if N > 1 else max(dlogits.shape[1], V))
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().mrl_policy_loss_fwd_bwd(_p(logits), _dtype_code(logits), N, V, ld, _p(ids), _p(mask),
                                         _p(cu_seqlens), S, _p(adv_seq), _p(logp_old), _p(tok_weight),
                                         _p(nll_weight), C.byref(lp), _p(dlogits), ld_out, _p(logp), _p(loss),
                                         _p(stats), _p(status), _p(workspace), ws_bytes, _stream(stream)),
           "mrl_policy_loss_fwd_bwd")


def mrl_policy_loss_fwd_bwd_static(logits, ids, mask, cu_seqlens, adv_seq, logp_old, tok_weight, nll_weight,
                                   lp: LossParams, dlogits, logp, loss, stats=None, status=None, V=None,
                                   stream=None):
    """mrl_policy_loss_fwd_bwd without a workspace argument: for callers that cannot allocate device
    memory, the library's own fixed scratch array is used (N <= STATIC_MAX_ROWS, S <= STATIC_MAX_SEQS)."""
    N = logits.shape[0]
    V = logits.shape[1] if V is None else V
    S = cu_seqlens.numel() - 1
    ld = logits.stride(0) if N > 1 else max(logits.shape[1], V)
    ld_out = ld if dlogits is None else (dlogits.stride(0) if N > 1 else max(dlogits.shape[1], V))
    _check(lib().mrl_policy_loss_fwd_bwd_static(_p(logits), _dtype_code(logits), N, V, ld, _p(ids), _p(mask),
                                                _p(cu_seqlens), S, _p(adv_seq), _p(logp_old), _p(tok_weight),
                                                _p(nll_weight), C.byref(lp), _p(dlogits), ld_out, _p(logp),
                                                _p(loss), _p(stats), _p(status), _stream(stream)),
           "mrl_policy_loss_fwd_bwd_static")


def host_pipeline_workspace_bytes(N: int, ld: int, dtype: int, S: int, slab_rows: int) -> int:
    return int(lib().mrl_host_pipeline_workspace_bytes(N, ld, dtype, S, slab_rows))


def mrl_policy_loss_fwd_bwd_host(h_logits, h_ids, h_mask, h_cu_seqlens, h_adv_seq, h_logp_old, h_tok_weight,
                                 h_nll_weight, lp: LossParams, h_dlogits, h_logp, h_loss, h_stats, h_status,
                                 slab_rows: int, workspace, V=None, stream=None):
    """The logits-in pass on HOST tensors (pinned for overlap), pipelined in micro-batches of whole sequences over
    three staging buffers in `workspace` (device).  Asynchronous: synchronise `stream` before reading the outputs."""
    for t in (h_logits, h_ids, h_mask, h_cu_seqlens, h_adv_seq, h_logp_old, h_tok_weight, h_nll_weight, h_dlogits,
              h_logp, h_loss, h_stats, h_status):
        if t is not None and t.is_cuda:
            raise MrlError(1, "mrl_policy_loss_fwd_bwd_host takes host tensors")
    N = h_logits.shape[0]
    V = h_logits.shape[1] if V is None else V
    S = h_cu_seqlens.numel() - 1
    ld = h_logits.stride(0) if N > 1 else max(h_logits.shape[1], V)
    ld_out = ld if h_dlogits is None else (h_dlogits.stride(0) if N > 1 else max(h_dlogits.shape[1], V))
    ws_bytes = workspace.numel() * workspace.element_size()
    _check(lib().mrl_policy_loss_fwd_bwd_host(_p(h_logits), _dtype_code(h_logits), N, V, ld, _p(h_ids), _p(h_mask),
                                              _p(h_cu_seqlens), S, _p(h_adv_seq), _p(h_logp_old), _p(h_tok_weight),
                                              _p(h_nll_weight), C.byref(lp), _p(h_dlogits), ld_out, _p(h_logp),
                                              _p(h_loss), _p(h_stats), _p(h_status), int(slab_rows), _p(workspace),
                                              ws_bytes, _stream(stream)), "mrl_policy_loss_fwd_bwd_host")


def mrl_fused_lmhead_loss_fwd_bwd(hidden, W, ids, mask, cu_seqlens, adv_seq, logp_old, tok_weight, nll_weight,
                                  lp: LossParams, dHidden, dW, logp, loss, stats=None, status=None,
                                  workspace=None, stream=None):
    N, H = hidden.shape
    V = W.shape[0]
    S = cu_seqlens.numel() - 1
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().mrl_fused_lmhead_loss_fwd_bwd(_p(hidden), _p(W), N, H, V, _p(ids), _p(mask), _p(cu_seqlens), S,
                                               _p(adv_seq), _p(logp_old), _p(tok_weight), _p(nll_weight),
                                               C.byref(lp), _p(dHidden), _p(dW), _p(logp), _p(loss), _p(stats),
                                               _p(status), _p(workspace), ws_bytes, _stream(stream)),
           "mrl_fused_lmhead_loss_fwd_bwd")


def mrl_thl_word_align_logprobs(src_logp, src_word, src_cu, tgt_word, tgt_cu, word_cu, total_words, ignore_value,
                                out, src_total=None, tgt_total=None, status=None, workspace=None, stream=None):
    Bn = src_cu.numel() - 1
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().mrl_thl_word_align_logprobs(_p(src_logp), _p(src_word), _p(src_cu), _p(tgt_word), _p(tgt_cu),
                                             _p(word_cu), Bn, src_word.numel(), out.numel(), int(total_words),
                                             float(ignore_value), _p(out),
                                             _p(src_total), _p(tgt_total), _p(status), _p(workspace), ws_bytes,
                                             _stream(stream)), "mrl_thl_word_align_logprobs")


class DominantKernelTimer:
    """Registers n CUDA-event pairs around the dominant kernel of the following calls; `elapsed_ms()`
    returns the duration of every recorded launch (after a synchronise)."""

    def __init__(self, n: int):
        self.n = n
        self.start = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
        self.stop = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
        for e in self.start + self.stop:      # torch creates the CUDA event lazily: force it
            e.record()
        torch.cuda.synchronize()
        self._a = (C.c_void_p * n)(*[e.cuda_event for e in self.start])
        self._b = (C.c_void_p * n)(*[e.cuda_event for e in self.stop])

    def __enter__(self):
        _check(lib().mrl_profile_dominant_kernel(self._a, self._b, self.n), "mrl_profile_dominant_kernel")
        return self

    def __exit__(self, *exc):
        self.last_kernel = lib().mrl_profile_last_kernel().decode()
        lib().mrl_profile_dominant_kernel(None, None, 0)

    def elapsed_ms(self, count: int):
        return [self.start[i].elapsed_time(self.stop[i]) for i in range(min(count, self.n))]
