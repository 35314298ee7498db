"""ctypes binding of liboapl.so: same names as the C entry points, argument
marshalling only.  Tensors are torch CUDA tensors used as device memory; every
step of the path runs in the library's kernels.  There is no fallback: a missing
library raises at first use.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liboapl.so")

OAPL_OK = 0
STATUS = {0: "OK", -1: "INVALID_ARG", -2: "MISALIGNED", -3: "WORKSPACE_TOO_SMALL",
          -4: "UNSUPPORTED_SHAPE", -5: "BAD_TARGET", -6: "BAD_SEQ_ORDER", -7: "NONFINITE_INPUT",
          -8: "DEVICE_TIMEOUT", -9: "CUDA", -10: "BAD_STATE", -11: "SEQUENCE_TOO_LONG", -12: "OUT_OF_RANGE",
          -13: "BOUND_EXCEEDED"}
OAPL_FLAG_FUSED = 1

EXPORTS = ["oapl_workspace_bytes", "oapl_token_logprobs", "oapl_value_estimate", "oapl_loss_fwd",
           "oapl_loss_bwd", "oapl_get_last_status", "oapl_get_live_rows", "oapl_launch_count",
           "oapl_status_string", "oapl_debug_gemm", "oapl_profile_enable", "oapl_profile_read",
           "oapl_token_logprobs_static", "oapl_loss_fwd_bwd", "oapl_profile_read_clocks", "oapl_entropy", "oapl_group_advantage",
           "oapl_grpo_loss_fwd_bwd", "oapl_adamw_workspace_bytes", "oapl_adamw_step", "oapl_loss_fwd_bwd_ex",
           "oapl_get_range_count", "oapl_profile_applies", "oapl_range_slots", "oapl_batch_stats"]


class OaplProblem(ctypes.Structure):
    _fields_ = [("N", ctypes.c_int64), ("d", ctypes.c_int32), ("V", ctypes.c_int32),
                ("S", ctypes.c_int32), ("P", ctypes.c_int32),
                ("H", ctypes.c_void_p), ("W", ctypes.c_void_p), ("targets", ctypes.c_void_p),
                ("mask", ctypes.c_void_p), ("seq_id", ctypes.c_void_p), ("group_id", ctypes.c_void_p),
                ("reward", ctypes.c_void_p), ("logp_inf", ctypes.c_void_p),
                ("beta_v", ctypes.c_float), ("beta_loss", ctypes.c_float), ("loss_scale", ctypes.c_float)]


class OaplCallOptions(ctypes.Structure):
    _fields_ = [("live_rows_bound", ctypes.c_int64), ("max_seq_rows_bound", ctypes.c_int32),
                ("dW_ready_event", ctypes.c_void_p)]


class OaplError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS.get(status, status)} ({lib().oapl_status_string(status).decode()})")


_lib = None


def lib() -> ctypes.CDLL:
    """Load liboapl.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2602_19362_b200.build` "
                               "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, f32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_float, ctypes.c_size_t
        pp = ctypes.POINTER(OaplProblem)
        L.oapl_workspace_bytes.restype = sz
        L.oapl_workspace_bytes.argtypes = [pp, i32]
        L.oapl_token_logprobs.restype = i32
        L.oapl_token_logprobs.argtypes = [pp, vp, vp, vp, sz, i32, vp]
        L.oapl_value_estimate.restype = i32
        L.oapl_value_estimate.argtypes = [vp, vp, ctypes.c_int32, ctypes.c_int32, f32, vp, vp]
        L.oapl_loss_fwd.restype = i32
        L.oapl_loss_fwd.argtypes = [pp, vp, vp, vp, vp, vp, vp, sz, i32, vp]
        L.oapl_loss_bwd.restype = i32
        L.oapl_loss_bwd.argtypes = [pp, vp, vp, i32, vp, sz, i32, vp]
        L.oapl_get_last_status.restype = i32
        L.oapl_get_last_status.argtypes = [vp, vp]
        L.oapl_get_live_rows.restype = i64
        L.oapl_get_live_rows.argtypes = [vp, vp]
        L.oapl_launch_count.restype = ctypes.c_uint64
        L.oapl_launch_count.argtypes = []
        L.oapl_status_string.restype = ctypes.c_char_p
        L.oapl_status_string.argtypes = [i32]
        L.oapl_debug_gemm.restype = i32
        L.oapl_debug_gemm.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, ctypes.c_longlong, i32, vp, vp]
        L.oapl_loss_fwd_bwd_ex.restype = i32
        L.oapl_loss_fwd_bwd_ex.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, i32, vp, sz, i32,
                                           ctypes.POINTER(OaplCallOptions), vp]
        L.oapl_get_range_count.restype = i32
        L.oapl_get_range_count.argtypes = [vp, vp]
        L.oapl_batch_stats.restype = i32
        L.oapl_batch_stats.argtypes = [pp, vp, vp, vp, sz, i32, vp]
        L.oapl_range_slots.restype = i32
        L.oapl_range_slots.argtypes = [i64, i64, ctypes.c_int32, ctypes.c_int32]
        L.oapl_profile_applies.restype = i32
        L.oapl_profile_applies.argtypes = [i32, i32]
        L.oapl_loss_fwd_bwd.restype = i32
        L.oapl_loss_fwd_bwd.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, i32, vp, sz, i32, vp]
        L.oapl_token_logprobs_static.restype = i32
        L.oapl_token_logprobs_static.argtypes = [pp, vp, vp, vp, vp]
        L.oapl_group_advantage.restype = i32
        L.oapl_group_advantage.argtypes = [vp, vp, ctypes.c_int32, ctypes.c_int32, f32, vp, vp]
        L.oapl_grpo_loss_fwd_bwd.restype = i32
        L.oapl_grpo_loss_fwd_bwd.argtypes = [pp, vp, vp, f32, vp, vp, vp, vp, vp, vp, i32, vp, sz, i32, vp]
        L.oapl_adamw_workspace_bytes.restype = sz
        L.oapl_adamw_workspace_bytes.argtypes = []
        L.oapl_adamw_step.restype = i32
        L.oapl_adamw_step.argtypes = [vp, vp, vp, vp, vp, i64, i64, f32, f32, f32, f32, f32, f32, vp, vp, vp, sz, vp]
        L.oapl_entropy.restype = i32
        L.oapl_entropy.argtypes = [pp, vp, vp, vp, vp, sz, i32, vp]
        L.oapl_profile_enable.restype = i32
        L.oapl_profile_enable.argtypes = [i32]
        L.oapl_profile_read.restype = i32
        L.oapl_profile_read.argtypes = [vp, vp, i32, vp]
        L.oapl_profile_read_clocks.restype = i32
        L.oapl_profile_read_clocks.argtypes = [vp, i32]
        _lib = L
    return _lib


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check_dev(t, dtype, name):
    if t is None:
        return
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of {dtype}")


def make_problem(batch: dict, beta_v=None, beta_loss=None, loss_scale=None) -> OaplProblem:
    """Fill the C struct from a batch dict (see synth.make_batch).  The dict's
    tensors must stay alive while the struct is in use."""
    _check_dev(batch["H"], torch.bfloat16, "H")
    _check_dev(batch["W"], torch.bfloat16, "W")
    _check_dev(batch["targets"], torch.int32, "targets")
    _check_dev(batch["mask"], torch.uint8, "mask")
    _check_dev(batch["seq_id"], torch.int32, "seq_id")
    _check_dev(batch.get("group_id"), torch.int32, "group_id")
    _check_dev(batch.get("reward"), torch.float32, "reward")
    _check_dev(batch.get("logp_inf"), torch.float32, "logp_inf")
    p = OaplProblem()
    p.N, p.d, p.V, p.S, p.P = batch["N"], batch["d"], batch["V"], batch["S"], batch["P"]
    p.H, p.W = batch["H"].data_ptr(), batch["W"].data_ptr()
    p.targets, p.mask, p.seq_id = batch["targets"].data_ptr(), batch["mask"].data_ptr(), batch["seq_id"].data_ptr()
    for k in ("group_id", "reward", "logp_inf"):
        t = batch.get(k)
        setattr(p, k, None if t is None else t.data_ptr())
    p.beta_v = batch.get("beta_v", 1.0) if beta_v is None else beta_v
    p.beta_loss = batch.get("beta_loss", 1.0) if beta_loss is None else beta_loss
    p.loss_scale = batch.get("loss_scale", 1.0) if loss_scale is None else loss_scale
    return p


def oapl_workspace_bytes(problem: OaplProblem, flags: int = 0) -> int:
    return int(lib().oapl_workspace_bytes(ctypes.byref(problem), flags))


def alloc_workspace(problem: OaplProblem, flags: int = 0, device="cuda") -> torch.Tensor:
    n = oapl_workspace_bytes(problem, flags)
    if n == 0:
        raise OaplError(-1, "oapl_workspace_bytes")
    ws = torch.empty(n + 1024, dtype=torch.uint8, device=device)
    off = (-ws.data_ptr()) % 1024
    return ws[off:off + n]


def oapl_token_logprobs(problem, token_logp, seq_logp, ws, flags=0):
    rc = lib().oapl_token_logprobs(ctypes.byref(problem), _ptr(token_logp), _ptr(seq_logp), _ptr(ws),
                                   ws.numel(), flags, _stream())
    if rc != OAPL_OK:
        raise OaplError(rc, "oapl_token_logprobs")


def oapl_value_estimate(reward, group_id, P, beta_v, vhat):
    rc = lib().oapl_value_estimate(_ptr(reward), _ptr(group_id), reward.numel(), P, beta_v, _ptr(vhat), _stream())
    if rc != OAPL_OK:
        raise OaplError(rc, "oapl_value_estimate")


def oapl_loss_fwd(problem, loss, seq_logp, vhat, delta, token_logp, ws, flags=0):
    rc = lib().oapl_loss_fwd(ctypes.byref(problem), _ptr(loss), _ptr(seq_logp), _ptr(vhat), _ptr(delta),
                             _ptr(token_logp), _ptr(ws), ws.numel(), flags, _stream())
    if rc != OAPL_OK:
        raise OaplError(rc, "oapl_loss_fwd")


def oapl_loss_bwd(problem, dH, dW, accumulate_dW, ws, flags=0):
    rc = lib().oapl_loss_bwd(ctypes.byref(problem), _ptr(dH), _ptr(dW), int(accumulate_dW), _ptr(ws),
                             ws.numel(), flags, _stream())
    if rc != OAPL_OK:
        raise OaplError(rc, "oapl_loss_bwd")


def oapl_group_advantage(reward, group_id, P, eps, advantage):
    rc = lib().oapl_group_advantage(_ptr(reward), _ptr(group_id), reward.numel(), P, eps, _ptr(advantage),
                                    _stream())
    if rc != OAPL_OK:
        raise OaplError(rc, "oapl_group_advantage")


def oapl_grpo_loss_fwd_bwd(problem, logp_old, advantage, clip_eps, loss, seq_logp, token_logp, clip_frac, dH, dW,
                           accumulate_dW, ws, flags=0):
    rc = lib().oapl_grpo_loss_fwd_bwd(ctypes.byref(problem), _ptr(logp_old), _ptr(advantage), clip_eps,
                                      _ptr(loss), _ptr(seq_logp), _ptr(token_logp), _ptr(clip_frac), _ptr(dH),
                                      _ptr(dW), int(accumulate_dW), _ptr(ws), ws.numel(), flags, _stream())
    if rc != OAPL_OK:
        raise OaplError(rc, "oapl_grpo_loss_fwd_bwd")


def oapl_adamw_step(W, master, dW, m, v, step, lr, beta1, beta2, eps, weight_decay, clip_norm,
                    other_sq_norm=None, grad_norm=None, ws=None):
    if ws is None:
        ws = torch.empty(int(lib().oapl_adamw_workspace_bytes()), dtype=torch.uint8, device=W.device)
    rc = lib().oapl_adamw_step(_ptr(W), _ptr(master), _ptr(dW), _ptr(m), _ptr(v), W.numel(), int(step), lr, beta1,
                               beta2, eps, weight_decay, clip_norm, _ptr(other_sq_norm), _ptr(grad_norm), _ptr(ws),
                               ws.numel(), _stream())
    if rc != OAPL_OK:
        raise OaplError(rc, "oapl_adamw_step")
    return ws


def oapl_entropy(problem, token_entropy, seq_entropy, mean_entropy, ws, flags=0):
    rc = lib().oapl_entropy(ctypes.byref(problem), _ptr(token_entropy), _ptr(seq_entropy), _ptr(mean_entropy),
                            _ptr(ws), ws.numel(), flags, _stream())
    if rc != OAPL_OK:
        raise OaplError(rc, "oapl_entropy")


STATS = ("live_tokens", "mean_abs_log_ratio", "max_abs_log_ratio", "mean_token_log_ratio", "mean_advantage",
         "frac_groups_all_equal", "mean_reward")


def oapl_batch_stats(problem, vhat, stats, ws, flags=0):
    rc = lib().oapl_batch_stats(ctypes.byref(problem), _ptr(vhat), _ptr(stats), _ptr(ws), ws.numel(), flags,
                                _stream())
    if rc != OAPL_OK:
        raise OaplError(rc, "oapl_batch_stats")


def oapl_get_last_status(ws) -> int:
    return int(lib().oapl_get_last_status(_ptr(ws), _stream()))


def oapl_get_live_rows(ws) -> int:
    return int(lib().oapl_get_live_rows(_ptr(ws), _stream()))


def oapl_launch_count() -> int:
    return int(lib().oapl_launch_count())


def oapl_debug_gemm(A, B, C, M, N, K, a_mn, b_mn, err, wide=False, wait_cycles=0, skip_step=0):
    if err is None or err.numel() < 2 or err.dtype != torch.int32:
        raise TypeError("err: int32 CUDA tensor of two elements (status word, lock-step counter)")
    rc = lib().oapl_debug_gemm(_ptr(A), _ptr(B), _ptr(C), M, N, K, int(a_mn), int(b_mn), int(wide),
                               int(wait_cycles), int(skip_step), _ptr(err), _stream())
    if rc != OAPL_OK:
        raise OaplError(rc, "oapl_debug_gemm")


KINDS = ("lse_fwd", "grad_chunk", "dH", "dW", "debug", "lse_e")


def oapl_profile_enable(on: bool):
    rc = lib().oapl_profile_enable(int(on))
    if rc != OAPL_OK:
        raise OaplError(rc, "oapl_profile_enable")


def oapl_profile_read(with_dropped: bool = False):
    """{kind: (milliseconds, launches)} since the last read; with_dropped=True also returns the
    number of launches that were not recorded."""
    ms = (ctypes.c_float * len(KINDS))()
    cnt = (ctypes.c_int * len(KINDS))()
    dropped = ctypes.c_int(0)
    rc = lib().oapl_profile_read(ms, cnt, len(KINDS), ctypes.byref(dropped))
    if rc != OAPL_OK:
        raise OaplError(rc, "oapl_profile_read")
    out = {k: (float(ms[i]), int(cnt[i])) for i, k in enumerate(KINDS)}
    return (out, int(dropped.value)) if with_dropped else out


def oapl_profile_read_clocks() -> dict:
    """{kind: SM MHz the kind's launches ran at} since the last read (0 = did not run)."""
    mhz = (ctypes.c_float * len(KINDS))()
    rc = lib().oapl_profile_read_clocks(mhz, len(KINDS))
    if rc != OAPL_OK:
        raise OaplError(rc, "oapl_profile_read_clocks")
    return {k: float(mhz[i]) for i, k in enumerate(KINDS)}


def oapl_token_logprobs_static(problem, token_logp, seq_logp, device_status=None):
    """oapl_token_logprobs without a workspace: the scratch is a fixed array inside the
    library, for callers that must not allocate (N <= 2048, d <= 1024, S <= 2048)."""
    rc = lib().oapl_token_logprobs_static(ctypes.byref(problem), _ptr(token_logp), _ptr(seq_logp),
                                          _ptr(device_status), _stream())
    if rc != OAPL_OK:
        raise OaplError(rc, "oapl_token_logprobs_static")


def make_options(live_rows_bound: int = 0, max_seq_rows_bound: int = 0, dW_ready_event=None) -> OaplCallOptions:
    """Fill oapl_call_options.  dW_ready_event is a torch.cuda.Event that has been recorded at
    least once (torch creates the underlying CUDA event at the first record) or None."""
    o = OaplCallOptions()
    o.live_rows_bound = int(live_rows_bound)
    o.max_seq_rows_bound = int(max_seq_rows_bound)
    if dW_ready_event is None:
        o.dW_ready_event = None
    else:
        handle = int(dW_ready_event.cuda_event)
        if handle == 0:
            raise ValueError("dW_ready_event: record the torch.cuda.Event once before passing it")
        o.dW_ready_event = handle
    return o


def oapl_loss_fwd_bwd_ex(problem, loss, seq_logp, vhat, delta, token_logp, dH, dW, accumulate_dW, ws, options,
                         flags=0):
    rc = lib().oapl_loss_fwd_bwd_ex(ctypes.byref(problem), _ptr(loss), _ptr(seq_logp), _ptr(vhat), _ptr(delta),
                                    _ptr(token_logp), _ptr(dH), _ptr(dW), int(accumulate_dW), _ptr(ws),
                                    ws.numel(), flags, ctypes.byref(options) if options is not None else None,
                                    _stream())
    if rc != OAPL_OK:
        raise OaplError(rc, "oapl_loss_fwd_bwd_ex")


def oapl_get_range_count(ws) -> int:
    return int(lib().oapl_get_range_count(_ptr(ws), _stream()))


def oapl_loss_fwd_bwd(problem, loss, seq_logp, vhat, delta, token_logp, dH, dW, accumulate_dW, ws, flags=0):
    rc = lib().oapl_loss_fwd_bwd(ctypes.byref(problem), _ptr(loss), _ptr(seq_logp), _ptr(vhat), _ptr(delta),
                                 _ptr(token_logp), _ptr(dH), _ptr(dW), int(accumulate_dW), _ptr(ws),
                                 ws.numel(), flags, _stream())
    if rc != OAPL_OK:
        raise OaplError(rc, "oapl_loss_fwd_bwd")
