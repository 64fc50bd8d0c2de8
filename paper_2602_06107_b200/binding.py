"""ctypes binding of libjackpot: argument marshalling only.

Every function has the name and argument order of the C entry point it calls
(see include/jackpot.h); tensors are torch CUDA tensors whose ``data_ptr()`` is
passed through.  There is no fallback: if ``libjackpot.so`` is missing or a call
fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libjackpot.so")

JP_BF16, JP_F32 = 0, 1
JP_LAMBDA_FIXED, JP_LAMBDA_FROM_BUDGET = 0, 1
JP_MAX_TOPK = 128
JP_STATIC_MAX_ROWS = 131072
JP_ERR_TOO_LARGE = -8
JP_DESC_KL = 1
JP_DESC_SPARSE_CAP = 2

EXPORTS = (
    "jp_create", "jp_destroy", "jp_set_stream", "jp_obrs_workspace_bytes", "jp_reserve",
    "jp_obrs_forward", "jp_obrs_forward_sparse_actor", "jp_lmhead_lse_topk", "jp_obrs_forward_lmhead", "jp_obrs_backward", "jp_batch_begin", "jp_batch_chunk", "jp_batch_finalize",
    "jp_obrs_forward_host", "jp_selftest_bounded_wait", "jp_obrs_apply_kappa", "jp_batch_totals", "jp_obrs_apply_totals", "jp_batch_logprobs", "jp_obrs_row_lambda", "jp_vshard_record_floats", "jp_vshard_local", "jp_vshard_local_push", "jp_vshard_merge", "jp_vshard_backward", "jp_budget_lambda_static", "jp_probe_stream", "jp_status_string", "jp_last_error", "jp_launch_count",
    "jp_enable_kernel_timing", "jp_stream_kernel_times",
)


class JackpotError(RuntimeError):
    pass


class jp_obrs_desc(ctypes.Structure):
    _fields_ = [
        ("T", ctypes.c_int64), ("V", ctypes.c_int64), ("ld", ctypes.c_int64),
        ("dtype", ctypes.c_int32), ("lambda_mode", ctypes.c_int32),
        ("c1", ctypes.c_float), ("flags", ctypes.c_int32),
        ("token_offset", ctypes.c_int64),
        ("topk_idx_actor", ctypes.c_void_p), ("topk_idx_policy", ctypes.c_void_p),
        ("topk_val_actor", ctypes.c_void_p), ("topk_val_policy", ctypes.c_void_p),
        ("accept_prob", ctypes.c_void_p), ("uniform", ctypes.c_void_p),
        ("z_approx", ctypes.c_void_p), ("z_exact", ctypes.c_void_p),
        ("lse_actor", ctypes.c_void_p), ("lse_policy", ctypes.c_void_p),
    ]


class jp_stats(ctypes.Structure):
    _fields_ = [
        ("n_valid", ctypes.c_int64), ("n_accept", ctypes.c_int64),
        ("n_bad_token", ctypes.c_int64), ("n_nonfinite", ctypes.c_int64),
        ("alpha_hat", ctypes.c_double), ("mean_accept_prob", ctypes.c_double),
        ("z_approx_mean", ctypes.c_double), ("kappa", ctypes.c_double),
        ("lambda_used", ctypes.c_double), ("mean_kl_p_q", ctypes.c_double),
        ("status", ctypes.c_int32), ("pad", ctypes.c_int32),
    ]

    def as_dict(self):
        d = {n: getattr(self, n) for n, _ in self._fields_ if n != "pad"}
        if d["mean_kl_p_q"] != d["mean_kl_p_q"]:      # NaN in the struct: the divergence was not asked for
            d["mean_kl_p_q"] = None
        return d


class jp_obrs_bwd_desc(ctypes.Structure):
    _fields_ = [
        ("advantages", ctypes.c_void_p), ("lambda_distill", ctypes.c_float),
        ("grad_out", ctypes.c_float), ("n_valid", ctypes.c_int64),
        ("record_offset", ctypes.c_int64),
        ("logp_ref", ctypes.c_void_p), ("logp_actor_ref", ctypes.c_void_p), ("logp_inf", ctypes.c_void_p),
        ("eps_lo", ctypes.c_float), ("eps_hi", ctypes.c_float), ("c2", ctypes.c_float), ("tis_cap", ctypes.c_float),
        ("out_obj_policy", ctypes.c_void_p), ("out_obj_actor", ctypes.c_void_p), ("out_kl", ctypes.c_void_p),
        ("out_loss", ctypes.c_void_p),
    ]


STATS_BYTES = ctypes.sizeof(jp_stats)
_lib = None


def load():
    """Loads libjackpot.so; raises if it was not built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise JackpotError(f"{LIB_PATH} not found: build it with "
                           "`python -m paper_2602_06107_b200.build` (no CPU fallback exists)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i64, i32, f32, u64 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_float, ctypes.c_uint64
    lib.jp_create.argtypes = [ctypes.POINTER(vp), ctypes.c_int, vp]
    lib.jp_destroy.argtypes = [vp]
    lib.jp_set_stream.argtypes = [vp, vp]
    lib.jp_obrs_workspace_bytes.argtypes = [i64, i64, ctypes.c_int]
    lib.jp_obrs_workspace_bytes.restype = ctypes.c_size_t
    lib.jp_reserve.argtypes = [vp, i64, i64, ctypes.c_int]
    lib.jp_obrs_forward.argtypes = [vp, ctypes.POINTER(jp_obrs_desc), vp, vp, vp, vp, f32, ctypes.c_int, u64,
                                    vp, vp, vp, vp, vp]
    lib.jp_obrs_forward_sparse_actor.argtypes = [vp, ctypes.POINTER(jp_obrs_desc), vp, vp, vp, vp, vp, vp, ctypes.c_int,
                                                 f32, ctypes.c_int, u64, vp, vp, vp, vp, vp, vp]
    lib.jp_lmhead_lse_topk.argtypes = [vp, vp, i64, vp, i64, vp, vp, i64, i64, i64, ctypes.c_int, vp, vp, vp, vp, vp]
    lib.jp_obrs_forward_lmhead.argtypes = [vp, ctypes.POINTER(jp_obrs_desc), vp, i64, vp, i64, i64, vp, i64, vp, i64, i64,
                                           vp, vp, f32, ctypes.c_int, u64, vp, vp, vp, vp, vp]
    lib.jp_obrs_forward_host.argtypes = lib.jp_obrs_forward.argtypes + [i64]
    lib.jp_obrs_backward.argtypes = [vp, ctypes.POINTER(jp_obrs_desc), ctypes.POINTER(jp_obrs_bwd_desc),
                                     vp, vp, vp, vp, vp, vp, vp, vp]
    lib.jp_obrs_apply_kappa.argtypes = [vp, ctypes.c_double, f32, vp]
    lib.jp_batch_logprobs.argtypes = [vp, vp, vp, vp]
    lib.jp_selftest_bounded_wait.argtypes = [vp, i64, vp]
    lib.jp_batch_totals.argtypes = [vp, vp]
    lib.jp_obrs_apply_totals.argtypes = [vp, vp, f32, vp, vp]
    lib.jp_obrs_row_lambda.argtypes = [vp, ctypes.POINTER(jp_obrs_desc), vp, vp, vp, f32, vp, vp, vp, vp]
    lib.jp_vshard_record_floats.argtypes = [ctypes.c_int]
    lib.jp_vshard_record_floats.restype = ctypes.c_size_t
    lib.jp_vshard_local.argtypes = [vp, ctypes.POINTER(jp_obrs_desc), vp, vp, vp, vp, i64, i64, ctypes.c_int, vp]
    lib.jp_vshard_local_push.argtypes = [vp, ctypes.POINTER(jp_obrs_desc), vp, vp, vp, vp, i64, i64, ctypes.c_int,
                                         ctypes.c_int, ctypes.c_int, ctypes.POINTER(vp)]
    lib.jp_vshard_merge.argtypes = [vp, ctypes.c_int, ctypes.c_int, vp, i64, i64, ctypes.c_int]
    lib.jp_vshard_backward.argtypes = [vp, ctypes.POINTER(jp_obrs_desc), ctypes.POINTER(jp_obrs_bwd_desc),
                                       vp, vp, vp, vp, i64, vp, vp, vp, vp]
    lib.jp_budget_lambda_static.argtypes = [vp, vp, vp, i64, f32, vp, vp]
    lib.jp_probe_stream.argtypes = [vp, vp, i64, ctypes.c_int, vp, ctypes.POINTER(ctypes.c_float)]
    lib.jp_batch_begin.argtypes = [vp, i64, i64, i32, ctypes.c_int, f32]
    lib.jp_batch_chunk.argtypes = [vp, ctypes.POINTER(jp_obrs_desc), vp, vp, vp, vp]
    lib.jp_batch_finalize.argtypes = [vp, ctypes.POINTER(jp_obrs_desc), f32, i32, u64, vp, vp, vp, vp, vp]
    lib.jp_status_string.argtypes = [ctypes.c_int]
    lib.jp_status_string.restype = ctypes.c_char_p
    lib.jp_last_error.argtypes = [vp]
    lib.jp_last_error.restype = ctypes.c_char_p
    lib.jp_launch_count.argtypes = [vp]
    lib.jp_launch_count.restype = i64
    lib.jp_enable_kernel_timing.argtypes = [vp, ctypes.c_int]
    lib.jp_stream_kernel_times.argtypes = [vp, ctypes.POINTER(ctypes.c_float), i64]
    lib.jp_stream_kernel_times.restype = i64
    for name in EXPORTS:
        getattr(lib, name)          # raises AttributeError if the library lacks an entry point
    _lib = lib
    return lib


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        return ctypes.c_void_p(t.data_ptr())
    return ctypes.c_void_p(int(t))


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return JP_BF16
    if t.dtype == torch.float32:
        return JP_F32
    raise JackpotError(f"logits must be bfloat16 or float32, got {t.dtype}")


class Context:
    """Owns one jp_ctx bound to a device and to torch's current stream on it."""

    def __init__(self, device: int = 0, stream=None):
        self.lib = load()
        self.device = device
        h = ctypes.c_void_p()
        if stream is None:
            stream = torch.cuda.current_stream(device).cuda_stream
        st = self.lib.jp_create(ctypes.byref(h), device, ctypes.c_void_p(stream))
        if st != 0:
            raise JackpotError(f"jp_create failed: {self.lib.jp_status_string(st).decode()}")
        self.h = h

    def close(self):
        if getattr(self, "h", None):
            self.lib.jp_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def check(self, st: int):
        if st != 0:
            raise JackpotError(f"{self.lib.jp_status_string(st).decode()} ({st}): "
                               f"{self.lib.jp_last_error(self.h).decode()}")

    def launch_count(self) -> int:
        return int(self.lib.jp_launch_count(self.h))


def make_desc(logits: torch.Tensor, *, lambda_mode=JP_LAMBDA_FIXED, c1=0.0, token_offset=0, aux=None,
              T=None, flags=0) -> jp_obrs_desc:
    d = jp_obrs_desc()
    d.T = logits.shape[0] if T is None else T
    d.V = logits.shape[1]
    d.ld = logits.stride(0)
    d.dtype = _dtype_code(logits)
    d.lambda_mode = lambda_mode
    d.c1 = c1
    d.token_offset = token_offset
    d.flags = flags
    for name, t in (aux or {}).items():
        setattr(d, name, t.data_ptr() if t is not None else None)
    return d


def jp_reserve(ctx: Context, T_max: int, V: int, k: int):
    ctx.check(ctx.lib.jp_reserve(ctx.h, T_max, V, k))


def jp_obrs_forward(ctx: Context, desc: jp_obrs_desc, actor_logits, policy_logits, tokens, mask,
                    lambda_or_budget: float, k: int, seed: int, out_accept, out_weight, out_logp_actor,
                    out_logp_policy, out_stats):
    ctx.check(ctx.lib.jp_obrs_forward(ctx.h, ctypes.byref(desc), _ptr(actor_logits), _ptr(policy_logits),
                                      _ptr(tokens), _ptr(mask), lambda_or_budget, k, seed,
                                      _ptr(out_accept), _ptr(out_weight), _ptr(out_logp_actor),
                                      _ptr(out_logp_policy), _ptr(out_stats)))


def jp_obrs_forward_sparse_actor(ctx: Context, desc: jp_obrs_desc, policy_logits, tokens, mask, logp_inf_token,
                                 topk_inf_idx, topk_inf_logp, k_inf: int, lambda_or_budget: float, k: int, seed: int,
                                 out_accept, out_weight, out_logp_policy, out_z_lower, out_z_upper, out_stats):
    ctx.check(ctx.lib.jp_obrs_forward_sparse_actor(ctx.h, ctypes.byref(desc), _ptr(policy_logits), _ptr(tokens),
                                                   _ptr(mask), _ptr(logp_inf_token), _ptr(topk_inf_idx),
                                                   _ptr(topk_inf_logp), k_inf, lambda_or_budget, k, seed,
                                                   _ptr(out_accept), _ptr(out_weight), _ptr(out_logp_policy),
                                                   _ptr(out_z_lower), _ptr(out_z_upper), _ptr(out_stats)))


def jp_lmhead_lse_topk(ctx: Context, hidden, weight, tokens, mask, k: int, out_lse, out_logp_token, out_topk_idx,
                       out_topk_val, out_status=None):
    """hidden [T, H] and weight [V, H]: bf16 CUDA tensors (rows may be padded: the stride is passed on)."""
    T, H = hidden.shape
    V = weight.shape[0]
    ctx.check(ctx.lib.jp_lmhead_lse_topk(ctx.h, _ptr(hidden), hidden.stride(0), _ptr(weight), weight.stride(0),
                                         _ptr(tokens), _ptr(mask), T, H, V, k, _ptr(out_lse), _ptr(out_logp_token),
                                         _ptr(out_topk_idx), _ptr(out_topk_val), _ptr(out_status)))


def jp_obrs_forward_lmhead(ctx: Context, desc: jp_obrs_desc, hidden_actor, weight_actor, hidden_policy, weight_policy,
                           tokens, mask, lambda_or_budget: float, k: int, seed: int, out_accept, out_weight,
                           out_logp_actor, out_logp_policy, out_stats):
    """hidden_* [T, H_*] and weight_* [V, H_*]: bf16 CUDA tensors (strides are passed on); desc carries T and V."""
    ctx.check(ctx.lib.jp_obrs_forward_lmhead(
        ctx.h, ctypes.byref(desc), _ptr(hidden_actor), hidden_actor.stride(0), _ptr(weight_actor), weight_actor.stride(0),
        hidden_actor.shape[1], _ptr(hidden_policy), hidden_policy.stride(0), _ptr(weight_policy),
        weight_policy.stride(0), hidden_policy.shape[1], _ptr(tokens), _ptr(mask), lambda_or_budget, k, seed,
        _ptr(out_accept), _ptr(out_weight), _ptr(out_logp_actor), _ptr(out_logp_policy), _ptr(out_stats)))


def jp_obrs_forward_host(ctx: Context, desc: jp_obrs_desc, actor_logits, policy_logits, tokens, mask,
                         lambda_or_budget: float, k: int, seed: int, out_accept, out_weight,
                         out_logp_actor, out_logp_policy, out_stats, chunk_rows: int = 0):
    """All tensors are CPU tensors (pinned for asynchronous copies); out_stats is a
    CPU uint8 tensor of STATS_BYTES bytes or None."""
    ctx.check(ctx.lib.jp_obrs_forward_host(ctx.h, ctypes.byref(desc), _ptr(actor_logits),
                                           _ptr(policy_logits), _ptr(tokens), _ptr(mask),
                                           lambda_or_budget, k, seed, _ptr(out_accept), _ptr(out_weight),
                                           _ptr(out_logp_actor), _ptr(out_logp_policy), _ptr(out_stats),
                                           chunk_rows))


def jp_obrs_backward(ctx: Context, desc: jp_obrs_desc, bwd: jp_obrs_bwd_desc, actor_logits, policy_logits,
                     tokens, mask, accept, weight, d_actor_logits, d_policy_logits):
    ctx.check(ctx.lib.jp_obrs_backward(ctx.h, ctypes.byref(desc), ctypes.byref(bwd), _ptr(actor_logits),
                                       _ptr(policy_logits), _ptr(tokens), _ptr(mask), _ptr(accept),
                                       _ptr(weight), _ptr(d_actor_logits), _ptr(d_policy_logits)))


def jp_obrs_row_lambda(ctx: Context, desc, za, zp, mask, budget: float, out_lambda, out_kl_before=None,
                       out_kl_after=None, out_iterations=None):
    ctx.check(ctx.lib.jp_obrs_row_lambda(ctx.h, ctypes.byref(desc), _ptr(za), _ptr(zp), _ptr(mask), budget,
                                         _ptr(out_lambda), _ptr(out_kl_before), _ptr(out_kl_after),
                                         _ptr(out_iterations)))


def jp_vshard_record_floats(k: int) -> int:
    return int(load().jp_vshard_record_floats(k))


def jp_vshard_local(ctx: Context, desc, za, zp, tokens, mask, vocab_offset: int, V_total: int, k: int, out_packed):
    ctx.check(ctx.lib.jp_vshard_local(ctx.h, ctypes.byref(desc), _ptr(za), _ptr(zp), _ptr(tokens), _ptr(mask),
                                      vocab_offset, V_total, k, _ptr(out_packed)))


def jp_vshard_local_push(ctx: Context, desc, za, zp, tokens, mask, vocab_offset: int, V_total: int, k: int,
                         my_shard: int, gathered_of_shard):
    """``gathered_of_shard``: per shard, its gathered buffer as this device addresses it (tensor or raw pointer)."""
    n = len(gathered_of_shard)
    arr = (ctypes.c_void_p * n)(*[_ptr(g) for g in gathered_of_shard])
    ctx.check(ctx.lib.jp_vshard_local_push(ctx.h, ctypes.byref(desc), _ptr(za), _ptr(zp), _ptr(tokens), _ptr(mask),
                                           vocab_offset, V_total, k, n, my_shard, arr))


def jp_vshard_merge(ctx: Context, n_shards: int, my_shard: int, gathered, T: int, V_total: int, k: int):
    ctx.check(ctx.lib.jp_vshard_merge(ctx.h, n_shards, my_shard, _ptr(gathered), T, V_total, k))


def jp_vshard_backward(ctx: Context, desc, bwd, za, zp, tokens, mask, vocab_offset: int, accept, weight, d_actor,
                       d_policy):
    ctx.check(ctx.lib.jp_vshard_backward(ctx.h, ctypes.byref(desc), ctypes.byref(bwd), _ptr(za), _ptr(zp),
                                         _ptr(tokens), _ptr(mask), vocab_offset, _ptr(accept), _ptr(weight),
                                         _ptr(d_actor), _ptr(d_policy)))


def jp_batch_logprobs(ctx: Context, out_logp_actor, out_logp_policy, out_valid):
    ctx.check(ctx.lib.jp_batch_logprobs(ctx.h, _ptr(out_logp_actor), _ptr(out_logp_policy), _ptr(out_valid)))


def jp_obrs_apply_kappa(ctx: Context, kappa: float, c1: float, out_weight):
    ctx.check(ctx.lib.jp_obrs_apply_kappa(ctx.h, kappa, c1, _ptr(out_weight)))


def jp_selftest_bounded_wait(ctx: Context, limit_cycles: int, out_status):
    ctx.check(ctx.lib.jp_selftest_bounded_wait(ctx.h, limit_cycles, _ptr(out_status)))


def jp_batch_totals(ctx: Context, out_totals):
    ctx.check(ctx.lib.jp_batch_totals(ctx.h, _ptr(out_totals)))


def jp_obrs_apply_totals(ctx: Context, totals, c1: float, out_weight, out_stats=None):
    ctx.check(ctx.lib.jp_obrs_apply_totals(ctx.h, _ptr(totals), c1, _ptr(out_weight), _ptr(out_stats)))


def jp_budget_lambda_static(logp_actor, logp_policy, mask, T: int, budget: float, out_lambda, stream=None) -> int:
    """Calls the allocation-free budget solve on the current device and returns its
    status code (0 = ok) instead of raising, so that callers can test the limits."""
    lib = load()
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    return int(lib.jp_budget_lambda_static(_ptr(logp_actor), _ptr(logp_policy), _ptr(mask), T, budget,
                                           _ptr(out_lambda), ctypes.c_void_p(stream)))


def jp_probe_stream(src, dst=None, reps: int = 10, stream=None) -> float:
    """GB/s of a plain kernel that reads ``src`` (and writes it to ``dst`` if given): bytes moved / device time."""
    lib = load()
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    nbytes = src.numel() * src.element_size()
    ms = ctypes.c_float(0.0)
    st = lib.jp_probe_stream(_ptr(src), _ptr(dst), nbytes, reps, ctypes.c_void_p(stream), ctypes.byref(ms))
    if st != 0:
        raise JackpotError(f"jp_probe_stream: {lib.jp_status_string(st).decode()}")
    moved = nbytes * (2 if dst is not None else 1)
    return moved / (ms.value * 1e-3) / 1e9


def jp_batch_begin(ctx: Context, T_total: int, V: int, dtype: int, k: int, fixed_lambda_for_exact_mode=0.0):
    ctx.check(ctx.lib.jp_batch_begin(ctx.h, T_total, V, dtype, k, fixed_lambda_for_exact_mode))


def jp_batch_chunk(ctx: Context, desc: jp_obrs_desc, actor_logits, policy_logits, tokens, mask):
    ctx.check(ctx.lib.jp_batch_chunk(ctx.h, ctypes.byref(desc), _ptr(actor_logits), _ptr(policy_logits),
                                     _ptr(tokens), _ptr(mask)))


def jp_batch_finalize(ctx: Context, desc_outputs, lambda_or_budget: float, lambda_mode: int, seed: int,
                      out_accept, out_weight, out_logp_actor, out_logp_policy, out_stats):
    dref = ctypes.byref(desc_outputs) if desc_outputs is not None else None
    ctx.check(ctx.lib.jp_batch_finalize(ctx.h, dref, lambda_or_budget, lambda_mode, seed, _ptr(out_accept),
                                        _ptr(out_weight), _ptr(out_logp_actor), _ptr(out_logp_policy),
                                        _ptr(out_stats)))


def new_stats_buffer(device) -> torch.Tensor:
    return torch.zeros(STATS_BYTES, dtype=torch.uint8, device=device)


def read_stats(buf: torch.Tensor) -> dict:
    """Copies a device (or host) jp_stats buffer to the host and decodes it."""
    raw = bytes(buf.detach().cpu().numpy().tobytes())
    return jp_stats.from_buffer_copy(raw).as_dict()


def make_bwd_desc(advantages=None, lambda_distill=0.0, grad_out=1.0, n_valid=0, record_offset=0, *,
                  logp_ref=None, logp_actor_ref=None, logp_inf=None, eps_lo=0.0, eps_hi=0.0, c2=0.0, tis_cap=0.0,
                  out_obj_policy=None, out_obj_actor=None, out_kl=None, out_loss=None):
    b = jp_obrs_bwd_desc()
    b.advantages = advantages.data_ptr() if advantages is not None else None
    b.lambda_distill = lambda_distill
    b.grad_out = grad_out
    b.n_valid = n_valid
    b.record_offset = record_offset
    for name, t in (("logp_ref", logp_ref), ("logp_actor_ref", logp_actor_ref), ("logp_inf", logp_inf),
                    ("out_obj_policy", out_obj_policy), ("out_obj_actor", out_obj_actor), ("out_kl", out_kl),
                    ("out_loss", out_loss)):
        setattr(b, name, t.data_ptr() if t is not None else None)
    b.eps_lo, b.eps_hi, b.c2, b.tis_cap = eps_lo, eps_hi, c2, tis_cap
    return b


def jp_enable_kernel_timing(ctx: Context, on: bool):
    ctx.check(ctx.lib.jp_enable_kernel_timing(ctx.h, 1 if on else 0))


def jp_stream_kernel_times(ctx: Context, n: int):
    buf = (ctypes.c_float * n)()
    got = ctx.lib.jp_stream_kernel_times(ctx.h, buf, n)
    return [float(buf[i]) for i in range(got)]
