"""Thin ctypes binding over the C ABI of include/surelock.h: argument marshalling only.

Function names match the C entry points.  Tensors are torch CUDA tensors used as
device memory; their `data_ptr()` is what crosses the boundary.  Outputs that the
library owns are exposed as zero-copy torch views of the library's buffers.
There is no fallback: if the shared library is missing, `lib()` raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsurelock.so")
SL_BF16, SL_FP32 = 0, 1
_lib = None


class SurelockError(RuntimeError):
    pass


class _ModelCfg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "head_dim", "n_kv_heads", "d_ff", "vocab",
                                         "dtype")] + [("rms_eps", C.c_float), ("rope_theta", C.c_float),
                                                      ("mask_token_id", C.c_int32)]


class _Weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("tok_emb", "lm_head", "final_norm_g")] + \
               [(n, C.POINTER(C.c_void_p)) for n in ("attn_norm_g", "wq", "wk", "wv", "wo", "ffn_norm_g", "w_gate",
                                                     "w_up", "w_down")]


class _StepOut(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("active_idx", "row_offsets", "n_active", "logits", "hidden", "kl", "conf",
                                          "argmax")]


class _UnlockParams(C.Structure):
    _fields_ = [("period", C.c_int), ("eps_unlock", C.c_float), ("d_interval", C.c_int), ("d_cool", C.c_int),
                ("rho", C.c_float), ("m_percent", C.c_float)]


class _ProbeOut(C.Structure):
    _fields_ = [("step", C.c_int32), ("probed", C.c_int32)] + \
               [(n, C.c_void_p) for n in ("probed_idx", "n_probed", "drift", "conf", "theta", "n_unlocked", "t_star",
                                          "cool_until")]


def lib() -> C.CDLL:
    """Load libsurelock.so (built in-tree by `paper_2602_06412_b200.build`); raises if it is not there."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise SurelockError(f"{LIB_PATH} not built: run `python -m paper_2602_06412_b200.build` "
                            "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp, i32, f32, sz = C.c_void_p, C.c_int, C.c_float, C.c_size_t
    sig = {
        "surelock_init": (i32, [C.POINTER(vp), C.POINTER(_ModelCfg), C.POINTER(_Weights), i32, i32, vp]),
        "surelock_reset": (i32, [vp]),
        "surelock_step": (i32, [vp, vp, vp, vp, f32, C.POINTER(_StepOut)]),
        "surelock_step_host": (i32, [vp, vp, vp, vp, f32, vp, vp, vp, vp, vp]),
        "surelock_layer_step": (i32, [vp, i32, vp, vp, vp, C.POINTER(_StepOut)]),
        "surelock_status_poll": (i32, [vp, C.POINTER(i32)]),
        "surelock_kv_cache": (i32, [vp, i32, C.POINTER(vp), C.POINTER(vp), C.POINTER(sz)]),
        "surelock_prev_logits": (i32, [vp, C.POINTER(vp), C.POINTER(vp)]),
        "surelock_set_option": (i32, [vp, C.c_char_p, i32]),
        "surelock_last_launch_count": (i32, [vp]),
        "surelock_last_fallback_count": (i32, [vp]),
        "surelock_last_step_paths": (i32, [vp]),
        "surelock_attention_split_workspace_bytes": (C.c_size_t, [i32, i32, i32]),
        "surelock_attention_split": (i32, [vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, vp, i32, vp, vp]),
        "surelock_set_confidence_gate": (i32, [vp, f32, C.POINTER(vp)]),
        "surelock_set_unlocking": (i32, [vp, C.POINTER(_UnlockParams)]),
        "surelock_probe_unlock": (i32, [vp, vp, vp, C.POINTER(_ProbeOut)]),
        "surelock_conf_gate_lock": (i32, [vp, vp, vp, vp, i32, i32, vp, vp, f32, f32, vp, vp]),
        "surelock_update_mask": (i32, [vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp]),
        "surelock_state_bytes": (sz, [vp]),
        "surelock_state_export": (i32, [vp, vp, sz, C.POINTER(sz)]),
        "surelock_state_import": (i32, [vp, vp, sz]),
        "surelock_layer_trace": (i32, [vp, C.POINTER(vp), C.POINTER(sz)]),
        "surelock_kernel_times": (i32, [vp, vp, vp, i32]),
        "surelock_destroy": (None, [vp]),
        "surelock_strerror": (C.c_char_p, [i32]),
        "surelock_compact_scratch_bytes": (sz, [C.c_int64]),
        "surelock_compact": (i32, [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp]),
        "surelock_compact_from_ticket": (i32, [vp, i32, i32, vp, vp, vp, vp, vp, C.c_uint32, vp, vp]),
        "surelock_compact_noalloc": (i32, [vp, i32, i32, vp, vp, vp, vp, vp, vp]),
        "surelock_compact_noalloc_max_flags": (C.c_int64, []),
        "surelock_kv_scatter": (i32, [vp, vp, vp, vp, i32, i32, vp, vp, i32, vp]),
        "surelock_softmax_kl_sure": (i32, [vp, vp, vp, vp, vp, vp, i32, i32, i32, vp, vp, f32, vp, vp, vp, vp, vp]),
        "surelock_gemm": (i32, [vp, vp, vp, vp, i32, i32, i32, i32, i32, vp, vp, vp]),
        "surelock_gemm_workspace_bytes": (sz, []),
        "surelock_gemm_fused": (i32, [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, vp, vp]),
        "surelock_attention": (i32, [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, vp, i32, i32, vp, vp]),
    }
    for name, (res, args) in sig.items():
        f = getattr(L, name)
        f.restype, f.argtypes = res, args
    _lib = L
    return L


def _check(rc: int, what: str):
    if rc != 0:
        raise SurelockError(f"{what}: {lib().surelock_strerror(rc).decode()} ({rc})")


def _p(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_contiguous(), "tensors crossing the C ABI must be contiguous"
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return SL_BF16
    if t.dtype == torch.float32:
        return SL_FP32
    raise SurelockError(f"unsupported dtype {t.dtype}")


class _DevArray:
    def __init__(self, ptr, shape, typestr):
        self.__cuda_array_interface__ = dict(data=(ptr, False), shape=tuple(shape), typestr=typestr, version=2,
                                             strides=None)


def device_view(ptr: int, shape, dtype: torch.dtype) -> torch.Tensor:
    """Zero-copy torch view of library-owned device memory."""
    ts = {torch.int32: "<i4", torch.float32: "<f4", torch.uint8: "|u1", torch.bfloat16: "<i2"}[dtype]
    t = torch.as_tensor(_DevArray(ptr, shape, ts), device="cuda")
    return t.view(torch.bfloat16) if dtype == torch.bfloat16 else t


class StepOut:
    """Views of a step's packed outputs; every array has room for B*N rows, the first M = n_active are valid."""

    def __init__(self, raw: _StepOut, R: int, B: int, d: int, V: int, tdtype):
        self.active_idx = device_view(raw.active_idx, (R,), torch.int32)
        self.row_offsets = device_view(raw.row_offsets, (B + 1,), torch.int32)
        self.n_active = device_view(raw.n_active, (1,), torch.int32)
        self.hidden = device_view(raw.hidden, (R, d), torch.float32) if raw.hidden else None
        self.logits = device_view(raw.logits, (R, V), tdtype) if raw.logits and V > 0 else None
        self.kl = device_view(raw.kl, (R,), torch.float32) if raw.kl else None
        self.conf = device_view(raw.conf, (R,), torch.float32) if raw.conf else None
        self.argmax = device_view(raw.argmax, (R,), torch.int32) if raw.argmax else None

    def M(self) -> int:
        return int(self.n_active.item())


class Ctx:
    def __init__(self, handle, cfg, N, B, tdtype, keep):
        self.handle, self.cfg, self.N, self.B, self.tdtype, self._keep = handle, cfg, N, B, tdtype, keep

    def __del__(self):
        try:
            surelock_destroy(self)
        except Exception:
            pass


def surelock_init(cfg: Dict, weights: Dict, N: int, batch: int) -> Ctx:
    """cfg: dict with the model shape; weights: dict of CUDA tensors (layout of inputs.make_weights)."""
    layers = weights["layers"]
    tdtype = layers[0]["wq"].dtype
    mc = _ModelCfg(cfg["n_layers"], cfg["d_model"], cfg["n_heads"], cfg["head_dim"], cfg["n_heads"], cfg["d_ff"],
                   cfg["vocab"], _dt(layers[0]["wq"]), cfg["rms_eps"], cfg["rope_theta"], max(cfg["vocab"] - 1, 0))
    w = _Weights()
    keep = []
    for name in ("tok_emb", "lm_head", "final_norm_g"):
        setattr(w, name, _p(weights.get(name)) if cfg["vocab"] > 0 else None)
    for name in ("attn_norm_g", "wq", "wk", "wv", "wo", "ffn_norm_g", "w_gate", "w_up", "w_down"):
        arr = (C.c_void_p * len(layers))(*[_p(lw[name]) for lw in layers])
        keep.append(arr)
        setattr(w, name, C.cast(arr, C.POINTER(C.c_void_p)))
    h = C.c_void_p()
    _check(lib().surelock_init(C.byref(h), C.byref(mc), C.byref(w), N, batch, _stream()), "surelock_init")
    return Ctx(h, dict(cfg), N, batch, tdtype, (keep, weights))


def surelock_destroy(ctx: Ctx):
    if ctx.handle:
        lib().surelock_destroy(ctx.handle)
        ctx.handle = None


def surelock_reset(ctx: Ctx):
    _check(lib().surelock_reset(ctx.handle), "surelock_reset")


def surelock_step(ctx: Ctx, tokens, mask_state, lock_mask, kl_eps: float) -> StepOut:
    raw = _StepOut()
    _check(lib().surelock_step(ctx.handle, _p(tokens), _p(mask_state), _p(lock_mask), kl_eps, C.byref(raw)),
           "surelock_step")
    return StepOut(raw, ctx.N * ctx.B, ctx.B, ctx.cfg["d_model"], ctx.cfg["vocab"], ctx.tdtype)


def surelock_step_host(ctx: Ctx, tokens, mask_state, lock_mask, kl_eps: float, n_active, active_idx=None, kl=None,
                       conf=None, argmax=None):
    """All tensors are HOST (CPU, ideally pinned) tensors; lock_mask is updated in place."""
    _check(lib().surelock_step_host(ctx.handle, _p(tokens), _p(mask_state), _p(lock_mask), kl_eps, _p(n_active),
                                    _p(active_idx), _p(kl), _p(conf), _p(argmax)), "surelock_step_host")


def surelock_layer_step(ctx: Ctx, layer: int, hidden_in, lock_mask, hidden_out) -> StepOut:
    raw = _StepOut()
    _check(lib().surelock_layer_step(ctx.handle, layer, _p(hidden_in), _p(lock_mask), _p(hidden_out), C.byref(raw)),
           "surelock_layer_step")
    return StepOut(raw, ctx.N * ctx.B, ctx.B, ctx.cfg["d_model"], 0, ctx.tdtype)


def surelock_status_poll(ctx: Ctx) -> int:
    s = C.c_int(0)
    rc = lib().surelock_status_poll(ctx.handle, C.byref(s))
    if rc not in (0, -4):
        _check(rc, "surelock_status_poll")
    return s.value


def surelock_kv_cache(ctx: Ctx, layer: int):
    k, v, stride = C.c_void_p(), C.c_void_p(), C.c_size_t()
    _check(lib().surelock_kv_cache(ctx.handle, layer, C.byref(k), C.byref(v), C.byref(stride)), "surelock_kv_cache")
    shape = (ctx.B * ctx.N, ctx.cfg["n_heads"], ctx.cfg["head_dim"])
    return device_view(k.value, shape, ctx.tdtype), device_view(v.value, shape, ctx.tdtype)


def surelock_prev_logits(ctx: Ctx):
    buf, rop = C.c_void_p(), C.c_void_p()
    _check(lib().surelock_prev_logits(ctx.handle, C.byref(buf), C.byref(rop)), "surelock_prev_logits")
    R = ctx.B * ctx.N
    return device_view(buf.value, (R, ctx.cfg["vocab"]), ctx.tdtype), device_view(rop.value, (R,), torch.int32)


def surelock_set_option(ctx: Ctx, name: str, value: int):
    _check(lib().surelock_set_option(ctx.handle, name.encode(), value), "surelock_set_option")


def surelock_layer_trace(ctx: Ctx) -> torch.Tensor:
    """View [2L+1][B*N][d] fp32 of the residual stream of the last step: slot 2l = input of block l, 2l+1 = after
    its attention sub-block, 2L = output of the last block ("trace_layers" must be on)."""
    buf, stride = C.c_void_p(), C.c_size_t()
    _check(lib().surelock_layer_trace(ctx.handle, C.byref(buf), C.byref(stride)), "surelock_layer_trace")
    return device_view(buf.value, (2 * ctx.cfg["n_layers"] + 1, ctx.B * ctx.N, ctx.cfg["d_model"]), torch.float32)


def surelock_set_confidence_gate(ctx: Ctx, m_percent: float) -> torch.Tensor:
    """Switch the optional confidence gate on (0 <= m_percent <= 100) or off (negative).  Returns a view of the B
    per-sequence thresholds theta_m that later steps fill."""
    th = C.c_void_p()
    _check(lib().surelock_set_confidence_gate(ctx.handle, m_percent, C.byref(th)), "surelock_set_confidence_gate")
    return device_view(th.value, (ctx.B,), torch.float32)


class ProbeOut:
    """Views of the outputs of surelock_probe_unlock (the first n_probed rows of the packed arrays are valid)."""

    def __init__(self, raw: _ProbeOut, R: int, B: int):
        self.step, self.probed = int(raw.step), bool(raw.probed)
        if self.probed:
            self.probed_idx = device_view(raw.probed_idx, (R,), torch.int32)
            self.n_probed = device_view(raw.n_probed, (1,), torch.int32)
            self.drift = device_view(raw.drift, (R,), torch.float32)
            self.conf = device_view(raw.conf, (R,), torch.float32)
            self.theta = device_view(raw.theta, (B,), torch.float32)
            self.n_unlocked = device_view(raw.n_unlocked, (1,), torch.int32)
            self.t_star = device_view(raw.t_star, (R,), torch.int32)
            self.cool_until = device_view(raw.cool_until, (R,), torch.int32)


def surelock_set_unlocking(ctx: Ctx, period: int = 1, eps_unlock: float = 0.0, d_interval: int = 0, d_cool: int = 0,
                           rho: float = 1.0, m_percent: float = 20.0, off: bool = False):
    """Optional un-locking (App. "Optional Unlocking") on with these parameters, or off."""
    if off:
        _check(lib().surelock_set_unlocking(ctx.handle, None), "surelock_set_unlocking")
        return
    p = _UnlockParams(period, eps_unlock, d_interval, d_cool, rho, m_percent)
    _check(lib().surelock_set_unlocking(ctx.handle, C.byref(p)), "surelock_set_unlocking")


def surelock_probe_unlock(ctx: Ctx, tokens, lock_mask) -> ProbeOut:
    raw = _ProbeOut()
    _check(lib().surelock_probe_unlock(ctx.handle, _p(tokens), _p(lock_mask), C.byref(raw)), "surelock_probe_unlock")
    return ProbeOut(raw, ctx.B * ctx.N, ctx.B)


def surelock_conf_gate_lock(conf, kl, active_idx, row_offsets, B: int, N: int, mask_state, lock_mask, kl_eps: float,
                            m_percent: float, theta_out=None):
    _check(lib().surelock_conf_gate_lock(_p(conf), _p(kl), _p(active_idx), _p(row_offsets), B, N, _p(mask_state),
                                         _p(lock_mask), kl_eps, m_percent, _p(theta_out), _stream()),
           "surelock_conf_gate_lock")


def surelock_update_mask(conf, argmax, active_idx, row_offsets, B: int, N: int, lo: int, hi: int, k: int,
                         mask_token: int, tokens, mask_state, n_revealed=None):
    """UpdateMASK (Algorithm 1 line 16) on the device; tokens int32 [B][N] and mask_state uint8 [B][N] in place."""
    _check(lib().surelock_update_mask(_p(conf), _p(argmax), _p(active_idx), _p(row_offsets), B, N, lo, hi, k, mask_token,
                                      _p(tokens), _p(mask_state), _p(n_revealed), _stream()), "surelock_update_mask")


def surelock_state_export(ctx: Ctx) -> bytes:
    """Checkpoint of what the ctx holds between two steps (K/V cache, previous posterior), as host bytes."""
    cap = lib().surelock_state_bytes(ctx.handle)
    buf = (C.c_char * cap)()
    n = C.c_size_t(0)
    _check(lib().surelock_state_export(ctx.handle, C.cast(buf, C.c_void_p), cap, C.byref(n)), "surelock_state_export")
    return bytes(memoryview(buf)[: n.value])


def surelock_state_import(ctx: Ctx, state: bytes):
    buf = (C.c_char * len(state)).from_buffer_copy(state)
    _check(lib().surelock_state_import(ctx.handle, C.cast(buf, C.c_void_p), len(state)), "surelock_state_import")


def surelock_last_launch_count(ctx: Ctx) -> int:
    return lib().surelock_last_launch_count(ctx.handle)


def surelock_last_fallback_count(ctx: Ctx) -> int:
    return lib().surelock_last_fallback_count(ctx.handle)


def surelock_last_step_paths(ctx: Ctx) -> int:
    """Bit 0: the last call used the layer chain kernel; bit 1: split-key attention."""
    return lib().surelock_last_step_paths(ctx.handle)


KERNEL_CLASSES = ("compact", "gather", "rmsnorm", "gemm_qkv", "rope", "kv_scatter", "attention", "gemm_o",
                  "gemm_gateup", "gemm_down", "gemm_head", "softmax_kl", "conf_gate")


def surelock_kernel_times(ctx: Ctx):
    """{class: (ms, launches)} of the last step (needs surelock_set_option(ctx, "time_kernels", 1))."""
    n = len(KERNEL_CLASSES)
    ms = (C.c_float * n)()
    cnt = (C.c_int32 * n)()
    _check(lib().surelock_kernel_times(ctx.handle, C.cast(ms, C.c_void_p), C.cast(cnt, C.c_void_p), n),
           "surelock_kernel_times")
    return {k: (ms[i], cnt[i]) for i, k in enumerate(KERNEL_CLASSES)}


# ---- single stages -----------------------------------------------------------------------------------------
def surelock_compact_scratch_bytes(total: int) -> int:
    return lib().surelock_compact_scratch_bytes(total)


def surelock_compact(lock_mask, B: int, N: int, active_idx, row_offsets, n_active, row_of_pos, scratch, dev_status=None):
    _check(lib().surelock_compact(_p(lock_mask), B, N, _p(active_idx), _p(row_offsets), _p(n_active), _p(row_of_pos),
                                  _p(scratch), _p(dev_status), _stream()), "surelock_compact")


def surelock_compact_from_ticket(lock_mask, B: int, N: int, active_idx, row_offsets, n_active, row_of_pos, scratch,
                                 first_ticket: int, dev_status=None):
    """Diagnostic: the compaction with its chunk tickets starting at `first_ticket` (see the header)."""
    _check(lib().surelock_compact_from_ticket(_p(lock_mask), B, N, _p(active_idx), _p(row_offsets), _p(n_active),
                                              _p(row_of_pos), _p(scratch), first_ticket, _p(dev_status), _stream()),
           "surelock_compact_from_ticket")


def surelock_compact_noalloc(lock_mask, B: int, N: int, active_idx, row_offsets, n_active, row_of_pos=None,
                             dev_status=None):
    """Compaction without caller scratch and without any device allocation (fixed in-library array; see the header
    for the capacity and the rule that calls sharing a GPU must not overlap)."""
    _check(lib().surelock_compact_noalloc(_p(lock_mask), B, N, _p(active_idx), _p(row_offsets), _p(n_active),
                                          _p(row_of_pos), _p(dev_status), _stream()), "surelock_compact_noalloc")


def surelock_compact_noalloc_max_flags() -> int:
    return lib().surelock_compact_noalloc_max_flags()


def surelock_kv_scatter(k, v, active_idx, n_active, k_cache, v_cache):
    _check(lib().surelock_kv_scatter(_p(k), _p(v), _p(active_idx), _p(n_active), k.shape[0], k[0].numel(), _p(k_cache),
                                     _p(v_cache), _dt(k), _stream()), "surelock_kv_scatter")


def surelock_softmax_kl_sure(logits, prev_logits, row_of_pos_prev, prev_lse, active_idx, n_active, mask_state,
                             lock_mask, kl_eps: float, kl, conf, argmax, lse_out=None):
    _check(lib().surelock_softmax_kl_sure(_p(logits), _p(prev_logits), _p(row_of_pos_prev), _p(prev_lse),
                                          _p(active_idx), _p(n_active), logits.shape[0], logits.shape[1], _dt(logits),
                                          _p(mask_state), _p(lock_mask), kl_eps, _p(kl), _p(conf), _p(argmax),
                                          _p(lse_out), _stream()), "surelock_softmax_kl_sure")


def surelock_gemm_workspace_bytes() -> int:
    return lib().surelock_gemm_workspace_bytes()


def surelock_gemm(A, W, Cout, n_active, impl: int = 0, dev_status=None, workspace=None):
    """workspace: zero-filled uint8 CUDA tensor of surelock_gemm_workspace_bytes() bytes (enables split-K), or None."""
    _check(lib().surelock_gemm(_p(A), _p(W), _p(Cout), _p(n_active), A.shape[0], W.shape[0], A.shape[1], _dt(A), impl,
                               _p(workspace), _p(dev_status), _stream()), "surelock_gemm")


def surelock_gemm_fused(A, W, W2, Cout, n_active, epilogue: int, impl: int = 0, dev_status=None, workspace=None):
    """epilogue 1: Cout (fp32) += A W^T; 2: Cout = silu(A W^T) * (A W2^T); 0: plain store."""
    _check(lib().surelock_gemm_fused(_p(A), _p(W), _p(W2), _p(Cout), _p(n_active), A.shape[0], W.shape[0], A.shape[1],
                                     _dt(A), epilogue, impl, _p(workspace), _p(dev_status), _stream()),
           "surelock_gemm_fused")


def surelock_attention_split_workspace_bytes(B: int, H: int, head_dim: int) -> int:
    return lib().surelock_attention_split_workspace_bytes(B, H, head_dim)


def surelock_attention_split(q, k_cache, v_cache, row_offsets, B: int, N: int, o, workspace, splits: int = 0,
                             diag_skip: int = -1, dev_status=None):
    H, dh = q.shape[1], q.shape[2]
    _check(lib().surelock_attention_split(_p(q), _p(k_cache), _p(v_cache), _p(row_offsets), q.shape[0], B, N, H, dh,
                                          splits, _p(o), _p(workspace), diag_skip, _p(dev_status), _stream()),
           "surelock_attention_split")


def surelock_attention(q, k_cache, v_cache, active_idx, row_offsets, n_active, B: int, N: int, o, impl: int = 0,
                       dev_status=None):
    H, dh = q.shape[1], q.shape[2]
    _check(lib().surelock_attention(_p(q), _p(k_cache), _p(v_cache), _p(active_idx), _p(row_offsets), _p(n_active),
                                    q.shape[0], B, N, H, dh, _p(o), _dt(q), impl, _p(dev_status), _stream()),
           "surelock_attention")
