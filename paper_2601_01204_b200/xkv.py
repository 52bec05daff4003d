"""ctypes binding of libxkv.so: same names as the C ABI, argument marshalling only.

Every step of the path runs in the library's CUDA kernels.  torch is used for
device memory (the workspace, the frame tensors) and for the current stream.
There is no CPU fallback: importing this module without a built library, or
calling it without a CUDA device, raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libxkv.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2601_01204_b200.build` "
        "(there is no CPU fallback)")

lib = C.CDLL(LIB_PATH)

XKV_OK, XKV_E_INVALID, XKV_E_STATE, XKV_E_NOMEM, XKV_E_UNSUPPORTED, XKV_E_CUDA, XKV_E_TIMEOUT = 0, -1, -2, -3, -4, -5, -6
XKV_E_LIMIT = -7
XKV_E_RANGE = -8
STATIC_SCRATCH_BYTES = 32 << 20
BUF_K_CODES, BUF_K_PARAMS, BUF_V_CODES, BUF_V_PARAMS, BUF_ORIGIN, BUF_SCORES, BUF_KEPT, BUF_QVEC = range(8)
BUF_K_SLOT, BUF_K_TABLE, BUF_K_REF = 8, 9, 10
KEYS_REGROUP, KEYS_ONCE = 0, 1

EXPORTED = [
    "xkv_workspace_bytes", "xkv_create", "xkv_reset", "xkv_destroy", "kv_append", "kv_score_evict",
    "kv_quant_pack", "attn_packed_causal", "xkv_stream_step", "xkv_stream_step_host_bytes",
    "xkv_stream_step_host", "xkv_get_info", "xkv_debug_export", "xkv_poll_status", "xkv_strerror",
    "xkv_synth_fill", "xkv_profile_enable", "xkv_profile_read", "attn_packed_causal_static",
    "xkv_debug_rewind_attention", "attn_packed_causal_tail", "xkv_set_unquantised_tail",
    "xkv_debug_force_plain", "xkv_debug_limit_attention_blocks", "xkv_debug_timeout_probe",
    "xkv_debug_head_means", "kv_score_evict_w", "xkv_set_budget", "xkv_read_score_stats",
    "attn_packed_frame_causal", "xkv_prefill_chunk",
]
PROF_NAMES = ["append", "score_evict", "pack", "kbar", "maint", "attn", "attn_combine"]


class xkv_params(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_heads", "head_dim", "n_special", "pool_g", "quant_group",
                                         "kv_bits", "budget", "max_frame_tokens", "key_mode", "key_table_slots")]


class xkv_info(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("frames", "T", "T_first", "rest_base", "T_phys", "capacity", "cur",
                                         "last_evicted", "last_kept", "last_prunable", "stage", "n_pending")] + \
               [("launches", C.c_int64), ("workspace_bytes", C.c_uint64), ("key_table_slots", C.c_int32),
                ("budget", C.c_int32)]


class xkv_score_stats(C.Structure):
    _fields_ = [("count", C.c_int32), ("kept", C.c_int32), ("sum", C.c_float), ("sum_sq", C.c_float),
                ("threshold", C.c_float)]


class xkv_profile(C.Structure):
    _fields_ = [("ms", C.c_double * 7), ("launches", C.c_int64 * 7)]


_vp, _i32, _i64, _sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
lib.xkv_profile_enable.restype = C.c_int
lib.xkv_profile_enable.argtypes = [_vp, C.c_int]
lib.xkv_profile_read.restype = C.c_int
lib.xkv_profile_read.argtypes = [_vp, C.POINTER(xkv_profile), _vp]
lib.xkv_workspace_bytes.restype = _sz
lib.xkv_workspace_bytes.argtypes = [C.POINTER(xkv_params)]
lib.xkv_create.restype = C.c_int
lib.xkv_create.argtypes = [C.POINTER(xkv_params), _vp, _sz, _vp, C.POINTER(_vp)]
lib.xkv_reset.restype = C.c_int
lib.xkv_reset.argtypes = [_vp, _vp]
lib.xkv_destroy.restype = C.c_int
lib.xkv_destroy.argtypes = [_vp]
lib.kv_append.restype = C.c_int
lib.kv_append.argtypes = [_vp, _vp, _vp, _i32, _i64, _i64, _vp]
lib.kv_score_evict.restype = C.c_int
lib.kv_score_evict.argtypes = [_vp, _vp, _i32, _i64, _i64, _vp]
lib.kv_score_evict_w.restype = C.c_int
lib.kv_score_evict_w.argtypes = [_vp, _vp, _i32, _vp]
lib.xkv_set_budget.restype = C.c_int
lib.xkv_set_budget.argtypes = [_vp, _i32]
lib.xkv_read_score_stats.restype = C.c_int
lib.xkv_read_score_stats.argtypes = [_vp, C.POINTER(xkv_score_stats), _vp]
lib.attn_packed_frame_causal.restype = C.c_int
lib.attn_packed_frame_causal.argtypes = [_vp, _vp, _vp, C.POINTER(_i32), _i32, _i64, _i64, C.c_float, _vp]
lib.xkv_prefill_chunk.restype = C.c_int
lib.xkv_prefill_chunk.argtypes = [_vp, _vp, _vp, _vp, _vp, C.POINTER(_i32), _i32, _i64, _i64, _vp]
lib.kv_quant_pack.restype = C.c_int
lib.kv_quant_pack.argtypes = [_vp, _vp]
lib.attn_packed_causal.restype = C.c_int
lib.attn_packed_causal.argtypes = [_vp, _vp, _vp, _i32, _i64, _i64, C.c_float, _i32, _vp]
lib.xkv_set_unquantised_tail.restype = C.c_int
lib.xkv_set_unquantised_tail.argtypes = [_vp, _i32]
lib.attn_packed_causal_tail.restype = C.c_int
lib.attn_packed_causal_tail.argtypes = [_vp, _vp, _vp, _vp, _vp, _i32, _i64, _i64, C.c_float, _vp]
lib.attn_packed_causal_static.restype = C.c_int
lib.attn_packed_causal_static.argtypes = [_vp, _vp, _vp, _i32, _i64, _i64, C.c_float, _vp]
lib.xkv_stream_step.restype = C.c_int
lib.xkv_stream_step.argtypes = [C.POINTER(_vp), _i32, C.POINTER(_vp), C.POINTER(_vp), C.POINTER(_vp),
                                C.POINTER(_vp), _i32, _i64, _i64, _vp]
lib.xkv_stream_step_host_bytes.restype = _sz
lib.xkv_stream_step_host_bytes.argtypes = [C.POINTER(xkv_params), _i32]
lib.xkv_stream_step_host.restype = C.c_int
lib.xkv_stream_step_host.argtypes = [C.POINTER(_vp), _i32, C.POINTER(_vp), C.POINTER(_vp), C.POINTER(_vp),
                                     C.POINTER(_vp), _i32, _vp, _sz, _vp]
lib.xkv_get_info.restype = C.c_int
lib.xkv_get_info.argtypes = [_vp, C.POINTER(xkv_info)]
lib.xkv_debug_export.restype = _i64
lib.xkv_debug_export.argtypes = [_vp, _i32, _vp, _sz, _vp]
lib.xkv_debug_rewind_attention.restype = C.c_int
lib.xkv_debug_rewind_attention.argtypes = [_vp]
lib.xkv_debug_force_plain.restype = C.c_int
lib.xkv_debug_force_plain.argtypes = [_vp, _i32]
lib.xkv_debug_limit_attention_blocks.restype = C.c_int
lib.xkv_debug_limit_attention_blocks.argtypes = [_vp, _i32]
lib.xkv_debug_head_means.restype = C.c_int
lib.xkv_debug_head_means.argtypes = [_vp, _vp]
lib.xkv_debug_timeout_probe.restype = C.c_int
lib.xkv_debug_timeout_probe.argtypes = [_vp, _vp]
lib.xkv_poll_status.restype = C.c_int
lib.xkv_poll_status.argtypes = [_vp, _vp]
lib.xkv_strerror.restype = C.c_char_p
lib.xkv_strerror.argtypes = [C.c_int]
lib.xkv_synth_fill.restype = C.c_int
lib.xkv_synth_fill.argtypes = [_vp, C.c_uint64, _i32, _i32, _i32, _vp, _i32, C.c_float, _vp]


class XkvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib.xkv_strerror(status).decode()} ({status})")


def _check(status: int, where: str) -> None:
    if status != XKV_OK:
        raise XkvError(status, where)


def _stream() -> int:
    import torch
    if not torch.cuda.is_available():
        raise RuntimeError("xkv needs a CUDA device; there is no CPU fallback")
    return torch.cuda.current_stream().cuda_stream


def _strides(t) -> tuple[int, int]:
    """(tok_stride, head_stride) in elements of a bf16 tensor viewed as [H][n][d]."""
    assert t.dim() == 3 and t.stride(2) == 1, "expect a [H][n][d] view with contiguous channels"
    return t.stride(1), t.stride(0)


@dataclass
class Params:
    n_heads: int = 16
    head_dim: int = 64
    n_special: int = 5
    pool_g: int = 16
    quant_group: int = 64
    kv_bits: int = 4
    budget: int = 2048
    max_frame_tokens: int = 1374
    key_mode: int = 0          # KEYS_REGROUP or KEYS_ONCE
    key_table_slots: int = 0   # KEYS_ONCE: 0 = one slot per token slot (never runs out)

    def c(self) -> xkv_params:
        return xkv_params(self.n_heads, self.head_dim, self.n_special, self.pool_g, self.quant_group,
                          self.kv_bits, self.budget, self.max_frame_tokens, self.key_mode, self.key_table_slots)


def xkv_workspace_bytes(p: Params) -> int:
    return int(lib.xkv_workspace_bytes(C.byref(p.c())))


class Cache:
    """One layer's cache: owns the torch workspace tensor and the C handle."""

    def __init__(self, p: Params, device: str = "cuda:0"):
        import torch
        self.p = p
        nbytes = xkv_workspace_bytes(p)
        if nbytes == 0:
            raise XkvError(XKV_E_INVALID, "xkv_workspace_bytes")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=device)
        self.handle = _vp()
        _check(lib.xkv_create(C.byref(p.c()), self.workspace.data_ptr(), nbytes, _stream(), C.byref(self.handle)),
               "xkv_create")

    def close(self) -> None:
        if self.handle:
            lib.xkv_destroy(self.handle)
            self.handle = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the C calls, same names ------------------------------------------
    def xkv_reset(self) -> None:
        _check(lib.xkv_reset(self.handle, _stream()), "xkv_reset")

    def kv_append(self, k, v) -> None:
        ts, hs = _strides(k)
        assert _strides(v) == (ts, hs)
        _check(lib.kv_append(self.handle, k.data_ptr(), v.data_ptr(), k.shape[1], ts, hs, _stream()), "kv_append")

    def kv_score_evict(self, q) -> None:
        ts, hs = _strides(q)
        _check(lib.kv_score_evict(self.handle, q.data_ptr(), q.shape[1], ts, hs, _stream()), "kv_score_evict")

    def kv_score_evict_w(self, w, n: int) -> None:
        """kv_score_evict with the pooled query's row mean w (device tensor, 64 fp32) from the caller."""
        _check(lib.kv_score_evict_w(self.handle, w.data_ptr(), n, _stream()), "kv_score_evict_w")

    def xkv_set_budget(self, budget: int) -> None:
        _check(lib.xkv_set_budget(self.handle, budget), "xkv_set_budget")

    def xkv_read_score_stats(self) -> xkv_score_stats:
        st = xkv_score_stats()
        _check(lib.xkv_read_score_stats(self.handle, C.byref(st), _stream()), "xkv_read_score_stats")
        return st

    def attn_packed_frame_causal(self, q, frame_tokens, out=None, scale: float | None = None):
        """Frame-causal attention of a chunk of frames (q, out: [H][sum(frame_tokens)][d])."""
        import torch
        if out is None:
            out = torch.empty_like(q)
        ts, hs = _strides(q)
        assert _strides(out) == (ts, hs)
        if scale is None:
            scale = 1.0 / float(np.sqrt(self.p.head_dim))
        ft = (_i32 * len(frame_tokens))(*frame_tokens)
        _check(lib.attn_packed_frame_causal(self.handle, q.data_ptr(), out.data_ptr(), ft, len(frame_tokens), ts, hs,
                                            C.c_float(scale), _stream()), "attn_packed_frame_causal")
        return out

    def xkv_prefill_chunk(self, q, k, v, frame_tokens, out=None):
        """A chunk of frames through append, scoring (last frame's query), packing and frame-causal attention."""
        import torch
        if out is None:
            out = torch.empty_like(q)
        ts, hs = _strides(q)
        assert _strides(out) == (ts, hs) and _strides(k) == (ts, hs) and _strides(v) == (ts, hs)
        ft = (_i32 * len(frame_tokens))(*frame_tokens)
        _check(lib.xkv_prefill_chunk(self.handle, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), ft,
                                     len(frame_tokens), ts, hs, _stream()), "xkv_prefill_chunk")
        return out

    def kv_quant_pack(self) -> None:
        _check(lib.kv_quant_pack(self.handle, _stream()), "kv_quant_pack")

    def attn_packed_causal(self, q, out=None, scale: float | None = None, impl: int = 0):
        import torch
        if out is None:
            out = torch.empty_like(q)
        ts, hs = _strides(q)
        assert _strides(out) == (ts, hs)
        if scale is None:
            scale = 1.0 / float(np.sqrt(self.p.head_dim))
        _check(lib.attn_packed_causal(self.handle, q.data_ptr(), out.data_ptr(), q.shape[1], ts, hs,
                                      C.c_float(scale), impl, _stream()), "attn_packed_causal")
        return out

    def xkv_set_unquantised_tail(self, on: bool) -> None:
        _check(lib.xkv_set_unquantised_tail(self.handle, 1 if on else 0), "xkv_set_unquantised_tail")

    def attn_packed_causal_tail(self, q, k_t, v_t, out=None, scale: float | None = None):
        """attn_packed_causal with the newest frame's keys and values taken unquantised from k_t, v_t
        (the tensors given to kv_append for this frame)."""
        import torch
        if out is None:
            out = torch.empty_like(q)
        ts, hs = _strides(q)
        assert _strides(out) == (ts, hs) and _strides(k_t) == (ts, hs) and _strides(v_t) == (ts, hs)
        if scale is None:
            scale = 1.0 / float(np.sqrt(self.p.head_dim))
        _check(lib.attn_packed_causal_tail(self.handle, q.data_ptr(), k_t.data_ptr(), v_t.data_ptr(), out.data_ptr(),
                                           q.shape[1], ts, hs, C.c_float(scale), _stream()),
               "attn_packed_causal_tail")
        return out

    def attn_packed_causal_static(self, q, out=None, scale: float | None = None):
        """attn_packed_causal with the partial results in the library's fixed device array
        (for callers that may not allocate; may run with fewer thread blocks than the GPU has
        multiprocessors)."""
        import torch
        if out is None:
            out = torch.empty_like(q)
        ts, hs = _strides(q)
        assert _strides(out) == (ts, hs)
        if scale is None:
            scale = 1.0 / float(np.sqrt(self.p.head_dim))
        _check(lib.attn_packed_causal_static(self.handle, q.data_ptr(), out.data_ptr(), q.shape[1], ts, hs,
                                             C.c_float(scale), _stream()), "attn_packed_causal_static")
        return out

    def step(self, q, k, v, out=None, impl: int = 0):
        self.kv_append(k, v)
        self.kv_score_evict(q)
        self.kv_quant_pack()
        return self.attn_packed_causal(q, out, impl=impl)

    def xkv_get_info(self) -> xkv_info:
        info = xkv_info()
        _check(lib.xkv_get_info(self.handle, C.byref(info)), "xkv_get_info")
        return info

    def xkv_profile_enable(self, on: bool) -> None:
        _check(lib.xkv_profile_enable(self.handle, 1 if on else 0), "xkv_profile_enable")

    def xkv_profile_read(self) -> dict:
        pr = xkv_profile()
        _check(lib.xkv_profile_read(self.handle, C.byref(pr), _stream()), "xkv_profile_read")
        return {name: (pr.ms[i], pr.launches[i]) for i, name in enumerate(PROF_NAMES)}

    def xkv_debug_rewind_attention(self) -> None:
        _check(lib.xkv_debug_rewind_attention(self.handle), "xkv_debug_rewind_attention")

    def xkv_debug_force_plain(self, on: bool) -> None:
        _check(lib.xkv_debug_force_plain(self.handle, 1 if on else 0), "xkv_debug_force_plain")

    def xkv_debug_limit_attention_blocks(self, max_blocks: int) -> None:
        _check(lib.xkv_debug_limit_attention_blocks(self.handle, max_blocks), "xkv_debug_limit_attention_blocks")

    def xkv_debug_head_means(self) -> None:
        _check(lib.xkv_debug_head_means(self.handle, _stream()), "xkv_debug_head_means")

    def xkv_debug_timeout_probe(self) -> None:
        _check(lib.xkv_debug_timeout_probe(self.handle, _stream()), "xkv_debug_timeout_probe")

    def xkv_poll_status(self) -> int:
        return int(lib.xkv_poll_status(self.handle, _stream()))

    def xkv_debug_export(self, which: int, nbytes: int) -> np.ndarray:
        buf = np.empty(max(nbytes, 1), dtype=np.uint8)
        got = lib.xkv_debug_export(self.handle, which, buf.ctypes.data, nbytes, _stream())
        if got < 0:
            raise XkvError(int(got), "xkv_debug_export")
        return buf[:got]

    # ---- test helper: logical-order view of the packed cache ----------------
    def export(self) -> dict:
        """The cache in logical token order, in the same form as the oracle's export()."""
        info = self.xkv_get_info()
        H, d, cap = self.p.n_heads, self.p.head_dim, info.capacity
        T, Tf, base = info.T, info.T_first, info.rest_base
        R = T - Tf
        sl = np.concatenate([np.arange(Tf), base + np.arange(R)]).astype(np.int64)
        out = {"T": T, "T_first": Tf}
        out["origin"] = self.xkv_debug_export(BUF_ORIGIN, cap * 4).view(np.int32)[sl].copy()
        if self.p.kv_bits == 16:
            k = self.xkv_debug_export(BUF_K_CODES, H * cap * d * 2).view(np.uint16).reshape(H, cap, d)
            v = self.xkv_debug_export(BUF_V_CODES, H * cap * d * 2).view(np.uint16).reshape(H, cap, d)
            out["k_val"] = (k[:, sl].astype(np.uint32) << 16).view(np.float32)
            out["v_val"] = (v[:, sl].astype(np.uint32) << 16).view(np.float32)
            return out
        rb = d // 2 if self.p.kv_bits == 4 else d          # bytes of a code row
        k = self.xkv_debug_export(BUF_K_CODES, H * cap * rb).reshape(H, cap, rb)
        v = self.xkv_debug_export(BUF_V_CODES, H * cap * rb).reshape(H, cap, rb)
        kp = self.xkv_debug_export(BUF_K_PARAMS, H * (cap // 64) * 64 * 8).view(np.float32).reshape(H, cap // 64, d, 2)
        vp = self.xkv_debug_export(BUF_V_PARAMS, H * cap * 8).view(np.float32).reshape(H, cap, 2)
        out["k_packed"], out["v_packed"] = k[:, sl].copy(), v[:, sl].copy()
        if self.p.key_mode == KEYS_ONCE:
            ns = info.key_table_slots
            slots = self.xkv_debug_export(BUF_K_SLOT, cap * 4).view(np.int32)[sl]
            tab = self.xkv_debug_export(BUF_K_TABLE, ns * H * d * 8).view(np.float32).reshape(ns, H, d, 2)
            ref = self.xkv_debug_export(BUF_K_REF, ns * 4).view(np.int32)
            out["k_s_tok"] = np.ascontiguousarray(tab[slots, :, :, 0].transpose(1, 0, 2))
            out["k_z_tok"] = np.ascontiguousarray(tab[slots, :, :, 1].transpose(1, 0, 2))
            out["k_groups_live"] = int((ref > 0).sum())
            # bookkeeping of the table: every slot's count is the number of cached tokens that refer to it
            assert np.array_equal(np.bincount(slots, minlength=ns), ref), "key table reference counts"
            out["v_s"], out["v_z"] = vp[:, sl, 0].copy(), vp[:, sl, 1].copy()
            return out
        ngf, ngr = (Tf + 63) // 64, (R + 63) // 64
        out["k_s_first"], out["k_z_first"] = kp[:, :ngf, :, 0].copy(), kp[:, :ngf, :, 1].copy()
        g0 = base // 64
        out["k_s_rest"], out["k_z_rest"] = kp[:, g0:g0 + ngr, :, 0].copy(), kp[:, g0:g0 + ngr, :, 1].copy()
        out["v_s"], out["v_z"] = vp[:, sl, 0].copy(), vp[:, sl, 1].copy()
        return out


def _ptr_array(tensors) -> "C.Array":
    arr = (_vp * len(tensors))()
    for i, t in enumerate(tensors):
        arr[i] = t if isinstance(t, int) else t.data_ptr()
    return arr


def xkv_stream_step(layers: list[Cache], q: list, k: list, v: list, out: list) -> None:
    """One frame through all layers; q/k/v/out are lists of [H][n][d] bf16 device tensors."""
    L = len(layers)
    ts, hs = _strides(q[0])
    handles = (_vp * L)(*[c.handle.value for c in layers])
    _check(lib.xkv_stream_step(handles, L, _ptr_array(q), _ptr_array(k), _ptr_array(v), _ptr_array(out),
                               q[0].shape[1], ts, hs, _stream()), "xkv_stream_step")


def xkv_stream_step_host(layers: list[Cache], q: list, k: list, v: list, out: list, staging) -> None:
    """Same with HOST tensors (contiguous [H][n][d] bf16, ideally pinned); synchronises."""
    L = len(layers)
    handles = (_vp * L)(*[c.handle.value for c in layers])
    _check(lib.xkv_stream_step_host(handles, L, _ptr_array(q), _ptr_array(k), _ptr_array(v), _ptr_array(out),
                                    q[0].shape[1], staging.data_ptr(), staging.numel() * staging.element_size(),
                                    _stream()), "xkv_stream_step_host")


def xkv_stream_step_host_bytes(p: Params, n: int) -> int:
    return int(lib.xkv_stream_step_host_bytes(C.byref(p.c()), n))


def xkv_synth_fill(dst, seed: int, layer: int, frame: int, tensor: int) -> None:
    """Fill dst (bf16 [H][n][d], device) with the seeded inputs of `synth` for one tensor."""
    from . import synth
    H, n, d = dst.shape
    assert dst.is_contiguous()
    key = synth.tensor_key(seed, layer, frame, tensor)
    if tensor == synth.TENSOR_K:
        oc = np.ascontiguousarray(synth.outlier_channels(seed, layer, H, d), dtype=np.int32)
        _check(lib.xkv_synth_fill(dst.data_ptr(), key, H, n, d, oc.ctypes.data, oc.shape[1],
                                  C.c_float(synth.OUTLIER_GAIN), _stream()), "xkv_synth_fill")
    else:
        _check(lib.xkv_synth_fill(dst.data_ptr(), key, H, n, d, None, 0, C.c_float(1.0), _stream()),
               "xkv_synth_fill")
