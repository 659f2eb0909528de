"""ctypes binding of libbpc.so.  Argument marshalling only: every step of the path runs in the CUDA library.

PyTorch supplies device memory and streams; tensors are passed as raw device pointers.  Importing this
module loads the shared library and raises if it is missing (there is no fallback path).
"""
from __future__ import annotations

import ctypes
import math
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbpc.so")

BPC_OK = 0
STATUS_NAMES = {0: "BPC_OK", 1: "BPC_ERR_INVALID_ARG", 2: "BPC_ERR_UNSUPPORTED", 3: "BPC_ERR_CAPACITY",
                4: "BPC_ERR_NOT_FITTED", 5: "BPC_ERR_CUDA", 6: "BPC_ERR_DEVICE", 7: "BPC_ERR_SCRATCH_LIMIT"}
BPC_BF16, BPC_F32 = 0, 1
BPC_SCORE_HAMMING, BPC_SCORE_WEIGHTED7 = 0, 1


class BpcError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__("%s failed: %s" % (what, STATUS_NAMES.get(status, str(status))))
        self.status = status


class bpc_config(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("code_bits", ctypes.c_int32), ("n_max", ctypes.c_int32),
                ("kv_dtype", ctypes.c_int32), ("score_mode", ctypes.c_int32), ("sm_scale", ctypes.c_float),
                ("hash_sets", ctypes.c_int32), ("residual_correction", ctypes.c_int32), ("kv_row_stride", ctypes.c_int32), ("eas_ppm", ctypes.c_int32),
                ("fit_power_iters", ctypes.c_int32)]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError("libbpc.so is not built (run `python -m paper_2608_04405_b200.build`): %s" % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    cfgp = ctypes.POINTER(bpc_config)
    sig = {
        "bpc_create": (i32, [cfgp, ctypes.POINTER(vp)]),
        "bpc_destroy": (i32, [vp]),
        "bpc_codes_bytes": (sz, [cfgp]),
        "bpc_fit_workspace_bytes": (sz, [cfgp]),
        "bpc_fit_codes_offset": (sz, [cfgp]),
        "bpc_max_context": (i64, [cfgp]),
        "bpc_set_seq_lens": (i32, [vp, ctypes.POINTER(i32), vp]),
        "bpc_get_seq_lens": (i32, [vp, ctypes.POINTER(i32)]),
        "bpc_fit": (i32, [vp, vp, vp, vp, sz, vp]),
        "bpc_set_projection": (i32, [vp, vp, vp]),
        "bpc_get_projection": (i32, [vp, vp, vp, vp, vp]),
        "bpc_encode_keys": (i32, [vp, vp, vp, vp]),
        "bpc_build_eas": (i32, [vp, vp]),
        "bpc_get_eas": (i32, [vp, vp, vp, vp, vp]),
        "bpc_eas_capacity": (i32, [cfgp]),
        "bpc_exact_topk": (i32, [vp, vp, vp, i32, i32, vp, vp, vp, vp]),
        "bpc_append": (i32, [vp, vp, vp, vp, vp, vp, vp]),
        "bpc_decode_attn": (i32, [vp, vp, vp, vp, vp, i32, i32, vp, vp, vp]),
        "bpc_append_decode_attn": (i32, [vp, vp, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp]),
        "bpc_decode_attn_static": (i32, [cfgp, vp, vp, vp, vp, vp, vp, i32, i32, vp, vp]),
        "bpc_static_scratch_entries": (sz, []),
        "bpc_static_last_device_error": (i32, [ctypes.POINTER(i32), vp]),
        "bpc_debug_set_buffers": (i32, [vp, vp, vp]),
        "bpc_debug_set_phase_timer": (i32, [vp, vp]),
        "bpc_set_cluster_size": (i32, [vp, i32]),
        "bpc_plan_cluster_size": (i32, [cfgp, ctypes.POINTER(i32), i32]),
        "bpc_get_cluster_size": (i32, [vp]),
        "bpc_uses_streaming": (i32, [vp]),
        "bpc_status_of_device_error": (i32, [i32]),
        "bpc_debug_set_pdl": (i32, [vp, i32]),
        "bpc_debug_force_key_shift": (i32, [vp, i32]),
        "bpc_debug_set_tensor_core_encode": (i32, [vp, i32]),
        "bpc_debug_force_streaming": (i32, [vp, i32]),
        "bpc_debug_force_byte_keys": (i32, [vp, i32]),
        "bpc_uses_byte_keys": (i32, [vp]),
        "bpc_uses_work_items": (i32, [vp]),
        "bpc_work_item_grid": (i32, [vp]),
        "bpc_debug_set_decode_path": (i32, [vp, i32]),
        "bpc_debug_set_work_item_geometry": (i32, [vp, i32, i32]),
        "bpc_debug_set_work_item_trace": (i32, [vp, vp]),
        "bpc_last_device_error": (i32, [vp, ctypes.POINTER(i32), vp]),
        "bpc_last_cuda_error": (i32, [vp]),
        "bpc_launch_count": (i64, [vp]),
        "bpc_version": (ctypes.c_char_p, []),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    return lib


lib = _load()
EXPORTS = ["bpc_create", "bpc_destroy", "bpc_codes_bytes", "bpc_fit_workspace_bytes", "bpc_fit_codes_offset",
           "bpc_max_context",
           "bpc_set_seq_lens", "bpc_get_seq_lens", "bpc_fit", "bpc_set_projection", "bpc_get_projection",
           "bpc_encode_keys", "bpc_build_eas", "bpc_get_eas", "bpc_eas_capacity", "bpc_exact_topk", "bpc_append", "bpc_decode_attn", "bpc_append_decode_attn", "bpc_decode_attn_static", "bpc_static_scratch_entries", "bpc_static_last_device_error",
           "bpc_debug_set_buffers", "bpc_debug_set_phase_timer",
           "bpc_set_cluster_size", "bpc_plan_cluster_size",
           "bpc_get_cluster_size", "bpc_uses_streaming", "bpc_status_of_device_error", "bpc_debug_set_pdl", "bpc_debug_force_key_shift",
           "bpc_debug_set_tensor_core_encode", "bpc_debug_force_streaming", "bpc_debug_force_byte_keys", "bpc_uses_byte_keys", "bpc_uses_work_items", "bpc_work_item_grid", "bpc_debug_set_decode_path",
           "bpc_debug_set_work_item_geometry", "bpc_debug_set_work_item_trace", "bpc_last_device_error", "bpc_last_cuda_error", "bpc_launch_count", "bpc_version"]


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous(), "tensor must be contiguous"
    return t.data_ptr()


def _cache_ptr(t: torch.Tensor) -> int:
    """K/V caches may be strided views of one interleaved buffer: rows must be dense, the row stride is in the config."""
    assert t.stride(-1) == 1, "cache rows must be dense"
    return t.data_ptr()


def interleaved_kv(batch: int, n_kv_heads: int, n_max: int, head_dim: int, dtype: torch.dtype, device="cuda"):
    """One buffer [batch][n_kv_heads][n_max][2][head_dim]; returns (buffer, k_view, v_view) for kv_row_stride = 2*head_dim."""
    buf = torch.zeros(batch, n_kv_heads, n_max, 2, head_dim, dtype=dtype, device=device)
    return buf, buf[:, :, :, 0, :], buf[:, :, :, 1, :]


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(status: int, what: str) -> None:
    if status != BPC_OK:
        raise BpcError(status, what)


def make_config(batch: int, n_q_heads: int, n_kv_heads: int, n_max: int, code_bits: int, dtype: torch.dtype,
                score_mode: int = BPC_SCORE_HAMMING, sm_scale: float = 0.0, shared_projection: bool = False,
                residual_correction: bool = True, head_dim: int = 128, kv_row_stride: int = 0,
                eas_ppm: int = 0, fit_power_iters: int = 0) -> bpc_config:
    return bpc_config(batch, n_q_heads, n_kv_heads, head_dim, code_bits, n_max,
                      BPC_BF16 if dtype == torch.bfloat16 else BPC_F32, score_mode, sm_scale,
                      n_kv_heads if shared_projection else batch * n_kv_heads, 1 if residual_correction else 0, kv_row_stride, eas_ppm, fit_power_iters)


def plan_cluster_size(cfg: bpc_config, max_active, chunk_cap: int) -> int:
    """bpc_plan_cluster_size: the automatic cluster size for `cfg` on a device with the given limits (max_active[c] =
    resident clusters of c blocks, c = 1 .. 16; entry 0 ignored).  Pure host arithmetic."""
    arr = (ctypes.c_int32 * 17)(*[int(v) for v in max_active])
    return int(lib.bpc_plan_cluster_size(ctypes.byref(cfg), arr, int(chunk_cap)))


class Context:
    """Owns one bpc_ctx.  Methods carry the C entry points' names without the prefix."""

    def __init__(self, cfg: bpc_config):
        self.cfg = cfg
        self.units = cfg.batch * cfg.n_kv_heads
        self.dtype = torch.bfloat16 if cfg.kv_dtype == BPC_BF16 else torch.float32
        h = ctypes.c_void_p()
        _check(lib.bpc_create(ctypes.byref(cfg), ctypes.byref(h)), "bpc_create")
        self._h = h
        self._dbg = None

    def close(self) -> None:
        if getattr(self, "_h", None):
            lib.bpc_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- sizes
    def codes_bytes(self) -> int:
        return lib.bpc_codes_bytes(ctypes.byref(self.cfg))

    def alloc_codes(self, device="cuda") -> torch.Tensor:
        c = self.cfg
        if c.code_bits == 32:            # half a 64-bit word per key: one int32
            return torch.zeros(c.batch, c.n_kv_heads, c.n_max, 1, dtype=torch.int32, device=device)
        return torch.zeros(c.batch, c.n_kv_heads, c.n_max, c.code_bits // 64, dtype=torch.int64, device=device)

    def fit_workspace_bytes(self) -> int:
        return lib.bpc_fit_workspace_bytes(ctypes.byref(self.cfg))

    def fit_codes_offset(self) -> int:
        return lib.bpc_fit_codes_offset(ctypes.byref(self.cfg))

    def max_context(self) -> int:
        return lib.bpc_max_context(ctypes.byref(self.cfg))

    # -- state
    def set_seq_lens(self, lens: Sequence[int]) -> None:
        arr = (ctypes.c_int32 * self.cfg.batch)(*[int(v) for v in lens])
        _check(lib.bpc_set_seq_lens(self._h, arr, _stream()), "bpc_set_seq_lens")

    def get_seq_lens(self):
        arr = (ctypes.c_int32 * self.cfg.batch)()
        _check(lib.bpc_get_seq_lens(self._h, arr), "bpc_get_seq_lens")
        return list(arr)

    def set_cluster_size(self, cs: int) -> None:
        _check(lib.bpc_set_cluster_size(self._h, cs), "bpc_set_cluster_size")

    def get_cluster_size(self) -> int:
        return lib.bpc_get_cluster_size(self._h)

    # -- hot path
    def fit(self, k_cache: torch.Tensor, v_star: torch.Tensor, workspace: Optional[torch.Tensor] = None) -> None:
        if workspace is None:
            workspace = torch.empty(self.fit_workspace_bytes(), dtype=torch.uint8, device=k_cache.device)
        _check(lib.bpc_fit(self._h, _cache_ptr(k_cache), _ptr(v_star), _ptr(workspace), workspace.numel(), _stream()), "bpc_fit")

    def set_projection(self, P: torch.Tensor) -> None:
        assert P.dtype == torch.float32
        _check(lib.bpc_set_projection(self._h, _ptr(P), _stream()), "bpc_set_projection")

    def get_projection(self):
        c = self.cfg
        P = torch.empty(c.hash_sets, c.code_bits, c.head_dim, dtype=torch.float32, device="cuda")
        Ph = torch.empty_like(P)
        gram = torch.empty(c.hash_sets, c.code_bits, c.code_bits, dtype=torch.float32, device="cuda")
        _check(lib.bpc_get_projection(self._h, _ptr(P), _ptr(Ph), _ptr(gram), _stream()), "bpc_get_projection")
        return P, Ph, gram

    def encode_keys(self, k_cache: torch.Tensor, codes: torch.Tensor) -> None:
        _check(lib.bpc_encode_keys(self._h, _cache_ptr(k_cache), _ptr(codes), _stream()), "bpc_encode_keys")

    def build_eas(self) -> None:
        _check(lib.bpc_build_eas(self._h, _stream()), "bpc_build_eas")

    def exact_topk(self, q, k_cache, budget_ppm: int = 20000, budget_count: int = 0):
        """Quality yard-stick: exact scores of every cached key for every query head and the per-head top-k.
        Returns (scores [batch*n_q_heads, n_max] float32, sel [batch*n_q_heads, n_max] int32, count [batch*n_q_heads] int32)."""
        c = self.cfg
        heads = c.batch * c.n_q_heads
        scores = torch.zeros(heads, c.n_max, dtype=torch.float32, device=q.device)
        sel = torch.full((heads, c.n_max), -1, dtype=torch.int32, device=q.device)
        cnt = torch.zeros(heads, dtype=torch.int32, device=q.device)
        _check(lib.bpc_exact_topk(self._h, _ptr(q), _cache_ptr(k_cache), budget_ppm, budget_count, _ptr(scores), _ptr(sel),
                                  _ptr(cnt), _stream()), "bpc_exact_topk")
        return scores, sel, cnt

    def get_eas(self):
        c = self.cfg
        cap = lib.bpc_eas_capacity(ctypes.byref(c))
        err = torch.empty(self.units, c.n_max, dtype=torch.float32, device="cuda")
        idx = torch.empty(self.units, max(cap, 1), dtype=torch.int32, device="cuda")
        cnt = torch.empty(self.units, dtype=torch.int32, device="cuda")
        _check(lib.bpc_get_eas(self._h, _ptr(err), _ptr(idx), _ptr(cnt), _stream()), "bpc_get_eas")
        return err, idx, cnt

    def append(self, k_new, v_new, k_cache, v_cache, codes) -> None:
        _check(lib.bpc_append(self._h, _ptr(k_new), _ptr(v_new), _cache_ptr(k_cache), _cache_ptr(v_cache), _ptr(codes), _stream()),
               "bpc_append")

    def decode_attn(self, q, k_cache, v_cache, codes, budget_ppm: int = 20000, budget_count: int = 0,
                    out: Optional[torch.Tensor] = None, sel_idx: Optional[torch.Tensor] = None) -> torch.Tensor:
        c = self.cfg
        if out is None:
            out = torch.empty(c.batch, c.n_q_heads, c.head_dim, dtype=torch.float32, device=q.device)
        _check(lib.bpc_decode_attn(self._h, _ptr(q), _cache_ptr(k_cache), _cache_ptr(v_cache), _ptr(codes), budget_ppm, budget_count,
                                   _ptr(out), _ptr(sel_idx), _stream()), "bpc_decode_attn")
        return out

    def append_decode_attn(self, k_new, v_new, k_cache, v_cache, codes, q, budget_ppm: int = 20000, budget_count: int = 0,
                           out: Optional[torch.Tensor] = None, sel_idx: Optional[torch.Tensor] = None) -> torch.Tensor:
        c = self.cfg
        if out is None:
            out = torch.empty(c.batch, c.n_q_heads, c.head_dim, dtype=torch.float32, device=q.device)
        _check(lib.bpc_append_decode_attn(self._h, _ptr(k_new), _ptr(v_new), _cache_ptr(k_cache), _cache_ptr(v_cache),
                                          _ptr(codes), _ptr(q), budget_ppm, budget_count, _ptr(out), _ptr(sel_idx), _stream()),
               "bpc_append_decode_attn")
        return out

    # -- parity aids and diagnostics
    def debug_set_buffers(self, scores: Optional[torch.Tensor], qweights: Optional[torch.Tensor]) -> None:
        self._dbg = (scores, qweights)   # keep alive
        _check(lib.bpc_debug_set_buffers(self._h, _ptr(scores), _ptr(qweights)), "bpc_debug_set_buffers")

    def debug_set_phase_timer(self, stamps: Optional[torch.Tensor]) -> None:
        self._stamps = stamps
        _check(lib.bpc_debug_set_phase_timer(self._h, _ptr(stamps)), "bpc_debug_set_phase_timer")

    def uses_streaming(self) -> bool:
        return bool(lib.bpc_uses_streaming(self._h))

    def uses_work_items(self) -> bool:
        return bool(lib.bpc_uses_work_items(self._h))

    def work_item_grid(self) -> int:
        return lib.bpc_work_item_grid(self._h)

    def debug_set_decode_path(self, path: int) -> None:
        """0 = the library chooses, 1 = cluster kernel, 2 = work-item kernel."""
        _check(lib.bpc_debug_set_decode_path(self._h, path), "bpc_debug_set_decode_path")

    def debug_set_work_item_geometry(self, keys_per_scan_item: int = 0, rows_per_attend_item: int = 0) -> None:
        _check(lib.bpc_debug_set_work_item_geometry(self._h, keys_per_scan_item, rows_per_attend_item),
               "bpc_debug_set_work_item_geometry")

    def debug_set_work_item_trace(self, trace: Optional[torch.Tensor]) -> None:
        self._trace = trace
        _check(lib.bpc_debug_set_work_item_trace(self._h, _ptr(trace)), "bpc_debug_set_work_item_trace")

    def last_device_error(self) -> int:
        """The device error word (0 = none).  The C call returns BPC_ERR_DEVICE for a non-zero word; here the word itself
        is the result."""
        v = ctypes.c_int32(0)
        st = lib.bpc_last_device_error(self._h, ctypes.byref(v), _stream())
        if st not in (BPC_OK, 6):
            raise BpcError(st, "bpc_last_device_error")
        assert (st == 6) == (v.value != 0)
        return v.value

    def debug_set_pdl(self, on: bool) -> None:
        _check(lib.bpc_debug_set_pdl(self._h, 1 if on else 0), "bpc_debug_set_pdl")

    def debug_force_key_shift(self, shift: int) -> None:
        _check(lib.bpc_debug_force_key_shift(self._h, shift), "bpc_debug_force_key_shift")

    def debug_set_tensor_core_encode(self, on: bool) -> None:
        """False: bpc_encode_keys and the passes of bpc_fit run their CUDA-core kernels (cross-checks)."""
        _check(lib.bpc_debug_set_tensor_core_encode(self._h, 1 if on else 0), "bpc_debug_set_tensor_core_encode")

    def uses_byte_keys(self) -> bool:
        return bool(lib.bpc_uses_byte_keys(self._h))

    def debug_force_byte_keys(self, mode: int) -> None:
        """1 = byte score keys wherever possible, -1 = never, 0 = the library decides."""
        _check(lib.bpc_debug_force_byte_keys(self._h, mode), "bpc_debug_force_byte_keys")

    def debug_force_streaming(self, on: bool) -> None:
        _check(lib.bpc_debug_force_streaming(self._h, 1 if on else 0), "bpc_debug_force_streaming")

    def last_cuda_error(self) -> int:
        return lib.bpc_last_cuda_error(self._h)

    def launch_count(self) -> int:
        return lib.bpc_launch_count(self._h)


def bpc_decode_attn(ctx: Context, q, k_cache, v_cache, codes, budget) -> torch.Tensor:
    """Functional form of one decode step: budget is a fraction in (0, 1] or an integer key count."""
    if isinstance(budget, float):
        return ctx.decode_attn(q, k_cache, v_cache, codes, budget_ppm=int(round(budget * 1e6)))
    return ctx.decode_attn(q, k_cache, v_cache, codes, budget_ppm=0, budget_count=int(budget))


def bpc_decode_attn_static(cfg: bpc_config, q, k_cache, v_cache, codes, P_hash, unit_lens, budget_ppm: int = 20000,
                           budget_count: int = 0, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Decode step without a context and without any allocation inside the library (see bpc.h).  P_hash is the hash
    projection in the cache dtype, unit_lens an int32 device tensor with one length per (sequence, KV head)."""
    if out is None:
        out = torch.empty(cfg.batch, cfg.n_q_heads, cfg.head_dim, dtype=torch.float32, device=q.device)
    assert unit_lens.dtype == torch.int32
    _check(lib.bpc_decode_attn_static(ctypes.byref(cfg), _ptr(q), _cache_ptr(k_cache), _cache_ptr(v_cache), _ptr(codes),
                                      _ptr(P_hash), _ptr(unit_lens), budget_ppm, budget_count, _ptr(out), _stream()),
           "bpc_decode_attn_static")
    return out


def bpc_static_last_device_error() -> int:
    """Error word left by the last bpc_decode_attn_static call on the current device (0 = none)."""
    v = ctypes.c_int32(0)
    st = lib.bpc_static_last_device_error(ctypes.byref(v), _stream())
    if st not in (BPC_OK, 6):
        raise BpcError(st, "bpc_static_last_device_error")
    return v.value


def bpc_fit(ctx: Context, k_cache, v_star, workspace=None) -> None:
    ctx.fit(k_cache, v_star, workspace)


def bpc_encode_keys(ctx: Context, k_cache, codes) -> None:
    ctx.encode_keys(k_cache, codes)


def bpc_append(ctx: Context, k_new, v_new, k_cache, v_cache, codes) -> None:
    ctx.append(k_new, v_new, k_cache, v_cache, codes)
