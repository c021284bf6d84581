"""Thin ctypes binding of ``libmvla_prune.so`` (see ``include/mvla_prune.h``).

Argument marshalling only: every step of the prune path runs in the CUDA
library.  PyTorch supplies device memory and streams.  There is no CPU
fallback: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libmvla_prune.so")

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_OOM, ERR_CUDA = -1, -2, -3, -4
ERR_CAPACITY, ERR_TIMEOUT, ERR_STATE = -5, -6, -7
_ERR_NAMES = {-1: "MVLA_ERR_INVALID_ARG", -2: "MVLA_ERR_UNSUPPORTED", -3: "MVLA_ERR_OOM",
              -4: "MVLA_ERR_CUDA", -5: "MVLA_ERR_CAPACITY", -6: "MVLA_ERR_TIMEOUT",
              -7: "MVLA_ERR_STATE"}
DTYPE_BF16, DTYPE_FP32, DTYPE_FP8_E4M3 = 0, 1, 2
MODE_FIXED, MODE_ADAPTIVE, MODE_PATCH = 0, 1, 2
LABEL_BG, LABEL_ROB, LABEL_OBJ = 0, 1, 2
FLAG_RESET_STATE, FLAG_NO_STATE_UPDATE, FLAG_INPUTS_STABLE = 1, 2, 4
SALIENCE_AUTO, SALIENCE_FMA = 0, 1
SET_2D, SET_3D = 1, 2

EXPORTS = ("mvla_prune_create", "mvla_salience", "mvla_select", "mvla_compact",
           "mvla_prune_step", "mvla_prune_destroy", "mvla_patch_indicators", "mvla_patch_select",
           "mvla_salience_noalloc", "mvla_selftest_wait_timeout", "mvla_set_stage_event", "mvla_set_kernel_stamps",
           "mvla_logit_cache_stats")


class MvlaError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where} failed: {_ERR_NAMES.get(code, code)}")


class Config(C.Structure):
    _fields_ = [("device", C.c_int32), ("dtype", C.c_int32), ("n_heads", C.c_int32),
                ("head_dim", C.c_int32), ("d_model", C.c_int32), ("max_batch", C.c_int32),
                ("max_text", C.c_int32), ("max_2d", C.c_int32), ("max_3d", C.c_int32),
                ("n_prune_points", C.c_int32), ("n_state_slots", C.c_int32),
                ("window_k", C.c_int32), ("cold_start_full_keep", C.c_int32),
                ("salience_path", C.c_int32),
                ("tau_2d", C.c_double), ("tau_3d", C.c_double), ("beta", C.c_double),
                ("eps_3d", C.c_double), ("floor_ratio", C.c_double), ("obj_2d_min", C.c_double),
                ("patch_path", C.c_int32), ("kmeans_max_iter", C.c_int32), ("n_kv_heads", C.c_int32),
                ("logit_cache", C.c_int32), ("reserved0", C.c_int32)]


class CSample(C.Structure):
    _fields_ = [("seq_off", C.c_int32), ("off_txt", C.c_int32), ("n_txt", C.c_int32),
                ("off_2d", C.c_int32), ("n_2d", C.c_int32), ("off_3d", C.c_int32),
                ("n_3d", C.c_int32), ("state_slot", C.c_int32),
                ("keep_2d", C.c_double), ("keep_3d", C.c_double), ("keep_total", C.c_double)]


class CDiag(C.Structure):
    _fields_ = [("t", C.c_int32), ("c_s1", C.c_int32), ("c_s2", C.c_int32), ("c_final", C.c_int32),
                ("budget", C.c_int32), ("k_2d", C.c_int32), ("k_3d", C.c_int32),
                ("reserved", C.c_int32), ("x", C.c_float * 4), ("mhat", C.c_float * 4)]


class CTensors(C.Structure):
    _fields_ = [("q", C.c_void_p), ("k", C.c_void_p), ("v", C.c_void_p), ("hidden", C.c_void_p),
                ("rows", C.c_int64), ("rand_u", C.c_void_p), ("changed_rows", C.c_void_p)]


class COutputs(C.Structure):
    _fields_ = [("out_hidden", C.c_void_p), ("out_k", C.c_void_p), ("out_v", C.c_void_p),
                ("kept_idx", C.c_void_p), ("out_offsets", C.c_void_p), ("budgets", C.c_void_p),
                ("attn", C.c_void_p), ("ahat", C.c_void_p), ("z", C.c_void_p), ("diag", C.c_void_p),
                ("patch_x", C.c_void_p), ("patch_xhat", C.c_void_p), ("patch_info", C.c_void_p),
                ("patch_diag", C.c_void_p)]


class CPatchDiag(C.Structure):
    _fields_ = [("t", C.c_int32), ("iters", C.c_int32), ("n_label", C.c_int32 * 3), ("k_2d", C.c_int32),
                ("k_3d", C.c_int32), ("n_out", C.c_int32), ("centre", C.c_float * 3), ("mu_2d", C.c_float),
                ("mu_3d", C.c_float), ("reserved", C.c_float * 3)]


def load_library(path: str = LIB_PATH) -> C.CDLL:
    if not os.path.exists(path):
        raise OSError(f"{path} is missing: build it with `python -m paper_2604_09244_b200.build` "
                      "(there is no fallback path)")
    lib = C.CDLL(path)
    vp, i32, u32, i64 = C.c_void_p, C.c_int32, C.c_uint32, C.c_int64
    sp = C.POINTER(CSample)
    lib.mvla_prune_create.argtypes = [C.POINTER(Config), C.POINTER(vp)]
    lib.mvla_prune_create.restype = i32
    lib.mvla_salience.argtypes = [vp, i32, sp, vp, vp, vp, i64, vp, vp, vp]
    lib.mvla_salience.restype = i32
    lib.mvla_select.argtypes = [vp, i32, i32, sp, i32, u32, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.mvla_select.restype = i32
    lib.mvla_compact.argtypes = [vp, i32, sp, vp, vp, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.mvla_compact.restype = i32
    lib.mvla_prune_step.argtypes = [vp, i32, i32, sp, i32, u32, C.POINTER(CTensors),
                                    C.POINTER(COutputs), C.POINTER(i32), vp]
    lib.mvla_prune_step.restype = i32
    lib.mvla_prune_destroy.argtypes = [vp]
    lib.mvla_prune_destroy.restype = None
    lib.mvla_patch_indicators.argtypes = [vp, i32, sp, vp, vp, vp, i64, vp, vp, vp]
    lib.mvla_patch_indicators.restype = i32
    lib.mvla_patch_select.argtypes = [vp, i32, i32, sp, u32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.mvla_patch_select.restype = i32
    lib.mvla_logit_cache_stats.argtypes = [vp, C.POINTER(i64), C.POINTER(i64)]
    lib.mvla_logit_cache_stats.restype = i32
    lib.mvla_set_kernel_stamps.argtypes = [vp, vp]
    lib.mvla_set_kernel_stamps.restype = i32
    lib.mvla_set_stage_event.argtypes = [vp, vp]
    lib.mvla_set_stage_event.restype = i32
    lib.mvla_selftest_wait_timeout.argtypes = [vp, u32, vp]
    lib.mvla_selftest_wait_timeout.restype = i32
    return lib


_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = load_library()
    return _lib


def c_samples(samples: Sequence) -> "C.Array[CSample]":
    """From objects with the descriptor's field names (``workloads.Sample``)."""
    arr = (CSample * len(samples))()
    for i, s in enumerate(samples):
        arr[i] = CSample(int(s.seq_off), int(s.off_txt), int(s.n_txt), int(s.off_2d), int(s.n_2d),
                         int(s.off_3d), int(s.n_3d), int(getattr(s, "state_slot", 0)),
                         float(s.keep_2d), float(s.keep_3d), float(s.keep_total))
    return arr


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device-resident contiguous tensors only"
    return t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


@dataclass
class StepOutputs:
    """Caller-owned device buffers of one fused step (sized for the worst case)."""
    out_hidden: Optional[torch.Tensor]
    out_k: Optional[torch.Tensor]
    out_v: Optional[torch.Tensor]
    kept_idx: torch.Tensor
    out_offsets: torch.Tensor
    budgets: torch.Tensor
    attn: Optional[torch.Tensor] = None
    ahat: Optional[torch.Tensor] = None
    z: Optional[torch.Tensor] = None
    diag: Optional[torch.Tensor] = None   # int32 view of mvla_diag records, [batch, 16]
    total_kept: int = 0
    # patch-by-patch path
    patch_x: Optional[torch.Tensor] = None      # [sum P, 4]
    patch_xhat: Optional[torch.Tensor] = None   # [sum P, 4]
    patch_info: Optional[torch.Tensor] = None   # [sum P] int32
    patch_diag: Optional[torch.Tensor] = None   # int32 view of mvla_patch_diag records, [batch, 16]


class PruneContext:
    """Owns one ``mvla_ctx``."""

    def __init__(self, *, dtype: torch.dtype, n_heads: int, head_dim: int, d_model: int,
                 max_batch: int, max_text: int, max_2d: int, max_3d: int, n_prune_points: int = 1,
                 n_state_slots: int = 0, tau_2d: float = 0.08, tau_3d: float = 0.20,
                 beta: float = 0.85, window_k: int = 7, eps_3d: float = 0.02,
                 floor_ratio: float = 0.10, cold_start_full_keep: int = 1,
                 salience_path: int = SALIENCE_AUTO, device: Optional[int] = None, patch_path: int = 0,
                 obj_2d_min: float = 0.5, kmeans_max_iter: int = 32, n_kv_heads: int = 0, logit_cache: int = 0):
        self._h = C.c_void_p()
        self._lib = lib()
        if device is None:
            device = torch.cuda.current_device()
        self.device = torch.device("cuda", device)
        self.torch_dtype = dtype
        code = {torch.bfloat16: DTYPE_BF16, torch.float32: DTYPE_FP32, torch.float8_e4m3fn: DTYPE_FP8_E4M3}[dtype]
        self.hidden_dtype = torch.bfloat16 if dtype == torch.float8_e4m3fn else dtype   # e4m3 is for q, k, v only
        self.cfg = Config(device, code, n_heads, head_dim, d_model, max_batch, max_text, max_2d,
                          max_3d, n_prune_points, n_state_slots, window_k, cold_start_full_keep,
                          salience_path, tau_2d, tau_3d, beta, eps_3d, floor_ratio, obj_2d_min, patch_path,
                          kmeans_max_iter, n_kv_heads, logit_cache, 0)
        rc = self._lib.mvla_prune_create(C.byref(self.cfg), C.byref(self._h))
        if rc != OK:
            self._h = C.c_void_p()
            raise MvlaError(rc, "mvla_prune_create")

    def close(self):
        if getattr(self, "_h", None) is not None and self._h:
            torch.cuda.synchronize(self.device)
            self._lib.mvla_prune_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_stage_event(self, event: Optional[torch.cuda.Event]) -> None:
        """Measurement aid: `event` is recorded between the scoring kernel and the selection + copy kernel
        of every non-overlapped prune step (None switches it off)."""
        rc = self._lib.mvla_set_stage_event(self._h, event.cuda_event if event is not None else None)
        if rc != OK:
            raise MvlaError(rc, "mvla_set_stage_event")

    STAMP_SLOTS = 4096

    def logit_cache_stats(self):
        """(key tiles recomputed, key tiles reused) by prune_step so far."""
        a, b = C.c_int64(0), C.c_int64(0)
        rc = self._lib.mvla_logit_cache_stats(self._h, C.byref(a), C.byref(b))
        if rc != OK:
            raise MvlaError(rc, "mvla_logit_cache_stats")
        return a.value, b.value

    def set_kernel_stamps(self, buf: Optional[torch.Tensor]) -> None:
        """Measurement aid: `buf` (int64 device tensor [2, 4096, 2], zero-filled; None switches it off) receives
        the start / end time stamps of the CTAs of the step's two kernels (see the header)."""
        if buf is not None:
            assert buf.dtype == torch.int64 and buf.numel() == 2 * self.STAMP_SLOTS * 2 and buf.is_contiguous()
        rc = self._lib.mvla_set_kernel_stamps(self._h, _ptr(buf))
        if rc != OK:
            raise MvlaError(rc, "mvla_set_kernel_stamps")

    def selftest_wait_timeout(self, limit_us: int = 200, *, stream=None) -> None:
        """Makes one bounded device-side wait run out on purpose (see the header); afterwards every call
        on this context raises MVLA_ERR_TIMEOUT."""
        rc = self._lib.mvla_selftest_wait_timeout(self._h, int(limit_us), _stream(stream))
        if rc != OK:
            raise MvlaError(rc, "mvla_selftest_wait_timeout")

    # -- allocation helpers (shapes only) ---------------------------------
    def alloc_outputs(self, samples: Sequence, *, hidden=True, kv=True, extras=False, patch=False) -> StepOutputs:
        rows = sum(s.n_txt + s.n_2d + s.n_3d for s in samples)
        nvis = sum(s.n_2d + s.n_3d for s in samples)
        npat = sum(s.n_2d for s in samples)
        c, dev, dt = self.cfg, self.device, self.torch_dtype
        mk = lambda *shape, dtype=dt: torch.empty(*shape, dtype=dtype, device=dev)
        return StepOutputs(
            out_hidden=mk(rows, c.d_model, dtype=self.hidden_dtype) if hidden else None,
            out_k=mk(rows, c.n_kv_heads or c.n_heads, c.head_dim) if kv else None,
            out_v=mk(rows, c.n_kv_heads or c.n_heads, c.head_dim) if kv else None,
            kept_idx=mk(rows, dtype=torch.int32),
            out_offsets=mk(len(samples) + 1, dtype=torch.int32),
            budgets=mk(len(samples), 2, dtype=torch.int32),
            attn=mk(nvis, dtype=torch.float32) if extras else None,
            ahat=mk(nvis, dtype=torch.float32) if extras else None,
            z=mk(nvis, dtype=torch.float32) if extras else None,
            diag=torch.zeros(len(samples), 16, dtype=torch.int32, device=dev) if extras else None,
            patch_x=mk(npat, 4, dtype=torch.float32) if patch else None,
            patch_xhat=mk(npat, 4, dtype=torch.float32) if patch else None,
            patch_info=mk(npat, dtype=torch.int32) if patch else None,
            patch_diag=torch.zeros(len(samples), 16, dtype=torch.int32, device=dev) if patch else None)

    # -- the six entry points ----------------------------------------------
    def salience(self, samples, q, k, hidden=None, *, attn_out=None, l1_out=None, stream=None):
        cs = samples if isinstance(samples, C.Array) else c_samples(samples)
        nvis = sum(s.n_2d + s.n_3d for s in cs)
        if attn_out is None:
            attn_out = torch.empty(nvis, dtype=torch.float32, device=self.device)
        if hidden is not None and l1_out is None:
            l1_out = torch.empty(nvis, dtype=torch.float32, device=self.device)
        rc = self._lib.mvla_salience(self._h, len(cs), cs, _ptr(q), _ptr(k), _ptr(hidden), q.shape[0],
                                     _ptr(attn_out), _ptr(l1_out), _stream(stream))
        if rc != OK:
            raise MvlaError(rc, "mvla_salience")
        return attn_out, l1_out

    def select(self, prune_point, samples, mode, attn, l1=None, *, flags=0, out: StepOutputs = None,
               stream=None) -> StepOutputs:
        cs = samples if isinstance(samples, C.Array) else c_samples(samples)
        if out is None:
            out = self.alloc_outputs(cs, hidden=False, kv=False, extras=True)
        rc = self._lib.mvla_select(self._h, prune_point, len(cs), cs, mode, flags, _ptr(attn), _ptr(l1),
                                   _ptr(out.kept_idx), _ptr(out.out_offsets), _ptr(out.budgets),
                                   _ptr(out.ahat), _ptr(out.z), _ptr(out.diag), _stream(stream))
        if rc != OK:
            raise MvlaError(rc, "mvla_select")
        return out

    def compact(self, samples, kept_idx, out_offsets, total_kept, hidden=None, k=None, v=None, *,
                out_hidden=None, out_k=None, out_v=None, stream=None):
        cs = samples if isinstance(samples, C.Array) else c_samples(samples)
        mk = lambda src: None if src is None else torch.empty((total_kept,) + tuple(src.shape[1:]),
                                                              dtype=src.dtype, device=src.device)
        out_hidden = mk(hidden) if out_hidden is None else out_hidden
        out_k = mk(k) if out_k is None else out_k
        out_v = mk(v) if out_v is None else out_v
        rc = self._lib.mvla_compact(self._h, len(cs), cs, _ptr(kept_idx), _ptr(out_offsets), int(total_kept),
                                    _ptr(hidden), _ptr(k), _ptr(v), _ptr(out_hidden), _ptr(out_k),
                                    _ptr(out_v), _stream(stream))
        if rc != OK:
            raise MvlaError(rc, "mvla_compact")
        return out_hidden, out_k, out_v

    def patch_indicators(self, samples, q, k, hidden, *, attn_out=None, x_out=None, stream=None):
        """Per-token scores and the four per-patch indicators (``mvla_patch_indicators``)."""
        cs = samples if isinstance(samples, C.Array) else c_samples(samples)
        nvis = sum(s.n_2d + s.n_3d for s in cs)
        if attn_out is None:
            attn_out = torch.empty(nvis, dtype=torch.float32, device=self.device)
        if x_out is None:
            x_out = torch.empty(nvis // 2, 4, dtype=torch.float32, device=self.device)
        rc = self._lib.mvla_patch_indicators(self._h, len(cs), cs, _ptr(q), _ptr(k), _ptr(hidden), q.shape[0],
                                             _ptr(attn_out), _ptr(x_out), _stream(stream))
        if rc != OK:
            raise MvlaError(rc, "mvla_patch_indicators")
        return attn_out, x_out

    def patch_select(self, prune_point, samples, attn, x, rand_u, *, flags=0, out: StepOutputs = None,
                     stream=None) -> StepOutputs:
        """Alg. 1 stages 1-4 patch by patch (``mvla_patch_select``); kept counts land in ``out.budgets``."""
        cs = samples if isinstance(samples, C.Array) else c_samples(samples)
        if out is None:
            out = self.alloc_outputs(cs, hidden=False, kv=False, patch=True)
        rc = self._lib.mvla_patch_select(self._h, prune_point, len(cs), cs, flags, _ptr(attn), _ptr(x), _ptr(rand_u),
                                         _ptr(out.kept_idx), _ptr(out.out_offsets), _ptr(out.budgets),
                                         _ptr(out.patch_xhat), _ptr(out.patch_info), _ptr(out.patch_diag),
                                         _stream(stream))
        if rc != OK:
            raise MvlaError(rc, "mvla_patch_select")
        return out

    def prune_step(self, prune_point, samples, mode, q, k, v, hidden, *, flags=0,
                   out: StepOutputs = None, stream=None, rand_u=None, changed_rows=None) -> StepOutputs:
        cs = samples if isinstance(samples, C.Array) else c_samples(samples)
        if out is None:
            out = self.alloc_outputs(cs, hidden=hidden is not None, kv=v is not None, extras=True,
                                     patch=mode == MODE_PATCH)
        ch = None
        if changed_rows is not None:         # host bytes, read during the call
            import numpy as np
            changed_rows = np.ascontiguousarray(changed_rows, dtype=np.uint8)
            assert changed_rows.shape[0] == q.shape[0], "one byte per row of the packed tensors"
            ch = changed_rows.ctypes.data
        tin = CTensors(_ptr(q), _ptr(k), _ptr(v), _ptr(hidden), q.shape[0], _ptr(rand_u), ch)
        tout = COutputs(_ptr(out.out_hidden), _ptr(out.out_k), _ptr(out.out_v), _ptr(out.kept_idx),
                        _ptr(out.out_offsets), _ptr(out.budgets), _ptr(out.attn), _ptr(out.ahat),
                        _ptr(out.z), _ptr(out.diag), _ptr(out.patch_x), _ptr(out.patch_xhat),
                        _ptr(out.patch_info), _ptr(out.patch_diag))
        total = C.c_int32(0)
        rc = self._lib.mvla_prune_step(self._h, prune_point, len(cs), cs, mode, flags, C.byref(tin),
                                       C.byref(tout), C.byref(total), _stream(stream))
        if rc != OK:
            raise MvlaError(rc, "mvla_prune_step")
        out.total_kept = total.value
        return out


def context_for(wl, *, max_batch=None, n_prune_points=1, n_state_slots=0, salience_path=SALIENCE_AUTO,
                device=None, patch_path=None, logit_cache=0) -> PruneContext:
    """A context sized for a synthetic workload (see ``workloads``)."""
    dt = {"bf16": torch.bfloat16, "fp32": torch.float32, "fp8": torch.float8_e4m3fn}[wl.dtype]
    return PruneContext(dtype=dt, n_heads=wl.n_heads, head_dim=wl.head_dim, d_model=wl.d_model,
                        max_batch=max_batch or len(wl.samples),
                        max_text=max(s.n_txt for s in wl.samples),
                        max_2d=max(max(s.n_2d for s in wl.samples), 1),
                        max_3d=max(max(s.n_3d for s in wl.samples), 1),
                        n_prune_points=n_prune_points, n_state_slots=n_state_slots, tau_2d=wl.tau_2d, tau_3d=wl.tau_3d,
                        beta=wl.beta, window_k=wl.window_k, eps_3d=wl.eps_3d,
                        floor_ratio=wl.floor_ratio, cold_start_full_keep=wl.cold_start_full_keep,
                        salience_path=salience_path, device=device,
                        patch_path=int(wl.mode == MODE_PATCH) if patch_path is None else patch_path,
                        obj_2d_min=wl.extra.get("obj_2d_min", 0.5),
                        kmeans_max_iter=wl.extra.get("kmeans_max_iter", 32),
                        n_kv_heads=wl.extra.get("n_kv_heads", 0), logit_cache=logit_cache)


def to_device(arr, dtype: str, device) -> torch.Tensor:
    """float32 numpy array holding dtype-exact values -> device tensor of that dtype."""
    t = torch.from_numpy(arr)
    if dtype == "bf16":
        t = t.to(torch.bfloat16)      # exact: the values are already bf16-representable
    elif dtype == "fp8":
        t = t.to(torch.float8_e4m3fn)  # exact likewise
    return t.to(device).contiguous()


def salience_noalloc(samples, q: torch.Tensor, k: torch.Tensor, attn_out: torch.Tensor, *, stream=None) -> None:
    """Salience scores through ``mvla_salience_noalloc``: no context, and the library allocates
    nothing.  Meant for callers that must not allocate device memory when they call in (a frozen
    memory pool, a real-time loop): they hand in `attn_out` (float32, sum of visual tokens) that they
    allocated earlier, and the library's scratch is a fixed array inside its image.  Problems with
    ``n_heads * sum(n_vis) > 131072`` are refused (``MVLA_ERR_CAPACITY``).  Calls on one device share
    that array: do not let two of them overlap on the GPU.  The first call on a device should be
    made outside stream capture."""
    L = lib()
    fn = L.mvla_salience_noalloc
    fn.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.POINTER(CSample), C.c_void_p,
                   C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]
    fn.restype = C.c_int32
    cs = samples if isinstance(samples, C.Array) else c_samples(samples)
    code = {torch.bfloat16: DTYPE_BF16, torch.float32: DTYPE_FP32}[q.dtype]
    assert attn_out.dtype == torch.float32
    rc = fn(q.device.index, code, q.shape[1], q.shape[2], len(cs), cs, _ptr(q), _ptr(k), q.shape[0],
            _ptr(attn_out), _stream(stream))
    if rc != OK:
        raise MvlaError(rc, "mvla_salience_noalloc")
