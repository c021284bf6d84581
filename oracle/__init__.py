"""ctypes loader for the fp64 CPU oracle (``mvla_oracle.c``).

TEST INFRASTRUCTURE ONLY: only the test-suite, the smoke check and the
benchmark's CPU-baseline leg may import this package.  It imports nothing from
the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import List, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libmvla_oracle.so")
_lib = None

SET_2D, SET_3D = 1, 2
MODE_FIXED, MODE_ADAPTIVE = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP over heads only)."""
    srcs = [os.path.join(_HERE, f) for f in ("mvla_oracle.c", "mvla_patch_oracle.c")]
    deps = srcs + [os.path.join(_HERE, f) for f in ("mvla_oracle.h", "mvla_patch_oracle.h")]
    if (not force and os.path.exists(_LIB_PATH)
            and os.path.getmtime(_LIB_PATH) >= max(os.path.getmtime(d) for d in deps)):
        return _LIB_PATH
    cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
           "-o", _LIB_PATH] + srcs + ["-lm"]
    subprocess.run(cmd, check=True)
    return _LIB_PATH


class CSample(C.Structure):
    _fields_ = [("seq_off", C.c_int32), ("off_txt", C.c_int32), ("n_txt", C.c_int32),
                ("off_2d", C.c_int32), ("n_2d", C.c_int32), ("off_3d", C.c_int32),
                ("n_3d", C.c_int32), ("keep_2d", C.c_double), ("keep_3d", C.c_double),
                ("keep_total", C.c_double)]


class CParams(C.Structure):
    _fields_ = [("tau_2d", C.c_double), ("tau_3d", C.c_double), ("beta", C.c_double),
                ("window_k", C.c_int32), ("eps_3d", C.c_double), ("floor_ratio", C.c_double),
                ("cold_start_full_keep", C.c_int32)]


class CState(C.Structure):
    _fields_ = [("t", C.c_int32), ("ahat", C.POINTER(C.c_double)), ("mhat", C.c_double * 4)]


class CDiag(C.Structure):
    _fields_ = [("t", C.c_int32), ("x", C.c_double * 4), ("mhat", C.c_double * 4),
                ("c_s1", C.c_int32), ("c_s2", C.c_int32), ("c_final", C.c_int32),
                ("budget", C.c_int32), ("k_2d", C.c_int32), ("k_3d", C.c_int32),
                ("near_half", C.c_int32), ("near_gate", C.c_int32)]


class CPatchParams(C.Structure):
    _fields_ = [("tau_2d", C.c_double), ("tau_3d", C.c_double), ("beta", C.c_double),
                ("window_k", C.c_int32), ("eps_3d", C.c_double), ("obj_2d_min", C.c_double),
                ("bg_prune_prob", C.c_double), ("kmeans_max_iter", C.c_int32),
                ("cold_start_full_keep", C.c_int32)]


class CPatchState(C.Structure):
    _fields_ = [("t", C.c_int32), ("xhat", C.POINTER(C.c_double))]


class CPatchDiag(C.Structure):
    _fields_ = [("t", C.c_int32), ("iters", C.c_int32), ("n_label", C.c_int32 * 3),
                ("k_2d", C.c_int32), ("k_3d", C.c_int32), ("centre", C.c_double * 3),
                ("mu_2d", C.c_double), ("mu_3d", C.c_double), ("kmeans_margin", C.c_double)]


def load(path: str):
    """Load an oracle library from `path` and declare its signatures."""
    if True:
        L = C.CDLL(path)
        fp, dp, ip = C.POINTER(C.c_float), C.POINTER(C.c_double), C.POINTER(C.c_int32)
        sp, pp = C.POINTER(CSample), C.POINTER(CParams)
        L.oracle_salience.argtypes = [fp, fp, C.c_int32, C.c_int32, sp, dp]
        L.oracle_salience.restype = None
        L.oracle_salience_gqa.argtypes = [fp, fp, C.c_int32, C.c_int32, C.c_int32, sp, dp]
        L.oracle_salience_gqa.restype = None
        L.oracle_salience_cached.argtypes = [fp, fp, C.c_int32, C.c_int32, sp, C.POINTER(C.c_uint8), C.c_int32,
                                             dp, dp, ip]
        L.oracle_salience_cached.restype = None
        L.oracle_l1norm.argtypes = [fp, C.c_int32, sp, dp]
        L.oracle_l1norm.restype = None
        L.oracle_indicators.argtypes = [dp, dp, C.c_int32, C.c_int32, dp]
        L.oracle_indicators.restype = None
        L.oracle_state_update.argtypes = [C.c_int32, C.c_int32, C.c_double, C.c_int32, dp, dp]
        L.oracle_state_update.restype = None
        L.oracle_normalise.argtypes = [dp, C.c_int32, C.c_int32, dp]
        L.oracle_normalise.restype = None
        L.oracle_gates.argtypes = [dp, pp, ip, ip, ip, ip]
        L.oracle_gates.restype = None
        L.oracle_round_half_up.argtypes = [C.c_double]
        L.oracle_round_half_up.restype = C.c_int32
        L.oracle_budget_fixed.argtypes = [sp, ip, ip]
        L.oracle_budget_fixed.restype = None
        L.oracle_budget_total.argtypes = [sp]
        L.oracle_budget_total.restype = C.c_int32
        L.oracle_budget_adaptive.argtypes = [sp, pp, C.c_double, C.c_int32, ip, ip, ip]
        L.oracle_budget_adaptive.restype = None
        L.oracle_select.argtypes = [dp, sp, C.c_int32, C.c_int32, ip]
        L.oracle_select.restype = C.c_int32
        L.oracle_compact.argtypes = [C.c_void_p, C.c_int64, C.c_int32, ip, C.c_int32, C.c_void_p]
        L.oracle_compact.restype = None
        L.oracle_prune_step.argtypes = [fp, fp, fp, C.c_int32, C.c_int32, C.c_int32, sp, pp,
                                        C.c_int32, C.POINTER(CState), ip, C.POINTER(CDiag),
                                        dp, dp, dp, dp]
        L.oracle_prune_step.restype = C.c_int32
        L.oracle_decide_step.argtypes = [dp, dp, sp, pp, C.c_int32, C.POINTER(CState), ip,
                                         C.POINTER(CDiag), dp, dp]
        L.oracle_decide_step.restype = C.c_int32
        L.oracle_set_num_threads.argtypes = [C.c_int32]
        L.oracle_set_num_threads.restype = None
        L.oracle_num_threads.argtypes = []
        L.oracle_num_threads.restype = C.c_int32
        # Alg. 1 patch by patch
        ppp, psp, pdp = C.POINTER(CPatchParams), C.POINTER(CPatchState), C.POINTER(CPatchDiag)
        L.oracle_attention.argtypes = [fp, fp, C.c_int32, C.c_int32, sp, dp]
        L.oracle_attention.restype = None
        L.oracle_ortho_decompose.argtypes = [dp, dp, C.c_int32, dp, dp]
        L.oracle_ortho_decompose.restype = None
        L.oracle_patch_indicators.argtypes = [dp, C.c_int32, C.c_int32, dp, dp]
        L.oracle_patch_indicators.restype = None
        L.oracle_kmeans1d.argtypes = [dp, C.c_int32, C.c_int32, ip, dp, dp]
        L.oracle_kmeans1d.restype = C.c_int32
        L.oracle_patch_c_s1.argtypes = [C.c_double, C.c_double, C.c_double]
        L.oracle_patch_c_s1.restype = C.c_int32
        L.oracle_patch_c_s2.argtypes = [C.c_int32, C.c_double, C.c_double, C.c_double, C.c_double,
                                        C.c_double, ppp]
        L.oracle_patch_c_s2.restype = C.c_int32
        L.oracle_patch_fuse.argtypes = [C.c_int32, C.c_int32]
        L.oracle_patch_fuse.restype = C.c_int32
        L.oracle_patch_select.argtypes = [dp, dp, dp, sp, ppp, psp, ip, ip, ip, pdp]
        L.oracle_patch_select.restype = C.c_int32
        L.oracle_patch_step.argtypes = [fp, fp, fp, C.c_int32, C.c_int32, C.c_int32, sp, dp, ppp, psp,
                                        ip, ip, ip, pdp, dp, dp]
        L.oracle_patch_step.restype = C.c_int32
    return L


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = load(_LIB_PATH)
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def set_num_threads(n: int) -> None:
    """Threads the head loops use from now on (reporting: the oracle timed on one core and on all)."""
    lib().oracle_set_num_threads(int(n))


# --------------------------------------------------------------------------
# numpy-facing wrappers
# --------------------------------------------------------------------------
def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(C.POINTER(C.c_float))


def _f64(a):
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a, a.ctypes.data_as(C.POINTER(C.c_double))


def c_sample(s) -> CSample:
    """From any object with the descriptor's field names."""
    return CSample(int(s.seq_off), int(s.off_txt), int(s.n_txt), int(s.off_2d), int(s.n_2d),
                   int(s.off_3d), int(s.n_3d), float(s.keep_2d), float(s.keep_3d),
                   float(s.keep_total))


def c_params(tau_2d=0.08, tau_3d=0.20, beta=0.85, window_k=7, eps_3d=0.02, floor_ratio=0.10,
             cold_start_full_keep=1) -> CParams:
    return CParams(float(tau_2d), float(tau_3d), float(beta), int(window_k), float(eps_3d),
                   float(floor_ratio), int(cold_start_full_keep))


def params_of(wl) -> CParams:
    return c_params(wl.tau_2d, wl.tau_3d, wl.beta, wl.window_k, wl.eps_3d, wl.floor_ratio,
                    wl.cold_start_full_keep)


def salience(q, k, n_heads, head_dim, s) -> np.ndarray:
    q, qp = _f32(q)
    k, kp = _f32(k)
    cs = c_sample(s)
    out = np.zeros(cs.n_2d + cs.n_3d, dtype=np.float64)
    lib().oracle_salience(qp, kp, n_heads, head_dim, C.byref(cs), out.ctypes.data_as(C.POINTER(C.c_double)))
    return out


def salience_gqa(q, k, n_heads, n_kv_heads, head_dim, s) -> np.ndarray:
    """q: [rows, H, d]; k: [rows, H_kv, d]."""
    q, qp = _f32(q)
    k, kp = _f32(k)
    cs = c_sample(s)
    out = np.zeros(cs.n_2d + cs.n_3d, dtype=np.float64)
    lib().oracle_salience_gqa(qp, kp, n_heads, n_kv_heads, head_dim, C.byref(cs),
                              out.ctypes.data_as(C.POINTER(C.c_double)))
    return out


class LogitCache:
    """The previous action step's logits of one sample, [H, n_txt, n_vis] (see oracle_salience_cached)."""

    def __init__(self, n_heads: int, s):
        self.logits = np.zeros((n_heads, int(s.n_txt), int(s.n_2d) + int(s.n_3d)), dtype=np.float64)
        self.valid = False


def salience_cached(q, k, n_heads, head_dim, s, changed, cache: LogitCache):
    """Returns (scores, number of visual keys whose logits were recomputed); updates `cache`."""
    q, qp = _f32(q)
    k, kp = _f32(k)
    cs = c_sample(s)
    out = np.zeros(cs.n_2d + cs.n_3d, dtype=np.float64)
    mp = None
    if changed is not None:
        changed = np.ascontiguousarray(changed, dtype=np.uint8)
        mp = changed.ctypes.data_as(C.POINTER(C.c_uint8))
    n = C.c_int32()
    lib().oracle_salience_cached(qp, kp, n_heads, head_dim, C.byref(cs), mp, int(cache.valid),
                                 cache.logits.ctypes.data_as(C.POINTER(C.c_double)),
                                 out.ctypes.data_as(C.POINTER(C.c_double)), C.byref(n))
    cache.valid = True
    return out, n.value


def l1norm(hidden, d_model, s) -> np.ndarray:
    h, hp = _f32(hidden)
    cs = c_sample(s)
    out = np.zeros(cs.n_2d + cs.n_3d, dtype=np.float64)
    lib().oracle_l1norm(hp, d_model, C.byref(cs), out.ctypes.data_as(C.POINTER(C.c_double)))
    return out


def indicators(a, l1, n_2d, n_3d) -> np.ndarray:
    a, ap = _f64(a)
    lp = None
    if l1 is not None:
        l1, lp = _f64(l1)
    x = np.zeros(4, dtype=np.float64)
    lib().oracle_indicators(ap, lp, n_2d, n_3d, x.ctypes.data_as(C.POINTER(C.c_double)))
    return x


def state_update(t, window_k, beta, x, xhat) -> np.ndarray:
    x, xp = _f64(x)
    xhat = np.array(xhat, dtype=np.float64, copy=True)
    lib().oracle_state_update(t, window_k, beta, len(x), xp, xhat.ctypes.data_as(C.POINTER(C.c_double)))
    return xhat


def normalise(ahat, n_2d, n_3d) -> np.ndarray:
    a, ap = _f64(ahat)
    z = np.zeros_like(a)
    lib().oracle_normalise(ap, n_2d, n_3d, z.ctypes.data_as(C.POINTER(C.c_double)))
    return z


def gates(mhat, params: CParams):
    m, mp = _f64(mhat)
    c1, c2, cf, ng = C.c_int32(), C.c_int32(), C.c_int32(), C.c_int32()
    lib().oracle_gates(mp, C.byref(params), C.byref(c1), C.byref(c2), C.byref(cf), C.byref(ng))
    return c1.value, c2.value, cf.value, ng.value


def budget_fixed(s):
    cs = c_sample(s)
    k2, k3 = C.c_int32(), C.c_int32()
    lib().oracle_budget_fixed(C.byref(cs), C.byref(k2), C.byref(k3))
    return k2.value, k3.value


def budget_total(s) -> int:
    cs = c_sample(s)
    return lib().oracle_budget_total(C.byref(cs))


def budget_adaptive(s, params: CParams, mhat_s2_3d: float, c_final: int):
    cs = c_sample(s)
    k2, k3, nh = C.c_int32(), C.c_int32(), C.c_int32()
    lib().oracle_budget_adaptive(C.byref(cs), C.byref(params), float(mhat_s2_3d), int(c_final),
                                 C.byref(k2), C.byref(k3), C.byref(nh))
    return k2.value, k3.value, nh.value


def select(z, s, k_2d, k_3d) -> np.ndarray:
    z, zp = _f64(z)
    cs = c_sample(s)
    out = np.zeros(cs.n_txt + cs.n_2d + cs.n_3d, dtype=np.int32)
    n = lib().oracle_select(zp, C.byref(cs), k_2d, k_3d, out.ctypes.data_as(C.POINTER(C.c_int32)))
    return out[:n].copy()


def compact(src: np.ndarray, seq_off: int, kept_idx: np.ndarray) -> np.ndarray:
    """src: [rows, ...] array of any dtype; returns the kept rows (byte copy)."""
    src = np.ascontiguousarray(src)
    kept = np.ascontiguousarray(kept_idx, dtype=np.int32)
    row_bytes = src.strides[0]
    dst = np.zeros((len(kept),) + src.shape[1:], dtype=src.dtype)
    lib().oracle_compact(src.ctypes.data, row_bytes, int(seq_off),
                         kept.ctypes.data_as(C.POINTER(C.c_int32)), len(kept), dst.ctypes.data)
    return dst


@dataclass
class StepResult:
    kept_idx: np.ndarray
    attn: np.ndarray
    l1: Optional[np.ndarray]
    ahat: np.ndarray
    z: np.ndarray
    t: int
    x: np.ndarray
    mhat: np.ndarray
    c_s1: int
    c_s2: int
    c_final: int
    k_2d: int
    k_3d: int
    near_half: bool
    near_gate: bool


class State:
    """Smoothed state of one (prune point, sample)."""

    def __init__(self, n_vis: int):
        self.ahat = np.zeros(n_vis, dtype=np.float64)
        self.c = CState(0, self.ahat.ctypes.data_as(C.POINTER(C.c_double)), (C.c_double * 4)(0, 0, 0, 0))

    @property
    def t(self) -> int:
        return self.c.t


def prune_step(q, k, hidden, n_heads, head_dim, d_model, s, params: CParams, mode: int,
               state: State) -> StepResult:
    q, qp = _f32(q)
    k, kp = _f32(k)
    hp = None
    if hidden is not None:
        hidden, hp = _f32(hidden)
    cs = c_sample(s)
    nv = cs.n_2d + cs.n_3d
    kept = np.zeros(cs.n_txt + nv, dtype=np.int32)
    attn = np.zeros(nv); l1 = np.zeros(nv); ahat = np.zeros(nv); z = np.zeros(nv)
    dg = CDiag()
    dp = lambda a: a.ctypes.data_as(C.POINTER(C.c_double))
    n = lib().oracle_prune_step(qp, kp, hp, n_heads, head_dim, d_model, C.byref(cs), C.byref(params),
                                mode, C.byref(state.c), kept.ctypes.data_as(C.POINTER(C.c_int32)),
                                C.byref(dg), dp(attn), dp(l1), dp(ahat), dp(z))
    return StepResult(kept[:n].copy(), attn, l1 if mode == MODE_ADAPTIVE else None, ahat, z, dg.t,
                      np.array(dg.x[:]), np.array(dg.mhat[:]), dg.c_s1, dg.c_s2, dg.c_final,
                      dg.k_2d, dg.k_3d, bool(dg.near_half), bool(dg.near_gate))


def decide_step(a, l1, s, params: CParams, mode: int, state: State) -> StepResult:
    """Alg. 1 from the scores on: `a` [n_vis] attention scores, `l1` [n_vis] feature norms or None."""
    a, ap = _f64(a)
    lp = None
    if l1 is not None:
        l1, lp = _f64(l1)
    cs = c_sample(s)
    nv = cs.n_2d + cs.n_3d
    kept = np.zeros(cs.n_txt + nv, dtype=np.int32)
    ahat = np.zeros(nv); z = np.zeros(nv)
    dg = CDiag()
    dp = lambda v: v.ctypes.data_as(C.POINTER(C.c_double))
    n = lib().oracle_decide_step(ap, lp, C.byref(cs), C.byref(params), mode, C.byref(state.c),
                                 kept.ctypes.data_as(C.POINTER(C.c_int32)), C.byref(dg), dp(ahat), dp(z))
    return StepResult(kept[:n].copy(), a.copy(), None if l1 is None else l1.copy(), ahat, z, dg.t,
                      np.array(dg.x[:]), np.array(dg.mhat[:]), dg.c_s1, dg.c_s2, dg.c_final,
                      dg.k_2d, dg.k_3d, bool(dg.near_half), bool(dg.near_gate))


def run_workload_step(wl, step: int, states: List[State]) -> List[StepResult]:
    """All samples of one action step of a workload (see the seeded input
    generators); `states` has one State per sample."""
    ten = wl.steps[step]
    p = params_of(wl)
    return [prune_step(ten.q, ten.k, ten.hidden if wl.mode == MODE_ADAPTIVE else None,
                       wl.n_heads, wl.head_dim, wl.d_model, s, p, wl.mode, states[b])
            for b, s in enumerate(wl.samples)]


# --------------------------------------------------------------------------
# Alg. 1 patch by patch (mvla_patch_oracle.c)
# --------------------------------------------------------------------------
LABEL_BG, LABEL_ROB, LABEL_OBJ = 0, 1, 2


def c_patch_params(tau_2d=0.08, tau_3d=0.20, beta=0.85, window_k=7, eps_3d=0.02, obj_2d_min=0.5,
                   bg_prune_prob=0.9, kmeans_max_iter=32, cold_start_full_keep=1) -> CPatchParams:
    return CPatchParams(float(tau_2d), float(tau_3d), float(beta), int(window_k), float(eps_3d),
                        float(obj_2d_min), float(bg_prune_prob), int(kmeans_max_iter),
                        int(cold_start_full_keep))


def patch_params_of(wl) -> CPatchParams:
    return c_patch_params(wl.tau_2d, wl.tau_3d, wl.beta, wl.window_k, wl.eps_3d,
                          wl.extra.get("obj_2d_min", 0.5), 1.0 - wl.floor_ratio,
                          wl.extra.get("kmeans_max_iter", 32), wl.cold_start_full_keep)


def attention(q, k, n_heads, head_dim, s) -> np.ndarray:
    """alpha[h, i, j]: [H, n_txt, n_vis]."""
    q, qp = _f32(q)
    k, kp = _f32(k)
    cs = c_sample(s)
    out = np.zeros((n_heads, cs.n_txt, cs.n_2d + cs.n_3d), dtype=np.float64)
    lib().oracle_attention(qp, kp, n_heads, head_dim, C.byref(cs), out.ctypes.data_as(C.POINTER(C.c_double)))
    return out


def ortho_decompose(a2, a3):
    a2, p2 = _f64(a2)
    a3, p3 = _f64(a3)
    para, ortho = np.zeros_like(a2), np.zeros_like(a2)
    dp = lambda a: a.ctypes.data_as(C.POINTER(C.c_double))
    lib().oracle_ortho_decompose(p2, p3, len(a2), dp(para), dp(ortho))
    return para, ortho


def patch_indicators(alpha, l1) -> np.ndarray:
    """alpha: [rows, 2P]; l1: [2P] -> x [P, 4]."""
    alpha, ap = _f64(alpha)
    l1, lp = _f64(l1)
    rows, nv = alpha.shape
    x = np.zeros((nv // 2, 4), dtype=np.float64)
    lib().oracle_patch_indicators(ap, rows, nv // 2, lp, x.ctypes.data_as(C.POINTER(C.c_double)))
    return x


def kmeans1d(v, max_iter=32):
    v, vp = _f64(v)
    labels = np.zeros(len(v), dtype=np.int32)
    centre = np.zeros(3, dtype=np.float64)
    margin = C.c_double()
    it = lib().oracle_kmeans1d(vp, len(v), max_iter, labels.ctypes.data_as(C.POINTER(C.c_int32)),
                               centre.ctypes.data_as(C.POINTER(C.c_double)), C.byref(margin))
    return labels, centre, it, margin.value


def patch_c_s1(m, tau_2d, tau_3d) -> int:
    return lib().oracle_patch_c_s1(float(m), float(tau_2d), float(tau_3d))


def patch_c_s2(label, m2, m3, mu_2d, mu_3d, u, params: CPatchParams) -> int:
    return lib().oracle_patch_c_s2(int(label), float(m2), float(m3), float(mu_2d), float(mu_3d),
                                   float(u), C.byref(params))


def patch_fuse(c_s1, c_s2) -> int:
    return lib().oracle_patch_fuse(int(c_s1), int(c_s2))


class PatchState:
    """Smoothed per-patch indicators of one (prune point, sample)."""

    def __init__(self, n_patch: int):
        self.xhat = np.zeros((n_patch, 4), dtype=np.float64)
        self.c = CPatchState(0, self.xhat.ctypes.data_as(C.POINTER(C.c_double)))

    @property
    def t(self) -> int:
        return self.c.t


@dataclass
class PatchResult:
    kept_idx: np.ndarray
    labels: np.ndarray
    cand: np.ndarray          # [P, 3] = (C_S1, C_S2, C_final)
    attn: Optional[np.ndarray]
    x: Optional[np.ndarray]
    xhat: np.ndarray
    t: int
    iters: int
    n_label: np.ndarray
    k_2d: int
    k_3d: int
    centre: np.ndarray
    mu_2d: float
    mu_3d: float
    kmeans_margin: float


def _patch_result(n, kept, labels, cand, attn, x, state, dg) -> PatchResult:
    return PatchResult(kept[:n].copy(), labels, cand, attn, x, state.xhat.copy(), dg.t, dg.iters,
                       np.array(dg.n_label[:]), dg.k_2d, dg.k_3d, np.array(dg.centre[:]), dg.mu_2d,
                       dg.mu_3d, dg.kmeans_margin)


def patch_select(a, x, u, s, params: CPatchParams, state: PatchState) -> PatchResult:
    a, ap = _f64(a)
    x, xp = _f64(x)
    u, up = _f64(u)
    cs = c_sample(s)
    P = cs.n_2d
    kept = np.zeros(cs.n_txt + 2 * P, dtype=np.int32)
    labels = np.zeros(P, dtype=np.int32)
    cand = np.zeros((P, 3), dtype=np.int32)
    dg = CPatchDiag()
    ip = lambda v: v.ctypes.data_as(C.POINTER(C.c_int32))
    n = lib().oracle_patch_select(ap, xp, up, C.byref(cs), C.byref(params), C.byref(state.c), ip(labels),
                                  ip(cand), ip(kept), C.byref(dg))
    return _patch_result(n, kept, labels, cand, None, None, state, dg)


def patch_step(q, k, hidden, n_heads, head_dim, d_model, s, u, params: CPatchParams,
               state: PatchState) -> PatchResult:
    q, qp = _f32(q)
    k, kp = _f32(k)
    hidden, hp = _f32(hidden)
    u, up = _f64(u)
    cs = c_sample(s)
    P = cs.n_2d
    assert cs.n_3d == P, "a patch owns one 2D and one 3D token"
    kept = np.zeros(cs.n_txt + 2 * P, dtype=np.int32)
    labels = np.zeros(P, dtype=np.int32)
    cand = np.zeros((P, 3), dtype=np.int32)
    attn = np.zeros(2 * P)
    x = np.zeros((P, 4))
    dg = CPatchDiag()
    ip = lambda v: v.ctypes.data_as(C.POINTER(C.c_int32))
    dp = lambda v: v.ctypes.data_as(C.POINTER(C.c_double))
    n = lib().oracle_patch_step(qp, kp, hp, n_heads, head_dim, d_model, C.byref(cs), up, C.byref(params),
                                C.byref(state.c), ip(labels), ip(cand), ip(kept), C.byref(dg), dp(attn), dp(x))
    assert n >= 0
    return _patch_result(n, kept, labels, cand, attn, x, state, dg)
