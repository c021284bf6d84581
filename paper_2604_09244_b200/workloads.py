"""Seeded synthetic inputs for the MVLA prune step.

This module only *draws data*: token hidden states, projection weights, the
Q/K/V projections of those hidden states, and the per-sample segment
descriptors.  It holds none of the pruning method's arithmetic (no attention,
no scoring, no selection), so both the CPU oracle's tests and the CUDA path's
tests may import it.

The inputs stand in for the paper's workload (Sec. 5.1 and App. "MVLA
Models": a LLaMA-2-7B-width backbone fed 256 image tokens from 16x16 patches
plus 256 point tokens and a language instruction), whose checkpoint and
simulator frames are not available.  Common recipe:

* ``numpy.random.default_rng(seed)`` (PCG64); draw order
  ``hidden -> W_q -> W_k -> W_v -> structure indices``;
* ``hidden ~ N(0, 1)``; ``W ~ N(0, 1/D)``; a salient token has its hidden row
  multiplied by a gain *before* projection;
* ``Q = hidden @ W_q`` (same for K, V) in fp32, reshaped ``[S, H, d]``;
* everything is rounded once to the workload's dtype (bf16: round to nearest
  even); the float32 arrays returned hold exactly those rounded values, so
  every consumer sees the same bits;
* sequence order inside a sample is ``[2D | 3D | text]``.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

MODE_FIXED = 0
MODE_ADAPTIVE = 1
MODE_PATCH = 2


# --------------------------------------------------------------------------
# dtype helpers (data conversion only)
# --------------------------------------------------------------------------
def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); the result
    is float32 holding exactly representable bf16 values."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are already bf16-exact."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def round_to_e4m3(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest 8-bit e4m3 value (finite format, largest magnitude 448, ties to
    even, saturating); the result is float32 holding exactly representable e4m3 values."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).clamp(-448.0, 448.0)
    return t.to(torch.float8_e4m3fn).to(torch.float32).numpy()


def e4m3_bits(x: np.ndarray) -> np.ndarray:
    """uint8 bit patterns of float32 values that are already e4m3-exact."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.float8_e4m3fn)
    return t.view(torch.uint8).numpy()


def round_to_dtype(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "fp8":
        return round_to_e4m3(x)
    if dtype == "bf16":
        return round_to_bf16(x)
    if dtype == "fp32":
        return np.ascontiguousarray(x, dtype=np.float32)
    raise ValueError(dtype)


# --------------------------------------------------------------------------
# descriptors
# --------------------------------------------------------------------------
@dataclass
class Sample:
    """One batch element: three contiguous segments inside the packed
    ``[sum S, .]`` tensors.  Offsets are rows relative to ``seq_off``."""
    seq_off: int
    off_txt: int
    n_txt: int
    off_2d: int
    n_2d: int
    off_3d: int
    n_3d: int
    keep_2d: float = 0.0      # FIXED mode: fraction of 2D tokens kept
    keep_3d: float = 0.0      # FIXED mode: fraction of 3D tokens kept
    keep_total: float = 0.0   # ADAPTIVE mode: fraction of all visual tokens kept
    state_slot: int = 0

    @property
    def n_vis(self) -> int:
        return self.n_2d + self.n_3d

    @property
    def seq_len(self) -> int:
        return self.n_txt + self.n_2d + self.n_3d


@dataclass
class Tensors:
    """Packed token-major tensors of one prune call (float32 arrays whose
    values are exact in the workload's dtype)."""
    hidden: np.ndarray  # [sum S, D]
    q: np.ndarray       # [sum S, H, d]
    k: np.ndarray       # [sum S, H, d]
    v: np.ndarray       # [sum S, H, d]


@dataclass
class Workload:
    name: str
    dtype: str                 # "bf16" | "fp32" | "fp8" (q, k, v in e4m3; hidden bf16)
    n_heads: int
    head_dim: int
    d_model: int
    mode: int                  # MODE_FIXED | MODE_ADAPTIVE | MODE_PATCH
    samples: List[Sample]
    steps: List[Tensors]       # one entry per action step (len 1 unless config 5)
    cold_start_full_keep: int = 0
    tau_2d: float = 0.35       # synthetic gate thresholds (both modalities ~N(0,1))
    tau_3d: float = 0.65
    beta: float = 0.85
    window_k: int = 7
    eps_3d: float = 0.02
    floor_ratio: float = 0.10
    seed: int = 0
    extra: dict = field(default_factory=dict)

    @property
    def total_rows(self) -> int:
        return sum(s.seq_len for s in self.samples)

    @property
    def total_vis(self) -> int:
        return sum(s.n_vis for s in self.samples)


def layout_2d_3d_txt(seq_off: int, n_txt: int, n_2d: int, n_3d: int, **kw) -> Sample:
    return Sample(seq_off=seq_off, off_2d=0, n_2d=n_2d, off_3d=n_2d, n_3d=n_3d,
                  off_txt=n_2d + n_3d, n_txt=n_txt, **kw)


# --------------------------------------------------------------------------
# drawing
# --------------------------------------------------------------------------
def _draw_weights(rng: np.random.Generator, D: int, out: int = 0, out_kv: int = 0):
    out = out or D          # projection width H*d (equal to D in the paper-shaped workloads)
    out_kv = out_kv or out  # narrower when the key / value heads are grouped
    std = 1.0 / np.sqrt(D)
    wq = rng.standard_normal((D, out), dtype=np.float32) * np.float32(std)
    wk = rng.standard_normal((D, out_kv), dtype=np.float32) * np.float32(std)
    wv = rng.standard_normal((D, out_kv), dtype=np.float32) * np.float32(std)
    return wq, wk, wv


def _project(hidden: np.ndarray, w, H: int, d: int, dtype: str, H_kv: int = 0) -> Tensors:
    """hidden is fp32 (not yet rounded).  Projections are taken from the
    unrounded fp32 hidden, then all four tensors are rounded once."""
    wq, wk, wv = w
    S = hidden.shape[0]
    q = (hidden @ wq).reshape(S, H, d)
    k = (hidden @ wk).reshape(S, H_kv or H, d)
    v = (hidden @ wv).reshape(S, H_kv or H, d)
    # "fp8": q, k, v in e4m3, the hidden states stay bf16
    return Tensors(hidden=round_to_dtype(hidden, "bf16" if dtype == "fp8" else dtype), q=round_to_dtype(q, dtype),
                   k=round_to_dtype(k, dtype), v=round_to_dtype(v, dtype))


def _rhu(x: float) -> int:
    return int(np.floor(x + 0.5))


def _spike_rows(rng, sample: Sample, frac: float) -> np.ndarray:
    """Row indices (relative to the sample) of `rhu(frac*N_m)` tokens per modality."""
    rows = []
    for off, n in ((sample.off_2d, sample.n_2d), (sample.off_3d, sample.n_3d)):
        m = _rhu(frac * n)
        idx = rng.choice(n, size=m, replace=False)
        rows.append(off + np.sort(idx))
    return np.concatenate(rows)


# --------------------------------------------------------------------------
# the five configurations
# --------------------------------------------------------------------------
def config1_tiny(seed: int = 0) -> Workload:
    """Tiny reference: batch 1, D=512, 8 heads x 64, 16 text + 64 2D + 128 3D,
    fp32, 4 boosted (x4) tokens per modality, adaptive keep 50 %."""
    D, H, d = 512, 8, 64
    s = layout_2d_3d_txt(0, 16, 64, 128, keep_total=0.5)
    rng = np.random.default_rng(seed)
    hidden = rng.standard_normal((s.seq_len, D), dtype=np.float32)
    w = _draw_weights(rng, D)
    boost = np.concatenate([s.off_2d + np.sort(rng.choice(s.n_2d, 4, replace=False)),
                            s.off_3d + np.sort(rng.choice(s.n_3d, 4, replace=False))])
    hidden[boost] *= np.float32(4.0)
    return Workload("tiny_ref", "fp32", H, d, D, MODE_ADAPTIVE, [s],
                    [_project(hidden, w, H, d, "fp32")], seed=seed,
                    extra={"boosted": boost})


def config2_single_frame(seed: int = 1, n_txt=32, n_2d=256, n_3d=512,
                         D=4096, H=32, d=128, dtype="bf16") -> Workload:
    """7B-shaped single frame: 32 text + 256 2D (16x16) + 512 3D, bf16,
    5 % spikes x4 per modality, FIXED keep 40 % (2D) / 30 % (3D)."""
    s = layout_2d_3d_txt(0, n_txt, n_2d, n_3d, keep_2d=0.40, keep_3d=0.30)
    rng = np.random.default_rng(seed)
    hidden = rng.standard_normal((s.seq_len, D), dtype=np.float32)
    w = _draw_weights(rng, D)
    spikes = _spike_rows(rng, s, 0.05)
    hidden[spikes] *= np.float32(4.0)
    return Workload("single_frame_7b", dtype, H, d, D, MODE_FIXED, [s],
                    [_project(hidden, w, H, d, dtype)], seed=seed,
                    extra={"spikes": spikes})


def _region_gain(rng, n_views: int, side: int, n_regions: int) -> np.ndarray:
    """Gain map of `n_views` grids of side x side tokens with `n_regions`
    3x3 blocks of gain 1 + 3 exp(-r^2/2); overlaps take the larger gain."""
    g = np.ones((n_views, side, side), dtype=np.float32)
    for _ in range(n_regions):
        vw = int(rng.integers(n_views))
        cy = int(rng.integers(side))
        cx = int(rng.integers(side))
        for dy in (-1, 0, 1):
            for dx in (-1, 0, 1):
                y, x = cy + dy, cx + dx
                if 0 <= y < side and 0 <= x < side:
                    val = np.float32(1.0 + 3.0 * np.exp(-(dy * dy + dx * dx) / 2.0))
                    g[vw, y, x] = max(g[vw, y, x], val)
    return g.reshape(-1)


def config3_multi_view(seed: int = 2, D=4096, H=32, d=128, dtype="bf16") -> Workload:
    """Multi-view, first prune point: 48 text + 3 views x 256 2D + 1024 3D
    (a 32x32 grid), 8 salient 3x3 regions per modality, adaptive keep 25 %."""
    s = layout_2d_3d_txt(0, 48, 3 * 256, 1024, keep_total=0.25)
    rng = np.random.default_rng(seed)
    hidden = rng.standard_normal((s.seq_len, D), dtype=np.float32)
    w = _draw_weights(rng, D)
    g2 = _region_gain(rng, 3, 16, 8)
    g3 = _region_gain(rng, 1, 32, 8)
    hidden[s.off_2d:s.off_2d + s.n_2d] *= g2[:, None]
    hidden[s.off_3d:s.off_3d + s.n_3d] *= g3[:, None]
    wl = Workload("multi_view_p1", dtype, H, d, D, MODE_ADAPTIVE, [s],
                  [_project(hidden, w, H, d, dtype)], seed=seed)
    wl.extra["hidden_fp32_rounded"] = wl.steps[0].hidden
    return wl


def config3_second_point(first: Workload, kept_rows: np.ndarray, k_2d: int, k_3d: int,
                         layer: int = 8) -> Workload:
    """Second prune point of the multi-view workload: the rows of the first
    point's (dtype-rounded) hidden states listed in `kept_rows` (the first
    point's kept positions, ascending) re-projected with fresh weights drawn
    from seed + layer.  `k_2d`, `k_3d` are the first point's budgets, which
    become this point's segment lengths."""
    s0 = first.samples[0]
    assert len(kept_rows) == s0.n_txt + k_2d + k_3d
    s = layout_2d_3d_txt(0, s0.n_txt, k_2d, k_3d, keep_total=s0.keep_total)
    rng = np.random.default_rng(first.seed + layer)
    w = _draw_weights(rng, first.d_model)
    hidden = np.ascontiguousarray(first.steps[0].hidden[np.asarray(kept_rows)])
    return Workload("multi_view_p2", first.dtype, first.n_heads, first.head_dim, first.d_model,
                    MODE_ADAPTIVE, [s],
                    [_project(hidden, w, first.n_heads, first.head_dim, first.dtype)],
                    seed=first.seed + layer)


def config4_batched(seed: int = 3, batch: int = 16, D=4096, H=32, d=128, dtype="bf16",
                    n_2d=256, n_3d=512, txt_lo=16, txt_hi=64) -> Workload:
    """Batched serving: per-sample text length U{16..64}, 256 2D + 512 3D,
    5 % spikes x4, per-sample adaptive keep ratio U[0.2, 0.6] rounded to 1e-3;
    packed ragged."""
    rng = np.random.default_rng(seed)
    n_txts = rng.integers(txt_lo, txt_hi + 1, size=batch)
    keeps = np.round(rng.uniform(0.2, 0.6, size=batch), 3)
    samples, off = [], 0
    for b in range(batch):
        s = layout_2d_3d_txt(off, int(n_txts[b]), n_2d, n_3d, keep_total=float(keeps[b]),
                             state_slot=b)
        samples.append(s)
        off += s.seq_len
    hidden = rng.standard_normal((off, D), dtype=np.float32)
    w = _draw_weights(rng, D)
    for s in samples:
        hidden[s.seq_off + _spike_rows(rng, s, 0.05)] *= np.float32(4.0)
    return Workload("batched_serving", dtype, H, d, D, MODE_ADAPTIVE, samples,
                    [_project(hidden, w, H, d, dtype)], seed=seed)


def config5_action_iteration(seed: int = 4, T: int = 16, D=4096, H=32, d=128, dtype="bf16",
                             n_txt=32, n_2d=256, n_3d=1024, drift: str = "all") -> Workload:
    """Action iteration: T sequential steps of 32 text + 256 2D + 1024 3D.
    Step 1 is structured like the single-frame workload (5 % spikes x4); each
    later step adds N(0, sigma=0.1) to the (unrounded) hidden rows of a fresh
    random 10 % of all tokens and re-projects those rows with the same
    weights.  Adaptive keep 30 %, cold start on (step 1 keeps everything).
    ``extra["changed_rows"][t]`` is the truthful mask (uint8 per row) of the rows
    step t rewrote (all ones at t = 0).  ``drift="visual_local"`` is the variant
    in which consecutive frames share most of their content: the instruction
    (text rows) stays fixed and the 10 % of rows that drift are one contiguous
    run of visual tokens whose position moves from step to step."""
    s = layout_2d_3d_txt(0, n_txt, n_2d, n_3d, keep_total=0.30)
    rng = np.random.default_rng(seed)
    hidden = rng.standard_normal((s.seq_len, D), dtype=np.float32)
    w = _draw_weights(rng, D)
    hidden[_spike_rows(rng, s, 0.05)] *= np.float32(4.0)
    wq, wk, wv = w
    S = s.seq_len
    q = hidden @ wq
    k = hidden @ wk
    v = hidden @ wv
    steps, masks = [], []
    for t in range(T):
        mask = np.ones(S, dtype=np.uint8)
        if t > 0:
            n_drift = _rhu(0.10 * S)
            if drift == "visual_local":
                nv = n_2d + n_3d                                  # visual tokens are rows 0 .. nv-1 of the layout
                start = int(rng.integers(0, nv - n_drift + 1))
                rows = np.arange(start, start + n_drift)
            else:
                rows = np.sort(rng.choice(S, size=n_drift, replace=False))
            mask[:] = 0
            mask[rows] = 1
            hidden[rows] += rng.standard_normal((len(rows), D), dtype=np.float32) * np.float32(0.1)
            q[rows] = hidden[rows] @ wq
            k[rows] = hidden[rows] @ wk
            v[rows] = hidden[rows] @ wv
        steps.append(Tensors(hidden=round_to_dtype(hidden.copy(), dtype),
                             q=round_to_dtype(q.reshape(S, H, d).copy(), dtype),
                             k=round_to_dtype(k.reshape(S, H, d).copy(), dtype),
                             v=round_to_dtype(v.reshape(S, H, d).copy(), dtype)))
        masks.append(mask)
    return Workload("action_iteration" if drift == "all" else "action_iteration_" + drift, dtype, H, d, D,
                    MODE_ADAPTIVE, [s], steps, cold_start_full_keep=1, seed=seed, extra={"changed_rows": masks})


def small_workload(seed: int, *, batch=2, D=256, H=4, d=64, dtype="bf16", mode=MODE_ADAPTIVE,
                   n_txt=(5, 19), n_2d=(70, 130), n_3d=(150, 37), keep=(0.4, 0.3),
                   keep_fixed=(0.4, 0.3), steps=1, cold_start=0, text_first=False, scale_3d: float = 1.0,
                   spike_frac=0.05, n_kv_heads: int = 0) -> Workload:
    """Small ragged cases for parity tests: arbitrary segment lengths (several
    128-key tiles plus a ragged tail), optional [text | 2D | 3D] order, an
    optional scale on the 3D hidden rows (to move the feature-norm share), and
    optionally several action steps (10 % of rows drift by N(0, 0.1)).  `keep`
    cycles over samples as the adaptive total keep ratio; `keep_fixed` is the
    (2D, 3D) pair used in FIXED mode."""
    rng = np.random.default_rng(seed)
    samples, off = [], 0
    for b in range(batch):
        nt, n2, n3 = n_txt[b % len(n_txt)], n_2d[b % len(n_2d)], n_3d[b % len(n_3d)]
        kw = dict(keep_2d=keep_fixed[0], keep_3d=keep_fixed[1], keep_total=keep[b % len(keep)],
                  state_slot=b)
        if text_first:
            s = Sample(seq_off=off, off_txt=0, n_txt=nt, off_2d=nt, n_2d=n2,
                       off_3d=nt + n2, n_3d=n3, **kw)
        else:
            s = layout_2d_3d_txt(off, nt, n2, n3, **kw)
        samples.append(s)
        off += s.seq_len
    hidden = rng.standard_normal((off, D), dtype=np.float32)
    w = _draw_weights(rng, D, H * d, n_kv_heads * d)
    for s in samples:
        if spike_frac > 0:
            hidden[s.seq_off + _spike_rows(rng, s, spike_frac)] *= np.float32(4.0)
        if scale_3d != 1.0:
            hidden[s.seq_off + s.off_3d: s.seq_off + s.off_3d + s.n_3d] *= np.float32(scale_3d)
    out = []
    for t in range(steps):
        if t > 0:
            rows = np.sort(rng.choice(off, size=max(1, _rhu(0.10 * off)), replace=False))
            hidden[rows] += rng.standard_normal((len(rows), D), dtype=np.float32) * np.float32(0.1)
        out.append(_project(hidden.copy(), w, H, d, dtype, n_kv_heads))
    return Workload(f"small_{seed}", dtype, H, d, D, mode, samples, out,
                    cold_start_full_keep=cold_start, seed=seed,
                    extra={"n_kv_heads": n_kv_heads} if n_kv_heads else {})

def patch_workload(seed: int = 5, *, batch: int = 1, D=4096, H=32, d=128, dtype="bf16", n_txt=(32,),
                   n_patch=(256,), steps: int = 1, cold_start: int = 0, text_first: bool = False) -> Workload:
    """Paired-patch workload in the shape of the paper's host model (App. "MVLA Models": 256 image
    tokens from 16x16 patches + 256 point tokens): patch p owns 2D token p and 3D token p of its
    sample.  Per sample about 4 % of the patches are "target object" patches (both hidden rows x4),
    12 % "robot" patches (both rows x2), the rest background; one object patch has its 3D row
    scaled by 0.05 (a 3D response near zero); of the other patches 20 % have the 3D row scaled by 0.4
    and 20 % by 2.5, which moves the patch's 3D feature share across both synthetic thresholds.
    ``extra["rand_u"][t]`` holds, per action step, one uniform float32 in [0, 1) per patch (samples
    back to back): the random numbers of the background rule, drawn here and handed to whoever runs
    the method.  Later steps drift like the action-iteration workload."""
    rng = np.random.default_rng(seed)
    samples, off = [], 0
    for b in range(batch):
        nt, P = n_txt[b % len(n_txt)], n_patch[b % len(n_patch)]
        if text_first:
            smp = Sample(seq_off=off, off_txt=0, n_txt=nt, off_2d=nt, n_2d=P, off_3d=nt + P, n_3d=P,
                         state_slot=b)
        else:
            smp = layout_2d_3d_txt(off, nt, P, P, state_slot=b)
        samples.append(smp)
        off += smp.seq_len
    hidden = rng.standard_normal((off, D), dtype=np.float32)
    w = _draw_weights(rng, D, H * d)
    roles = []
    for smp in samples:
        P = smp.n_2d
        perm = rng.permutation(P)
        n_obj, n_rob = max(1, _rhu(0.04 * P)), max(1, _rhu(0.12 * P))
        obj, rob, rest = perm[:n_obj], perm[n_obj:n_obj + n_rob], perm[n_obj + n_rob:]
        r2, r3 = smp.seq_off + smp.off_2d, smp.seq_off + smp.off_3d
        for idx, g in ((obj, 4.0), (rob, 2.0)):
            hidden[r2 + idx] *= np.float32(g)
            hidden[r3 + idx] *= np.float32(g)
        hidden[r3 + obj[0]] *= np.float32(0.05)
        others = np.concatenate([obj[1:], rob, rest])
        sel = rng.permutation(len(others))
        n20 = _rhu(0.2 * len(others))
        hidden[r3 + others[sel[:n20]]] *= np.float32(0.4)
        hidden[r3 + others[sel[n20:2 * n20]]] *= np.float32(2.5)
        roles.append({"obj": np.sort(obj), "rob": np.sort(rob)})
    n_pat = sum(smp.n_2d for smp in samples)
    out, us = [], []
    for t in range(steps):
        if t > 0:
            rows = np.sort(rng.choice(off, size=max(1, _rhu(0.10 * off)), replace=False))
            hidden[rows] += rng.standard_normal((len(rows), D), dtype=np.float32) * np.float32(0.1)
        out.append(_project(hidden.copy(), w, H, d, dtype))
        us.append(rng.random(n_pat, dtype=np.float32))
    return Workload(f"patch_{seed}", dtype, H, d, D, MODE_PATCH, samples, out,
                    cold_start_full_keep=cold_start, seed=seed, extra={"rand_u": us, "roles": roles})


def patch_mla(seed: int = 5, batch: int = 1) -> Workload:
    """The paper's host-model shape: 32 text + 256 image + 256 point tokens, D = 4096, 32 x 128, bf16."""
    return patch_workload(seed, batch=batch)


def by_name(name: str, seed: Optional[int] = None) -> Workload:
    table = {"config1": config1_tiny, "config2": config2_single_frame,
             "config3": config3_multi_view, "config4": config4_batched,
             "config5": config5_action_iteration, "patch_mla": patch_mla}
    fn = table[name]
    return fn() if seed is None else fn(seed=seed)
