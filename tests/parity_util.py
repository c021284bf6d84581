"""Shared helpers for the GPU-vs-oracle parity tests."""
import numpy as np
import torch

import oracle
from paper_2604_09244_b200 import mvla
from paper_2604_09244_b200 import workloads as W

LENIENT = []                  # (workload, step, sample) of every check that took the on-a-threshold branch
SALIENCE_RTOL = 2e-3          # bf16 inputs, fp32 accumulate (stated tolerance of the salience scores)
SALIENCE_ATOL = 1e-12


def device_tensors(wl, step=0, device="cuda"):
    t = wl.steps[step]
    # with e4m3 q / k / v the hidden states stay bf16
    return {name: mvla.to_device(getattr(t, name), "bf16" if (wl.dtype == "fp8" and name == "hidden") else wl.dtype, device)
            for name in ("q", "k", "v", "hidden")}


def diag_records(out, batch):
    """Decode the int32 view of the diag records."""
    raw = out.diag.cpu().numpy()
    recs = []
    for b in range(batch):
        ints = raw[b, :8]
        flt = raw[b, 8:].view(np.float32)
        recs.append(dict(t=int(ints[0]), c_s1=int(ints[1]), c_s2=int(ints[2]), c_final=int(ints[3]),
                         budget=int(ints[4]), k_2d=int(ints[5]), k_3d=int(ints[6]),
                         x=flt[:4].copy(), mhat=flt[4:8].copy()))
    return recs


def assert_salience_close(got, ref, what="attn"):
    got = np.asarray(got, dtype=np.float64)
    err = np.abs(got - ref)
    bound = SALIENCE_RTOL * np.abs(ref) + SALIENCE_ATOL
    worst = int(np.argmax(err - bound))
    assert (err <= bound).all(), f"{what}: |g-o|={err[worst]:.3e} at {worst}, ref={ref[worst]:.6e}"


def check_kept_against_oracle(s, kept_gpu, k2, k3, z_ref, rtol=SALIENCE_RTOL):
    """Kept-set rule: with theta the oracle's k_m-th largest score of a modality, the GPU set holds
    every token with z > theta(1+rtol), none with z < theta(1-rtol), and exactly k_m tokens."""
    kept = np.asarray(kept_gpu)
    assert (np.diff(kept) > 0).all(), "kept positions must be strictly increasing"
    txt = kept[(kept >= s.off_txt) & (kept < s.off_txt + s.n_txt)]
    assert len(txt) == s.n_txt, "every text token is kept"
    for off, n, base, k in ((s.off_2d, s.n_2d, 0, k2), (s.off_3d, s.n_3d, s.n_2d, k3)):
        mine = kept[(kept >= off) & (kept < off + n)] - off
        assert len(mine) == k, f"modality kept count {len(mine)} != budget {k}"
        if k == 0 or k == n:
            continue
        z = z_ref[base:base + n]
        theta = np.sort(z)[::-1][k - 1]
        mask = np.zeros(n, dtype=bool)
        mask[mine] = True
        must = z > theta * (1 + rtol)
        never = z < theta * (1 - rtol)
        assert mask[must].all(), "a token clearly above the threshold was dropped"
        assert not mask[never].any(), "a token clearly below the threshold was kept"


def check_stagewise_exact(s, kept_gpu, k2, k3, ahat_gpu):
    """The oracle's normalise + select on the GPU's own smoothed scores must give the GPU's list."""
    z = oracle.normalise(np.asarray(ahat_gpu, dtype=np.float64), s.n_2d, s.n_3d)
    ref = oracle.select(z, s, k2, k3)
    assert np.array_equal(np.asarray(kept_gpu), ref), "selection differs from the oracle on identical scores"


def check_compaction(wl_tensors_np, dev_out, s, kept_gpu, row0, dtype):
    """Bit-exact rows: out[row0 + r] == in[seq_off + kept[r]] for hidden, k, v."""
    for name, out_t in (("hidden", dev_out.out_hidden), ("k", dev_out.out_k), ("v", dev_out.out_v)):
        if out_t is None:
            continue
        src = getattr(wl_tensors_np, name)
        n = len(kept_gpu)
        got = out_t[row0:row0 + n]
        if dtype == "fp8" and name != "hidden":
            got_bits = got.view(torch.uint8).cpu().numpy().reshape(n, -1)
            src_bits = W.e4m3_bits(src[s.seq_off + np.asarray(kept_gpu)]).reshape(n, -1)
            ref_bits = W.e4m3_bits(oracle.compact(src, s.seq_off, kept_gpu)).reshape(n, -1)
        elif dtype in ("bf16", "fp8"):
            got_bits = got.view(torch.int16).cpu().numpy().view(np.uint16).reshape(n, -1)
            src_bits = W.bf16_bits(src[s.seq_off + np.asarray(kept_gpu)]).reshape(n, -1)
            ref_bits = W.bf16_bits(oracle.compact(src, s.seq_off, kept_gpu)).reshape(n, -1)
        else:
            got_bits = got.cpu().numpy().view(np.uint32).reshape(n, -1)
            src_bits = src[s.seq_off + np.asarray(kept_gpu)].view(np.uint32).reshape(n, -1)
            ref_bits = oracle.compact(src, s.seq_off, kept_gpu).view(np.uint32).reshape(n, -1)
        assert np.array_equal(got_bits, src_bits), f"{name}: compacted rows are not bit-exact copies"
        assert np.array_equal(got_bits, ref_bits), f"{name}: differs from the oracle's compaction"


def run_and_check_step(ctx, wl, step, states, *, prune_point=0, flags=0, dev=None, samples=None, changed_rows=None):
    """One fused GPU step against the oracle on the same inputs.  `states`: oracle State per sample.
    Returns (gpu outputs, list of oracle StepResult)."""
    dev = dev or device_tensors(wl, step)
    samples = samples or wl.samples
    out = ctx.prune_step(prune_point, samples, wl.mode, dev["q"], dev["k"], dev["v"], dev["hidden"],
                         flags=flags, changed_rows=changed_rows)
    torch.cuda.synchronize()
    refs = oracle.run_workload_step(wl, step, states)
    offs = out.out_offsets.cpu().numpy()
    budgets = out.budgets.cpu().numpy()
    kept_all = out.kept_idx.cpu().numpy()
    attn = out.attn.cpu().numpy()
    ahat = out.ahat.cpu().numpy()
    zg = out.z.cpu().numpy()
    recs = diag_records(out, len(samples))
    vis = 0
    assert offs[0] == 0 and offs[-1] == out.total_kept
    for b, (s, ref) in enumerate(zip(samples, refs)):
        nv = s.n_vis
        assert_salience_close(attn[vis:vis + nv], ref.attn, f"sample {b} attn")
        assert_salience_close(ahat[vis:vis + nv], ref.ahat, f"sample {b} ahat")
        assert_salience_close(zg[vis:vis + nv], ref.z, f"sample {b} z")
        k2, k3 = int(budgets[b, 0]), int(budgets[b, 1])
        assert recs[b]["t"] == ref.t
        np.testing.assert_allclose(recs[b]["x"][2:], ref.x[2:], rtol=1e-4)
        np.testing.assert_allclose(recs[b]["mhat"][2:], ref.mhat[2:], rtol=1e-4)
        if wl.mode == W.MODE_ADAPTIVE:
            np.testing.assert_allclose(recs[b]["x"][:2], ref.x[:2], rtol=1e-4)
            np.testing.assert_allclose(recs[b]["mhat"][:2], ref.mhat[:2], rtol=1e-4)
        if not ref.near_gate:
            assert (recs[b]["c_s1"], recs[b]["c_s2"], recs[b]["c_final"]) == (ref.c_s1, ref.c_s2, ref.c_final) \
                or wl.mode == W.MODE_FIXED
        assert k2 + k3 == ref.k_2d + ref.k_3d, "total budget is host-computed and must match"
        if not (ref.near_half or ref.near_gate):
            assert (k2, k3) == (ref.k_2d, ref.k_3d), f"sample {b}: budgets {(k2, k3)} vs {(ref.k_2d, ref.k_3d)}"
        else:
            # An operand sits on a threshold (or B w on a half): either side may be right, but the decision
            # must still be the rules' decision.  The oracle's own gate and budget functions are fed with the
            # GPU's smoothed indicators and have to reproduce the GPU's sets and split exactly.
            LENIENT.append((wl.name, step, b))
            mh = recs[b]["mhat"].astype(np.float64)
            c1, c2, cf, _ = oracle.gates(mh, oracle.params_of(wl))
            cold = ref.t == 1 and wl.cold_start_full_keep
            if wl.mode == W.MODE_ADAPTIVE and not cold:
                assert (recs[b]["c_s1"], recs[b]["c_s2"], recs[b]["c_final"]) == (c1, c2, cf)
                g2, g3, _ = oracle.budget_adaptive(s, oracle.params_of(wl), float(mh[3]), cf)
                assert (k2, k3) == (g2, g3), f"sample {b}: split {(k2, k3)} is not the rules' split {(g2, g3)} of its own indicators"
            else:
                assert (k2, k3) == (ref.k_2d, ref.k_3d)
        n_kept = s.n_txt + k2 + k3
        assert offs[b + 1] - offs[b] == n_kept
        kept = kept_all[offs[b]:offs[b + 1]]
        if (k2, k3) == (ref.k_2d, ref.k_3d):
            check_kept_against_oracle(s, kept, k2, k3, ref.z)
        check_stagewise_exact(s, kept, k2, k3, ahat[vis:vis + nv])
        check_compaction(wl.steps[step], out, s, kept, int(offs[b]), wl.dtype)
        vis += nv
    return out, refs
