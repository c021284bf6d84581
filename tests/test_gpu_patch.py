"""GPU parity of the patch-by-patch path (Alg. 1 taken literally) against the fp64 oracle, through the C ABI."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
from paper_2604_09244_b200 import mvla
from paper_2604_09244_b200 import workloads as W
from parity_util import assert_salience_close, check_compaction, device_tensors

pytestmark = pytest.mark.gpu

X_RTOL = 1e-4          # shares that are ratios of sums of positive terms
ORTHO_ATOL = 2e-5      # the orthogonal share is a sum of differences: absolute error ~1e-6 observed
DECISION_TOL = 2e-4    # an oracle operand closer than this to its threshold may fall on either side


def patch_diag_records(t, batch):
    raw = t.cpu().numpy()
    out = []
    for b in range(batch):
        i, f = raw[b, :8], raw[b, 8:].view(np.float32)
        out.append(dict(t=int(i[0]), iters=int(i[1]), n_label=i[2:5].copy(), k_2d=int(i[5]), k_3d=int(i[6]),
                        n_out=int(i[7]), centre=f[:3].copy(), mu_2d=float(f[3]), mu_3d=float(f[4])))
    return out


def unpack_info(info):
    info = np.asarray(info)
    return info & 3, np.stack([(info >> 2) & 3, (info >> 4) & 3, (info >> 6) & 3], axis=1)


def check_x(got, ref, what):
    np.testing.assert_allclose(got[:, :3], ref[:, :3], rtol=X_RTOL, err_msg=what)
    assert (np.abs(got[:, 3] - ref[:, 3]) <= 2e-3 * np.abs(ref[:, 3]) + ORTHO_ATOL).all(), what


def fragile_patches(r, u, p):
    """Patches whose oracle decision has an operand within DECISION_TOL of its threshold."""
    xh = r.xhat
    near = lambda v, thr: np.abs(v - thr) <= DECISION_TOL
    f = near(xh[:, 1], p.tau_2d) | near(xh[:, 1], p.tau_3d)
    rob, obj = r.labels == oracle.LABEL_ROB, r.labels == oracle.LABEL_OBJ
    f |= rob & (near(xh[:, 3], r.mu_3d) | near(xh[:, 2], r.mu_2d))
    f |= obj & (near(xh[:, 2], p.obj_2d_min) | near(xh[:, 3], p.eps_3d))
    return f


def stagewise_exact(s, attn_g, xhat_g, u, labels_g, cand_g, kept_g, p, cold):
    """Decisions recomputed by the oracle's own functions from the GPU's fp32 values must match exactly."""
    P = s.n_2d
    mass = attn_g[:P].astype(np.float64) + attn_g[P:].astype(np.float64)
    labels, _, _, margin = oracle.kmeans1d(mass, p.kmeans_max_iter)
    if margin > 1e-12:
        assert np.array_equal(labels, labels_g), "K-Means labels differ on identical inputs"
    xh = xhat_g.astype(np.float64)
    mu2, mu3 = xh[:, 2].mean(), xh[:, 3].mean()
    both = oracle.SET_2D | oracle.SET_3D
    keep = []
    for q in range(P):
        c1 = oracle.patch_c_s1(xh[q, 1], p.tau_2d, p.tau_3d)
        c2 = oracle.patch_c_s2(int(labels_g[q]), xh[q, 2], xh[q, 3], mu2, mu3, float(u[q]), p)
        cf = both if cold else oracle.patch_fuse(c1, c2)
        if abs(xh[q, 2] - mu2) > 1e-9 and abs(xh[q, 3] - mu3) > 1e-9:
            assert tuple(cand_g[q]) == (c1, c2, cf), f"patch {q}: {tuple(cand_g[q])} vs {(c1, c2, cf)}"
        if cand_g[q, 2] & oracle.SET_2D:
            keep.append(s.off_2d + q)
        if cand_g[q, 2] & oracle.SET_3D:
            keep.append(s.off_3d + q)
    keep += list(range(s.off_txt, s.off_txt + s.n_txt))
    assert np.array_equal(np.sort(np.array(keep, dtype=np.int64)), np.asarray(kept_g)), "kept list differs from its masks"


def run_patch_step(ctx, wl, step, states, flags=0):
    dev = device_tensors(wl, step)
    u_np = wl.extra["rand_u"][step]
    u_dev = torch.from_numpy(u_np).cuda()
    out = ctx.prune_step(0, wl.samples, mvla.MODE_PATCH, dev["q"], dev["k"], dev["v"], dev["hidden"], flags=flags,
                         rand_u=u_dev)
    torch.cuda.synchronize()
    p = oracle.patch_params_of(wl)
    t = wl.steps[step]
    offs = out.out_offsets.cpu().numpy()
    counts = out.budgets.cpu().numpy()
    kept_all = out.kept_idx.cpu().numpy()
    attn = out.attn.cpu().numpy()
    xg, xhg = out.patch_x.cpu().numpy(), out.patch_xhat.cpu().numpy()
    lab_all, cand_all = unpack_info(out.patch_info.cpu().numpy())
    recs = patch_diag_records(out.patch_diag, len(wl.samples))
    assert offs[0] == 0 and out.total_kept == wl.total_rows
    vis = pat = 0
    n_checked = n_patches = 0
    for b, s in enumerate(wl.samples):
        P = s.n_2d
        u = u_np[pat:pat + P]
        r = oracle.patch_step(t.q, t.k, t.hidden, wl.n_heads, wl.head_dim, wl.d_model, s, u, p, states[b])
        a_g = attn[vis:vis + 2 * P]
        assert_salience_close(a_g, r.attn, f"sample {b} attn")
        check_x(xg[pat:pat + P], r.x, f"sample {b} x")
        check_x(xhg[pat:pat + P], r.xhat, f"sample {b} xhat")
        labels_g, cand_g = lab_all[pat:pat + P], cand_all[pat:pat + P]
        kept = kept_all[offs[b]:offs[b + 1]]
        k2, k3 = int(counts[b, 0]), int(counts[b, 1])
        assert len(kept) == s.n_txt + k2 + k3 == recs[b]["n_out"]
        assert (np.diff(kept) > 0).all()
        assert recs[b]["t"] == r.t
        cold = r.t == 1 and wl.cold_start_full_keep
        stagewise_exact(s, a_g, xhg[pat:pat + P], u, labels_g, cand_g, kept, p, cold)
        # against the oracle's own run: classes when no point sits near a class boundary, then every
        # patch whose decision is not within tolerance of a threshold
        mass_err = np.abs((a_g[:P].astype(np.float64) + a_g[P:]) - (r.attn[:P] + r.attn[P:])).max()
        if r.kmeans_margin > 8 * mass_err:
            assert np.array_equal(labels_g, r.labels), f"sample {b}: K-Means classes differ"
            assert recs[b]["iters"] == r.iters
            np.testing.assert_allclose(recs[b]["centre"], r.centre, rtol=1e-4)
            solid = ~fragile_patches(r, u, p)
            assert np.array_equal(cand_g[solid], r.cand[solid]), f"sample {b}: candidate sets differ"
            n_checked += int(solid.sum())
            if solid.all():
                assert np.array_equal(kept, r.kept_idx) and (k2, k3) == (r.k_2d, r.k_3d)
        n_patches += P
        np.testing.assert_allclose([recs[b]["mu_2d"], recs[b]["mu_3d"]], [r.mu_2d, r.mu_3d], rtol=1e-4, atol=1e-5)
        check_compaction(t, out, s, kept, int(offs[b]), wl.dtype)
        vis += 2 * P
        pat += P
    assert offs[-1] == sum(s.n_txt for s in wl.samples) + counts.sum()
    return out, n_checked, n_patches


@pytest.mark.parametrize("dtype,path", [("fp32", mvla.SALIENCE_AUTO), ("bf16", mvla.SALIENCE_AUTO), ("bf16", mvla.SALIENCE_FMA)])
@pytest.mark.parametrize("text_first", [False, True])
def test_patch_indicators_small_ragged(dtype, path, text_first):
    wl = W.patch_workload(11, batch=3, D=256, H=4, d=64, dtype=dtype, n_txt=(5, 19, 33), n_patch=(70, 150, 129),
                          text_first=text_first)
    ctx = mvla.context_for(wl, salience_path=path)
    dev = device_tensors(wl)
    attn, x = ctx.patch_indicators(wl.samples, dev["q"], dev["k"], dev["hidden"])
    torch.cuda.synchronize()
    attn, x = attn.cpu().numpy(), x.cpu().numpy()
    t = wl.steps[0]
    vis = pat = 0
    for s in wl.samples:
        P = s.n_2d
        alpha = oracle.attention(t.q, t.k, wl.n_heads, wl.head_dim, s)
        ref = oracle.patch_indicators(alpha.reshape(-1, 2 * P), oracle.l1norm(t.hidden, wl.d_model, s))
        assert_salience_close(attn[vis:vis + 2 * P], alpha.mean(axis=(0, 1)))
        check_x(x[pat:pat + P], ref, "x")
        vis += 2 * P
        pat += P
    ctx.close()


def test_patch_select_on_given_inputs_is_exact():
    # the decision stage alone, on inputs that both sides read as the same fp32 values
    rng = np.random.default_rng(2)
    samples = [W.layout_2d_3d_txt(0, 7, 300, 300, state_slot=0),
               W.Sample(seq_off=607, off_txt=0, n_txt=3, off_2d=3, n_2d=41, off_3d=44, n_3d=41, state_slot=1),
               W.layout_2d_3d_txt(692, 2, 1024, 1024, state_slot=2)]
    ctx = mvla.PruneContext(dtype=torch.bfloat16, n_heads=4, head_dim=64, d_model=256, max_batch=3, max_text=8,
                            max_2d=1024, max_3d=1024, tau_2d=0.35, tau_3d=0.65, cold_start_full_keep=0, patch_path=1)
    p = oracle.c_patch_params(tau_2d=0.35, tau_3d=0.65, cold_start_full_keep=0)
    nP = sum(s.n_2d for s in samples)
    states = [oracle.PatchState(s.n_2d) for s in samples]
    for step in range(3):
        attn = (rng.random(2 * nP) ** 6).astype(np.float32)
        x = rng.random((nP, 4)).astype(np.float32)
        u = rng.random(nP).astype(np.float32)
        out = ctx.patch_select(0, samples, torch.from_numpy(attn).cuda(), torch.from_numpy(x).cuda(),
                               torch.from_numpy(u).cuda())
        torch.cuda.synchronize()
        offs, counts, kept_all = out.out_offsets.cpu().numpy(), out.budgets.cpu().numpy(), out.kept_idx.cpu().numpy()
        lab_all, cand_all = unpack_info(out.patch_info.cpu().numpy())
        xh_all = out.patch_xhat.cpu().numpy()
        vis = pat = 0
        for b, s in enumerate(samples):
            P = s.n_2d
            a_s, x_s, u_s = attn[vis:vis + 2 * P], x[pat:pat + P], u[pat:pat + P]
            r = oracle.patch_select(a_s, x_s, u_s, s, p, states[b])
            kept = kept_all[offs[b]:offs[b + 1]]
            np.testing.assert_allclose(xh_all[pat:pat + P], r.xhat, rtol=2e-6, atol=1e-7)
            stagewise_exact(s, a_s, xh_all[pat:pat + P], u_s, lab_all[pat:pat + P], cand_all[pat:pat + P], kept, p, False)
            if step == 0:                       # X^_1 = X_1 on both sides: every decision is on identical numbers
                assert np.array_equal(lab_all[pat:pat + P], r.labels)
                assert np.array_equal(cand_all[pat:pat + P], r.cand)
                assert np.array_equal(kept, r.kept_idx)
                assert (int(counts[b, 0]), int(counts[b, 1])) == (r.k_2d, r.k_3d)
            vis += 2 * P
            pat += P
        assert offs[0] == 0 and offs[-1] == sum(s.n_txt for s in samples) + counts.sum()
    ctx.close()


@pytest.mark.parametrize("seed", [5, 6])
def test_patch_step_host_model_shape(seed):
    wl = W.patch_mla(seed)                       # 32 text + 256 image + 256 point tokens, D = 4096, 32 x 128, bf16
    ctx = mvla.context_for(wl)
    out, n_checked, n_patches = run_patch_step(ctx, wl, 0, [oracle.PatchState(s.n_2d) for s in wl.samples])
    assert n_checked >= 0.9 * n_patches
    ctx.close()


def test_patch_step_ragged_batch_three_action_steps_with_cold_start():
    wl = W.patch_workload(21, batch=3, D=512, H=4, d=128, n_txt=(12, 30, 64), n_patch=(100, 256, 37), steps=3,
                          cold_start=1)
    ctx = mvla.context_for(wl)
    states = [oracle.PatchState(s.n_2d) for s in wl.samples]
    out, _, _ = run_patch_step(ctx, wl, 0, states)
    counts = out.budgets.cpu().numpy()
    assert all(tuple(counts[b]) == (s.n_2d, s.n_3d) for b, s in enumerate(wl.samples))      # t = 1 keeps everything
    checked = total = 0
    for step in (1, 2):
        out, c, n = run_patch_step(ctx, wl, step, states)
        checked += c
        total += n
    assert checked >= 0.8 * total
    assert out.budgets.cpu().numpy().sum() < sum(2 * s.n_2d for s in wl.samples)
    ctx.close()


def test_patch_step_fp32_and_more_samples_than_one_launch_carries():
    wl = W.patch_workload(33, batch=35, D=128, H=2, d=64, dtype="fp32", n_txt=(3, 9), n_patch=(20, 45, 33))
    ctx = mvla.context_for(wl)
    run_patch_step(ctx, wl, 0, [oracle.PatchState(s.n_2d) for s in wl.samples])
    ctx.close()


def test_patch_path_error_codes():
    wl = W.patch_workload(1, batch=1, D=128, H=2, d=64, n_txt=(4,), n_patch=(16,))
    dev = device_tensors(wl)
    u = torch.from_numpy(wl.extra["rand_u"][0]).cuda()
    plain = mvla.context_for(wl, patch_path=0)
    with pytest.raises(mvla.MvlaError) as e:
        plain.prune_step(0, wl.samples, mvla.MODE_PATCH, dev["q"], dev["k"], dev["v"], dev["hidden"], rand_u=u)
    assert e.value.code == mvla.ERR_UNSUPPORTED
    plain.close()
    ctx = mvla.context_for(wl)
    with pytest.raises(mvla.MvlaError) as e:      # the draws of the background rule are an input
        ctx.prune_step(0, wl.samples, mvla.MODE_PATCH, dev["q"], dev["k"], dev["v"], dev["hidden"])
    assert e.value.code == mvla.ERR_INVALID_ARG
    odd = [W.layout_2d_3d_txt(0, 4, 15, 13)]
    with pytest.raises(mvla.MvlaError) as e:      # a patch owns one token of each modality
        ctx.prune_step(0, odd, mvla.MODE_PATCH, dev["q"], dev["k"], dev["v"], dev["hidden"], rand_u=u)
    assert e.value.code == mvla.ERR_INVALID_ARG
    out = ctx.prune_step(0, wl.samples, mvla.MODE_PATCH, dev["q"], dev["k"], dev["v"], dev["hidden"], rand_u=u)
    torch.cuda.synchronize()
    assert int(out.out_offsets[-1]) <= wl.total_rows
    ctx.close()


def test_pipelined_patch_steps_match_serial_steps():
    # MVLA_FLAG_INPUTS_STABLE lets neighbouring steps overlap inside the library; results must not change.
    # Two episodes (state slots 0-1 and 2-3) interleaved over four action steps, seven rotating output sets.
    import dataclasses
    wl = W.patch_workload(27, batch=2, D=256, H=4, d=128, n_txt=(10, 32), n_patch=(130, 256), steps=4, cold_start=1)
    devs = [device_tensors(wl, t) for t in range(4)]
    us = [torch.from_numpy(wl.extra["rand_u"][t]).cuda() for t in range(4)]
    episodes = [wl.samples, [dataclasses.replace(s, state_slot=s.state_slot + 2) for s in wl.samples]]

    def run(flag):
        ctx = mvla.context_for(wl, n_state_slots=4)
        outs = [ctx.alloc_outputs(wl.samples, patch=True) for _ in range(7)]
        seen = []
        i = 0
        for t in range(4):
            for ep in episodes:
                o = outs[i % 7]
                ctx.prune_step(0, ep, mvla.MODE_PATCH, devs[t]["q"], devs[t]["k"], devs[t]["v"], devs[t]["hidden"],
                               flags=flag, out=o, rand_u=us[t])
                if i % 7 == 6 or (t == 3 and ep is episodes[-1]):
                    torch.cuda.synchronize()
                # results are complete in stream order: reading them on the same stream needs no sync
                n = int(o.out_offsets[-1])
                seen.append((o.out_offsets.cpu().numpy().copy(), o.kept_idx[:n].cpu().numpy().copy(),
                             o.budgets.cpu().numpy().copy(), o.patch_info.cpu().numpy().copy(),
                             o.out_hidden[:n].float().cpu().numpy().copy()))
                i += 1
        torch.cuda.synchronize()
        ctx.close()
        return seen

    serial, piped = run(0), run(mvla.FLAG_INPUTS_STABLE)
    assert len(serial) == len(piped) == 8
    for a, b in zip(serial, piped):
        for x, y in zip(a, b):
            assert np.array_equal(x, y)
    assert serial[0][2].sum() > serial[-1][2].sum()      # the cold-start step kept everything, later steps prune


def test_patch_step_leaves_the_bytes_behind_its_outputs_alone():
    # the row copy of this path is launched over the capacity (the row count is known only on the device):
    # rows and list entries past out_offsets[batch] must keep the pattern they were filled with
    wl = W.patch_workload(17, batch=3, D=256, H=4, d=128, n_txt=(7, 20, 33), n_patch=(90, 200, 130))
    ctx = mvla.context_for(wl)
    dev = device_tensors(wl)
    u = torch.from_numpy(wl.extra["rand_u"][0]).cuda()
    out = ctx.alloc_outputs(wl.samples, extras=True, patch=True)
    for t in (out.out_hidden, out.out_k, out.out_v):
        t.view(torch.int16).fill_(0x5A5A)
    out.kept_idx.fill_(-77)
    ctx.prune_step(0, wl.samples, mvla.MODE_PATCH, dev["q"], dev["k"], dev["v"], dev["hidden"], rand_u=u, out=out,
                   flags=mvla.FLAG_RESET_STATE)
    torch.cuda.synchronize()
    n = int(out.out_offsets[-1])
    assert 0 < n < out.kept_idx.numel()
    assert bool((out.kept_idx[n:] == -77).all()), "list entries past the total were written"
    for t in (out.out_hidden, out.out_k, out.out_v):
        assert bool((t[n:].view(torch.int16) == 0x5A5A).all()), "rows past the total were written"
    ctx.close()


@pytest.mark.parametrize("batch,n_txt,n_patch", [(1, (20,), (1000,)), (2, (48, 9), (600, 515)), (32, (7, 12, 5), (24, 40, 33))])
def test_patch_step_in_one_tail_kernel_at_the_edges_of_its_shapes(batch, n_txt, n_patch):
    # the serial step's single tail kernel: more patches than the selecting CTA has threads (several patches per
    # thread, two key tiles per scoring CTA), more than 32 text queries, and as many samples as one launch carries
    wl = W.patch_workload(57, batch=batch, D=128, H=2, d=64, n_txt=n_txt, n_patch=n_patch, steps=2)
    ctx = mvla.context_for(wl)
    states = [oracle.PatchState(s.n_2d) for s in wl.samples]
    checked = total = 0
    for step in (0, 1):
        _, c, n = run_patch_step(ctx, wl, step, states)
        checked += c
        total += n
    assert checked >= 0.8 * total
    ctx.close()
