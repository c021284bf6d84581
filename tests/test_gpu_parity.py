"""GPU parity: the CUDA library, called through its C ABI, against the fp64 CPU oracle on the same
seeded inputs.  Integer results (kept indices given identical scores, compacted rows) must be
bit-exact; salience scores within 2e-3 relative (bf16 inputs, fp32 accumulate)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_09244_b200 import mvla
from paper_2604_09244_b200 import workloads as W
from parity_util import (SALIENCE_RTOL, assert_salience_close, check_compaction, check_kept_against_oracle,
                         check_stagewise_exact, device_tensors, diag_records, run_and_check_step)

pytestmark = pytest.mark.gpu


# ------------------------------------------------------------------ compaction
@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_compact_bit_exact_ragged(dtype):
    wl = W.small_workload(21, batch=3, D=264 if dtype == "bf16" else 260, H=3, d=64, dtype=dtype,
                          n_txt=(5, 19, 1), n_2d=(70, 130, 3), n_3d=(150, 37, 9))
    ctx = mvla.context_for(wl)
    dev = device_tensors(wl)
    rng = np.random.default_rng(0)
    kept, offs = [], [0]
    for s in wl.samples:
        k = np.sort(rng.choice(s.seq_len, size=int(rng.integers(1, s.seq_len + 1)), replace=False))
        kept.append(k.astype(np.int32))
        offs.append(offs[-1] + len(k))
    kept_d = torch.from_numpy(np.concatenate(kept)).cuda()
    offs_d = torch.tensor(offs, dtype=torch.int32).cuda()
    oh, ok, ov = ctx.compact(wl.samples, kept_d, offs_d, offs[-1], dev["hidden"], dev["k"], dev["v"])
    torch.cuda.synchronize()

    class Out:
        out_hidden, out_k, out_v = oh, ok, ov
    for b, s in enumerate(wl.samples):
        check_compaction(wl.steps[0], Out, s, kept[b], offs[b], dtype)
    # a skipped pair stays untouched
    oh2, ok2, ov2 = ctx.compact(wl.samples, kept_d, offs_d, offs[-1], None, dev["k"], None)
    assert oh2 is None and ov2 is None
    torch.cuda.synchronize()
    assert torch.equal(ok2, ok)
    ctx.close()


# ------------------------------------------------------------------ selection on given scores
def test_select_exact_with_ties_and_edge_budgets():
    rng = np.random.default_rng(5)
    cases = [(40, 50, 0.5, 0.5), (1, 300, 1.0, 0.01), (257, 0, 0.3, 0.3), (0, 129, 0.0, 0.7),
             (1000, 1500, 0.1, 0.9), (64, 64, 0.0, 0.0), (33, 95, 1.0, 1.0)]
    for n2, n3, k2r, k3r in cases:
        s = W.layout_2d_3d_txt(0, 7, n2, n3, keep_2d=k2r, keep_3d=k3r)
        ctx = mvla.PruneContext(dtype=torch.float32, n_heads=2, head_dim=64, d_model=64, max_batch=1,
                                max_text=8, max_2d=max(n2, 1), max_3d=max(n3, 1), cold_start_full_keep=0)
        # few distinct values -> many exact ties at the k-th boundary
        attn = rng.integers(1, 6, size=n2 + n3).astype(np.float32)
        attn /= attn.sum()
        out = ctx.select(0, [s], mvla.MODE_FIXED, torch.from_numpy(attn).cuda())
        torch.cuda.synchronize()
        k2, k3 = out.budgets.cpu().numpy()[0]
        assert (k2, k3) == oracle.budget_fixed(s)
        offs = out.out_offsets.cpu().numpy()
        kept = out.kept_idx.cpu().numpy()[:offs[1]]
        ref = oracle.select(oracle.normalise(attn.astype(np.float64), n2, n3), s, int(k2), int(k3))
        assert np.array_equal(kept, ref), (n2, n3)
        assert np.array_equal(out.ahat.cpu().numpy(), attn)
        ctx.close()


def test_select_text_first_and_negative_scores():
    s = W.Sample(seq_off=0, off_txt=0, n_txt=3, off_2d=3, n_2d=200, off_3d=203, n_3d=77,
                 keep_2d=0.25, keep_3d=0.5)
    ctx = mvla.PruneContext(dtype=torch.float32, n_heads=2, head_dim=64, d_model=64, max_batch=1, max_text=8,
                            max_2d=200, max_3d=77, cold_start_full_keep=0)
    rng = np.random.default_rng(1)
    attn = rng.standard_normal(277).astype(np.float32)          # the ordering must hold for any sign
    out = ctx.select(0, [s], mvla.MODE_FIXED, torch.from_numpy(attn).cuda())
    torch.cuda.synchronize()
    kept = out.kept_idx.cpu().numpy()[:out.out_offsets.cpu().numpy()[1]]
    ref = oracle.select(attn.astype(np.float64), s, 50, 39)
    assert np.array_equal(kept, ref)
    ctx.close()


# ------------------------------------------------------------------ salience
@pytest.mark.parametrize("dtype,path", [("fp32", mvla.SALIENCE_AUTO), ("bf16", mvla.SALIENCE_FMA),
                                        ("bf16", mvla.SALIENCE_AUTO)])
@pytest.mark.parametrize("text_first", [False, True])
def test_salience_small_ragged(dtype, path, text_first):
    wl = W.small_workload(31, batch=3, D=256, H=4, d=64 if dtype == "fp32" else 128, dtype=dtype,
                          n_txt=(5, 19, 33), n_2d=(70, 130, 1), n_3d=(150, 37, 300), text_first=text_first)
    ctx = mvla.context_for(wl, salience_path=path)
    dev = device_tensors(wl)
    attn, l1 = ctx.salience(wl.samples, dev["q"], dev["k"], dev["hidden"])
    torch.cuda.synchronize()
    attn, l1 = attn.cpu().numpy(), l1.cpu().numpy()
    t = wl.steps[0]
    vis = 0
    for s in wl.samples:
        ref = oracle.salience(t.q, t.k, wl.n_heads, wl.head_dim, s)
        assert_salience_close(attn[vis:vis + s.n_vis], ref)
        assert abs(attn[vis:vis + s.n_vis].sum() - 1.0) < 1e-4
        np.testing.assert_allclose(l1[vis:vis + s.n_vis], oracle.l1norm(t.hidden, wl.d_model, s), rtol=1e-5)
        vis += s.n_vis
    ctx.close()


def test_salience_many_tiles_and_max_text():
    # 2500 keys -> 21 tiles -> 3 tiles per CTA in a cluster of 7; 64 text queries (the maximum)
    wl = W.small_workload(32, batch=1, D=128, H=2, d=128, dtype="bf16", n_txt=(64,), n_2d=(1100,), n_3d=(1400,))
    for path in (mvla.SALIENCE_AUTO, mvla.SALIENCE_FMA):
        ctx = mvla.context_for(wl, salience_path=path)
        dev = device_tensors(wl)
        attn, _ = ctx.salience(wl.samples, dev["q"], dev["k"])
        torch.cuda.synchronize()
        t = wl.steps[0]
        assert_salience_close(attn.cpu().numpy(), oracle.salience(t.q, t.k, 2, 128, wl.samples[0]))
        ctx.close()


def test_tensor_core_and_fma_paths_agree():
    wl = W.config2_single_frame(seed=7)
    dev = device_tensors(wl)
    res = []
    for path in (mvla.SALIENCE_AUTO, mvla.SALIENCE_FMA):
        ctx = mvla.context_for(wl, salience_path=path)
        attn, _ = ctx.salience(wl.samples, dev["q"], dev["k"])
        torch.cuda.synchronize()
        res.append(attn.cpu().numpy())
        ctx.close()
    np.testing.assert_allclose(res[0], res[1], rtol=1e-4, atol=1e-9)


# ------------------------------------------------------------------ the fused step on the five workloads
def _fresh_states(wl):
    return [oracle.State(s.n_vis) for s in wl.samples]


def test_step_config1_tiny_fp32():
    wl = W.config1_tiny()
    ctx = mvla.context_for(wl)
    out, refs = run_and_check_step(ctx, wl, 0, _fresh_states(wl))
    kept = out.kept_idx.cpu().numpy()[:out.total_kept]
    assert np.array_equal(kept, refs[0].kept_idx)
    ctx.close()


@pytest.mark.parametrize("seed", [1, 11, 12, 13])
def test_step_config2_single_frame(seed):
    wl = W.config2_single_frame(seed=seed)
    ctx = mvla.context_for(wl)
    out, refs = run_and_check_step(ctx, wl, 0, _fresh_states(wl))
    assert tuple(out.budgets.cpu().numpy()[0]) == (102, 154)
    assert out.total_kept == 288
    ctx.close()


@pytest.mark.parametrize("seed", [2, 21])
def test_step_config3_multi_view_two_points(seed):
    wl = W.config3_multi_view(seed=seed)
    ctx = mvla.context_for(wl, n_prune_points=2)
    out, refs = run_and_check_step(ctx, wl, 0, _fresh_states(wl), prune_point=0)
    assert out.total_kept == 48 + 448
    # second point: the generator re-projects the rows the ORACLE kept at the first point
    r = refs[0]
    wl2 = W.config3_second_point(wl, r.kept_idx, r.k_2d, r.k_3d)
    out2, refs2 = run_and_check_step(ctx, wl2, 0, _fresh_states(wl2), prune_point=1)
    assert out2.total_kept == 48 + 112
    ctx.close()


def test_step_config4_batched_serving():
    wl = W.config4_batched()
    ctx = mvla.context_for(wl)
    out, refs = run_and_check_step(ctx, wl, 0, _fresh_states(wl))
    offs = out.out_offsets.cpu().numpy()
    assert len(offs) == 17 and (np.diff(offs) > 0).all()
    ctx.close()


def test_step_config5_action_iteration():
    wl = W.config5_action_iteration()
    ctx = mvla.context_for(wl)
    states = _fresh_states(wl)
    s = wl.samples[0]
    for t in range(len(wl.steps)):
        out, refs = run_and_check_step(ctx, wl, t, states, flags=mvla.FLAG_RESET_STATE if t == 0 else 0)
        if t == 0:
            assert out.total_kept == s.seq_len                       # cold start keeps everything
            assert np.array_equal(out.kept_idx.cpu().numpy()[:s.seq_len], np.arange(s.seq_len))
        else:
            assert out.total_kept == s.n_txt + 384
        assert diag_records(out, 1)[0]["t"] == t + 1
    ctx.close()


def test_step_small_ragged_batch_with_state_and_dry_run():
    wl = W.small_workload(41, batch=3, D=256, H=4, d=128, dtype="bf16", n_txt=(5, 19, 33),
                          n_2d=(70, 130, 260), n_3d=(150, 37, 300), keep=(0.4, 0.3, 0.55), steps=9,
                          cold_start=1)
    ctx = mvla.context_for(wl)
    states = _fresh_states(wl)
    for t in range(9):                                                # crosses the Eq. 8 -> Eq. 9 switch at t = 7
        out, refs = run_and_check_step(ctx, wl, t, states)
        if t == 3:                                                    # a dry run leaves state and t untouched
            dev = device_tensors(wl, t)
            dry = ctx.prune_step(0, wl.samples, wl.mode, dev["q"], dev["k"], dev["v"], dev["hidden"],
                                 flags=mvla.FLAG_NO_STATE_UPDATE)
            torch.cuda.synchronize()
            assert diag_records(dry, 3)[0]["t"] == 5
    ctx.close()


@pytest.mark.parametrize("scale,expect", [(0.05, mvla.SET_2D), (0.136, mvla.SET_2D | mvla.SET_3D), (0.30, mvla.SET_3D)])
def test_paper_default_thresholds_all_three_branches(scale, expect):
    # 3D hidden rows scaled by s give a feature-norm share of about s/(1+s): 0.048, 0.12, 0.23 against
    # the paper's default thresholds 0.08 / 0.20
    wl = W.small_workload(51, batch=1, D=512, H=4, d=128, dtype="bf16", n_txt=(9,), n_2d=(200,), n_3d=(280,),
                          keep=(0.35,), scale_3d=scale, spike_frac=0.0)
    wl.tau_2d, wl.tau_3d = 0.08, 0.20
    ctx = mvla.context_for(wl)
    out, refs = run_and_check_step(ctx, wl, 0, _fresh_states(wl))
    assert diag_records(out, 1)[0]["c_s1"] == expect == refs[0].c_s1
    ctx.close()


def test_results_are_deterministic():
    wl = W.config2_single_frame(seed=3)
    ctx = mvla.context_for(wl)
    dev = device_tensors(wl)
    outs = []
    for _ in range(3):
        o = ctx.prune_step(0, wl.samples, wl.mode, dev["q"], dev["k"], dev["v"], dev["hidden"],
                           flags=mvla.FLAG_RESET_STATE)
        torch.cuda.synchronize()
        n = o.total_kept                                            # rows past it are unwritten scratch
        outs.append((o.attn.clone(), o.kept_idx[:n].clone(), o.out_hidden[:n].clone(), o.out_k[:n].clone()))
    for a in outs[1:]:
        assert all(torch.equal(x, y) for x, y in zip(a, outs[0]))
    ctx.close()


# ------------------------------------------------------------------ boundary behaviour
def test_error_codes_never_fault():
    wl = W.small_workload(61, batch=2, D=256, H=4, d=128, dtype="bf16")
    ctx = mvla.context_for(wl)
    dev = device_tensors(wl)
    good = list(wl.samples)

    def code(fn):
        with pytest.raises(mvla.MvlaError) as e:
            fn()
        return e.value.code

    import copy
    bad = copy.deepcopy(good); bad[0].n_txt = 0
    assert code(lambda: ctx.salience(bad, dev["q"], dev["k"])) == mvla.ERR_INVALID_ARG
    bad = copy.deepcopy(good); bad[0].off_3d = bad[0].off_2d          # overlapping segments
    assert code(lambda: ctx.salience(bad, dev["q"], dev["k"])) == mvla.ERR_INVALID_ARG
    bad = copy.deepcopy(good); bad[1].n_2d = 10 ** 6
    assert code(lambda: ctx.salience(bad, dev["q"], dev["k"])) == mvla.ERR_CAPACITY
    bad = copy.deepcopy(good); bad[1].seq_off = 10 ** 6               # beyond the rows given
    assert code(lambda: ctx.salience(bad, dev["q"], dev["k"])) == mvla.ERR_INVALID_ARG
    bad = copy.deepcopy(good); bad[1].state_slot = bad[0].state_slot  # two writers of one state
    assert code(lambda: ctx.prune_step(0, bad, wl.mode, dev["q"], dev["k"], dev["v"], dev["hidden"])) == mvla.ERR_STATE
    assert code(lambda: ctx.prune_step(3, good, wl.mode, dev["q"], dev["k"], dev["v"], dev["hidden"])) == mvla.ERR_STATE
    assert code(lambda: ctx.prune_step(0, good, wl.mode, dev["q"], dev["k"], dev["v"], dev["hidden"], flags=8)) == mvla.ERR_INVALID_ARG
    assert code(lambda: ctx.prune_step(0, good * 2, wl.mode, dev["q"], dev["k"], dev["v"], dev["hidden"])) == mvla.ERR_CAPACITY
    misaligned = dev["q"].view(-1)[1:1 + dev["q"].numel() - 8].contiguous()
    # .contiguous() of a slice is a fresh allocation, so build a truly misaligned pointer by hand
    import ctypes as C
    cs = mvla.c_samples(good)
    rc = ctx._lib.mvla_salience(ctx._h, 2, cs, dev["q"].data_ptr() + 2, dev["k"].data_ptr(), None,
                                dev["q"].shape[0], torch.empty(1000, device="cuda").data_ptr(), None, 0)
    assert rc == mvla.ERR_INVALID_ARG
    # the context is still usable afterwards
    ctx.prune_step(0, good, wl.mode, dev["q"], dev["k"], dev["v"], dev["hidden"])
    torch.cuda.synchronize()
    ctx.close()
    with pytest.raises(mvla.MvlaError) as e:
        mvla.PruneContext(dtype=torch.bfloat16, n_heads=4, head_dim=48, d_model=256, max_batch=1, max_text=8,
                          max_2d=8, max_3d=8)
    assert e.value.code == mvla.ERR_UNSUPPORTED


def test_inputs_stable_flag_changes_timing_only():
    # back-to-back steps on rotating buffers, with and without the promise that the inputs are not
    # produced by the preceding work: identical results, step after step
    wls = [W.config2_single_frame(seed=s) for s in (31, 32, 33)]
    wl = wls[0]
    ctx = mvla.context_for(wl)
    devs = [device_tensors(w) for w in wls]
    ref = []
    for d in devs:
        o = ctx.prune_step(0, wl.samples, wl.mode, d["q"], d["k"], d["v"], d["hidden"], flags=mvla.FLAG_RESET_STATE)
        torch.cuda.synchronize()
        n = o.total_kept
        ref.append((o.attn.clone(), o.kept_idx[:n].clone(), o.out_hidden[:n].clone(), o.out_v[:n].clone()))
    outs = [ctx.alloc_outputs(wl.samples, extras=True) for _ in range(3)]
    for rep in range(30):                                   # no synchronisation between the steps
        i = rep % 3
        d = devs[i]
        ctx.prune_step(0, wl.samples, wl.mode, d["q"], d["k"], d["v"], d["hidden"],
                       flags=mvla.FLAG_RESET_STATE | mvla.FLAG_INPUTS_STABLE, out=outs[i])
    torch.cuda.synchronize()
    for i in range(3):
        o, n = outs[i], len(ref[i][1])
        got = (o.attn, o.kept_idx[:n], o.out_hidden[:n], o.out_v[:n])
        assert all(torch.equal(x, y) for x, y in zip(got, ref[i]))
    ctx.close()


def test_pipelined_steps_with_state_match_serial_steps():
    # action steps with carry-over, enqueued back to back without synchronisation and with the
    # stable-inputs promise (scoring, selection and row copy of neighbouring steps overlap), against the
    # same steps run one at a time: identical bits, including when output buffers are reused
    wl = W.small_workload(43, batch=3, D=256, H=4, d=128, dtype="bf16", n_txt=(5, 19, 33), n_2d=(70, 130, 260),
                          n_3d=(150, 37, 300), keep=(0.4, 0.3, 0.55), steps=10, cold_start=1)
    devs = [device_tensors(wl, t) for t in range(10)]

    def run(flag, n_out, sync):
        ctx = mvla.context_for(wl)
        outs = [ctx.alloc_outputs(wl.samples, extras=True) for _ in range(n_out)]
        res = []
        for t, d in enumerate(devs):
            o = ctx.prune_step(0, wl.samples, wl.mode, d["q"], d["k"], d["v"], d["hidden"],
                               flags=flag | (mvla.FLAG_RESET_STATE if t == 0 else 0), out=outs[t % n_out])
            if sync:
                torch.cuda.synchronize()
            res.append((o.total_kept, t % n_out))
        torch.cuda.synchronize()
        snap = [None] * 10
        for t in range(10 - n_out, 10):                       # the last n_out steps are still in their buffers
            o, n = outs[t % n_out], res[t][0]
            snap[t] = (o.ahat.clone(), o.kept_idx[:n].clone(), o.budgets.clone(), o.out_hidden[:n].clone(),
                       o.out_k[:n].clone())
        ctx.close()
        return snap

    ref = run(0, 10, True)
    for n_out in (10, 3, 2, 1):                                # 1: every step reuses the same output buffers
        got = run(mvla.FLAG_INPUTS_STABLE, n_out, False)
        for t in range(10 - n_out, 10):
            assert all(torch.equal(x, y) for x, y in zip(got[t], ref[t])), (n_out, t)


def test_pipelined_steps_sharing_an_index_buffer_two_steps_apart():
    # Every step has its own row buffers, but steps t and t + 2 share kept_idx, and the caller's stream is
    # kept busy between the steps so that the row copies lag behind the selections running ahead on the
    # library's own streams.  A selection must not overwrite indices that an earlier copy has yet to read.
    import dataclasses
    wl = W.small_workload(47, batch=2, D=256, H=4, d=128, dtype="bf16", n_txt=(7, 21), n_2d=(90, 200),
                          n_3d=(160, 310), keep=(0.45, 0.35), steps=12, cold_start=0)
    devs = [device_tensors(wl, t) for t in range(12)]

    def run(flag, share, delay):
        ctx = mvla.context_for(wl)
        outs = [ctx.alloc_outputs(wl.samples, extras=True) for _ in range(12)]
        if share:
            outs = [dataclasses.replace(o, kept_idx=outs[t % 2].kept_idx) for t, o in enumerate(outs)]
        kept = []
        for t, d in enumerate(devs):
            if delay:
                torch.cuda._sleep(300000)                     # touches none of the step's buffers
            o = ctx.prune_step(0, wl.samples, wl.mode, d["q"], d["k"], d["v"], d["hidden"],
                               flags=flag | (mvla.FLAG_RESET_STATE if t == 0 else 0), out=outs[t])
            kept.append(o.total_kept)
            if not flag:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        res = [(o.out_hidden[:n].clone(), o.out_k[:n].clone(), o.budgets.clone()) for o, n in zip(outs, kept)]
        ctx.close()
        return res

    ref = run(0, False, False)
    got = run(mvla.FLAG_INPUTS_STABLE, True, True)
    for t in range(12):
        assert all(torch.equal(x, y) for x, y in zip(got[t], ref[t])), t


def test_pipelined_steps_of_interleaved_episodes_keep_their_states_apart():
    # three episodes (state slots) take turns; inside an episode the carry-over must see the steps in
    # call order although selections of different episodes are free to run beside one another
    import dataclasses
    wl = W.small_workload(53, batch=2, D=256, H=4, d=128, dtype="bf16", n_txt=(9, 30), n_2d=(100, 180),
                          n_3d=(140, 333), keep=(0.5, 0.3), steps=12, cold_start=1)
    devs = [device_tensors(wl, t) for t in range(12)]
    episodes = [[dataclasses.replace(s, state_slot=s.state_slot + 2 * e) for s in wl.samples] for e in range(3)]
    order = [0, 1, 2, 0, 0, 1, 2, 2, 1, 0, 2, 1]              # which episode each call belongs to

    def run(flag):
        ctx = mvla.context_for(wl, n_state_slots=6)
        outs = [ctx.alloc_outputs(wl.samples, extras=True) for _ in range(12)]
        seen, kept = set(), []
        for t, e in enumerate(order):
            d = devs[t]
            o = ctx.prune_step(0, episodes[e], wl.mode, d["q"], d["k"], d["v"], d["hidden"],
                               flags=flag | (0 if e in seen else mvla.FLAG_RESET_STATE), out=outs[t])
            seen.add(e)
            kept.append(o.total_kept)
            if not flag:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        res = [(o.ahat.clone(), o.kept_idx[:n].clone(), o.budgets.clone(), o.out_v[:n].clone())
               for o, n in zip(outs, kept)]
        ctx.close()
        return res

    ref, got = run(0), run(mvla.FLAG_INPUTS_STABLE)
    for t in range(12):
        assert all(torch.equal(x, y) for x, y in zip(got[t], ref[t])), t


def test_step_segments_in_order_3d_text_2d():
    # the three segments may come in any order; here [3D | text | 2D], two samples, adaptive budgets
    base = W.small_workload(47, batch=2, D=256, H=4, d=128, dtype="bf16", n_txt=(9, 30), n_2d=(140, 77),
                            n_3d=(200, 301), keep=(0.4, 0.3))
    t = base.steps[0]
    order, samples = [], []
    for s in base.samples:
        r = s.seq_off
        order += list(range(r + s.off_3d, r + s.off_3d + s.n_3d)) + list(range(r + s.off_txt, r + s.off_txt + s.n_txt)) \
            + list(range(r + s.off_2d, r + s.off_2d + s.n_2d))
        samples.append(W.Sample(seq_off=s.seq_off, off_3d=0, n_3d=s.n_3d, off_txt=s.n_3d, n_txt=s.n_txt,
                                off_2d=s.n_3d + s.n_txt, n_2d=s.n_2d, keep_total=s.keep_total,
                                state_slot=s.state_slot))
    order = np.array(order)
    ten = W.Tensors(hidden=np.ascontiguousarray(t.hidden[order]), q=np.ascontiguousarray(t.q[order]),
                    k=np.ascontiguousarray(t.k[order]), v=np.ascontiguousarray(t.v[order]))
    wl = W.Workload("segments_3d_txt_2d", base.dtype, base.n_heads, base.head_dim, base.d_model, base.mode,
                    samples, [ten])
    ctx = mvla.context_for(wl)
    out, refs = run_and_check_step(ctx, wl, 0, _fresh_states(wl))
    ctx.close()


@pytest.mark.parametrize("dtype,path", [("bf16", mvla.SALIENCE_AUTO), ("bf16", mvla.SALIENCE_FMA), ("fp32", mvla.SALIENCE_AUTO)])
def test_grouped_key_heads(dtype, path):
    # 8 query heads read 2 key heads: K and V rows are a quarter as wide as Q rows
    wl = W.small_workload(17, batch=2, D=256, H=8, d=64, dtype=dtype, mode=W.MODE_FIXED, n_txt=(9, 33),
                          n_2d=(130, 70), n_3d=(150, 300), n_kv_heads=2)
    t = wl.steps[0]
    assert t.k.shape[1] == 2 and t.q.shape[1] == 8
    ctx = mvla.context_for(wl, salience_path=path)
    dev = device_tensors(wl)
    attn, _ = ctx.salience(wl.samples, dev["q"], dev["k"])
    out = ctx.prune_step(0, wl.samples, wl.mode, dev["q"], dev["k"], dev["v"], dev["hidden"])
    torch.cuda.synchronize()
    attn, attn_step = attn.cpu().numpy(), out.attn.cpu().numpy()
    offs, kept_all, budgets = out.out_offsets.cpu().numpy(), out.kept_idx.cpu().numpy(), out.budgets.cpu().numpy()
    vis = 0
    for b, s in enumerate(wl.samples):
        ref = oracle.salience_gqa(t.q, t.k, 8, 2, 64, s)
        assert_salience_close(attn[vis:vis + s.n_vis], ref, "stand-alone scores")
        assert_salience_close(attn_step[vis:vis + s.n_vis], ref, "scores of the fused step")
        k2, k3 = oracle.budget_fixed(s)
        assert (int(budgets[b, 0]), int(budgets[b, 1])) == (k2, k3)
        kept = kept_all[offs[b]:offs[b + 1]]
        check_kept_against_oracle(s, kept, k2, k3, oracle.normalise(ref, s.n_2d, s.n_3d))
        check_stagewise_exact(s, kept, k2, k3, out.ahat.cpu().numpy()[vis:vis + s.n_vis])
        check_compaction(t, out, s, kept, int(offs[b]), wl.dtype)        # K / V rows of 2 x 64 elements
        vis += s.n_vis
    ctx.close()


@pytest.mark.parametrize("d", [96, 160, 256])
@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_other_head_dims(dtype, d):
    # 96 and 160 are not multiples of the 64-element TMA box: the last box is partly out of range and zero-filled
    wl = W.small_workload(19, batch=2, D=512, H=2, d=d, dtype=dtype, n_txt=(7, 30), n_2d=(140, 60), n_3d=(100, 270))
    ctx = mvla.context_for(wl)
    run_and_check_step(ctx, wl, 0, [oracle.State(s.n_vis) for s in wl.samples])
    ctx.close()


@pytest.mark.parametrize("mode", [W.MODE_FIXED, W.MODE_ADAPTIVE])
def test_step_with_an_empty_modality(mode):
    # one sample without 2D tokens, one without 3D tokens, one ordinary
    wl = W.small_workload(23, batch=3, D=256, H=4, d=64, dtype="bf16", mode=mode, n_txt=(6, 17, 9),
                          n_2d=(0, 150, 40), n_3d=(200, 0, 70))
    ctx = mvla.context_for(wl)
    out, refs = run_and_check_step(ctx, wl, 0, [oracle.State(s.n_vis) for s in wl.samples])
    b = out.budgets.cpu().numpy()
    assert b[0, 0] == 0 and b[1, 1] == 0
    ctx.close()


def test_step_more_samples_than_one_launch_carries():
    # 40 samples: the per-sample descriptors travel 32 to a launch, so every stage runs in two launches
    wl = W.small_workload(29, batch=40, D=128, H=2, d=64, dtype="bf16", n_txt=(3, 11, 6), n_2d=(33, 140, 64),
                          n_3d=(129, 20, 75), keep=(0.3, 0.5, 0.25))
    ctx = mvla.context_for(wl)
    states = [oracle.State(s.n_vis) for s in wl.samples]
    run_and_check_step(ctx, wl, 0, states)
    ctx.close()


def test_step_at_the_capacity_limits():
    # 64 text tokens, 2048 + 2048 visual tokens: 32 key tiles, four per CTA in a cluster of eight
    wl = W.small_workload(37, batch=1, D=64, H=1, d=64, dtype="bf16", n_txt=(64,), n_2d=(2048,), n_3d=(2048,),
                          keep=(0.1,))
    ctx = mvla.context_for(wl)
    run_and_check_step(ctx, wl, 0, [oracle.State(s.n_vis) for s in wl.samples])
    ctx.close()


def test_head_sharded_step_two_ranks_emulated_on_one_gpu():
    # Tensor-parallel serving: each rank scores its own heads, the scores are averaged over the ranks, every
    # rank selects on the same scores and copies its own K / V heads.  The two ranks run one after the other
    # here (their kernels do not wait on one another); the average is taken in place of the all-reduce.
    from paper_2604_09244_b200 import tensor_parallel as TP
    wl = W.small_workload(73, batch=2, D=256, H=8, d=64, dtype="bf16", mode=W.MODE_FIXED, n_txt=(9, 20),
                          n_2d=(130, 64), n_3d=(200, 300), n_kv_heads=4)
    t = wl.steps[0]
    dev = device_tensors(wl)
    world = 2
    ctxs, shards, partial = [], [], []
    for r in range(world):
        ctx = mvla.PruneContext(dtype=torch.bfloat16, n_heads=8 // world, n_kv_heads=4 // world, head_dim=64, d_model=256,
                                max_batch=2, max_text=32, max_2d=256, max_3d=512, tau_2d=wl.tau_2d, tau_3d=wl.tau_3d,
                                cold_start_full_keep=0)
        sh = {n: TP.head_shard(dev[n], r, world) for n in ("q", "k", "v")}
        a, _ = ctx.salience(wl.samples, sh["q"], sh["k"])
        ctxs.append(ctx); shards.append(sh); partial.append(a)
    torch.cuda.synchronize()
    attn = (partial[0] + partial[1]) / world                    # what the all-reduce leaves on every rank
    vis = 0
    for s in wl.samples:
        assert_salience_close(attn[vis:vis + s.n_vis].cpu().numpy(), oracle.salience_gqa(t.q, t.k, 8, 4, 64, s))
        vis += s.n_vis
    kept_by_rank = []
    for r in range(world):
        out = ctxs[r].alloc_outputs(wl.samples, extras=True)
        ctxs[r].select(0, wl.samples, wl.mode, attn, None, out=out)
        total = sum(s.seq_len for s in wl.samples)
        ctxs[r].compact(wl.samples, out.kept_idx, out.out_offsets, total, dev["hidden"], shards[r]["k"], shards[r]["v"],
                        out_hidden=out.out_hidden, out_k=out.out_k, out_v=out.out_v)
        torch.cuda.synchronize()
        offs, kept_all = out.out_offsets.cpu().numpy(), out.kept_idx.cpu().numpy()
        kept_by_rank.append(kept_all[:offs[-1]].copy())
        vis = 0
        for b, s in enumerate(wl.samples):
            kept = kept_all[offs[b]:offs[b + 1]]
            k2, k3 = oracle.budget_fixed(s)
            check_kept_against_oracle(s, kept, k2, k3, oracle.normalise(oracle.salience_gqa(t.q, t.k, 8, 4, 64, s), s.n_2d, s.n_3d))
            n = len(kept)
            rows = s.seq_off + kept
            assert torch.equal(out.out_hidden[offs[b]:offs[b] + n], dev["hidden"][rows])
            assert torch.equal(out.out_k[offs[b]:offs[b] + n], shards[r]["k"][rows])       # this rank's key heads
            assert torch.equal(out.out_v[offs[b]:offs[b] + n], shards[r]["v"][rows])
            vis += s.n_vis
    assert np.array_equal(kept_by_rank[0], kept_by_rank[1])      # identical scores, identical decisions
    # the packaged call on a group of one rank: same kept positions as the ranks above
    full = mvla.context_for(wl)
    o = TP.prune_step_head_sharded(full, 0, wl.samples, wl.mode, dev["q"], dev["k"], dev["v"], dev["hidden"])
    torch.cuda.synchronize()
    n = int(o.out_offsets[-1])
    assert np.array_equal(o.kept_idx[:n].cpu().numpy(), kept_by_rank[0])
    for c in ctxs + [full]:
        c.close()


def test_fp8_keys_small_ragged_and_grouped():
    # q, k, v in e4m3 (hidden bf16): ragged tiles, two samples, grouped key heads, head_dim 64 and 128
    for d, hkv in ((128, 0), (64, 2)):
        wl = W.small_workload(81, batch=2, D=256, H=4, d=d, dtype="fp8", n_txt=(7, 33), n_2d=(130, 70), n_3d=(150, 300),
                              n_kv_heads=hkv)
        ctx = mvla.context_for(wl)
        dev = device_tensors(wl)
        assert dev["k"].dtype == torch.float8_e4m3fn and dev["hidden"].dtype == torch.bfloat16
        attn, l1 = ctx.salience(wl.samples, dev["q"], dev["k"], dev["hidden"])
        torch.cuda.synchronize()
        attn = attn.cpu().numpy()
        t = wl.steps[0]
        vis = 0
        for s in wl.samples:
            ref = oracle.salience_gqa(t.q, t.k, 4, hkv or 4, d, s)
            assert_salience_close(attn[vis:vis + s.n_vis], ref, "e4m3 scores")
            vis += s.n_vis
        if not hkv:
            run_and_check_step(ctx, wl, 0, [oracle.State(s.n_vis) for s in wl.samples])
        ctx.close()


def test_fp8_step_single_frame_shape():
    wl = W.config2_single_frame(dtype="fp8")          # 32 text + 256 2D + 512 3D, D = 4096, 32 heads x 128
    ctx = mvla.context_for(wl)
    run_and_check_step(ctx, wl, 0, [oracle.State(s.n_vis) for s in wl.samples])
    ctx.close()


# ------------------------------------------------------------------ fused tail: ties, guard bands, bounded waits
def _duplicate_visual_rows(wl, group):
    """Make groups of `group` neighbouring visual tokens identical (hidden, q, k, v): tokens of one 128-key
    tile then get bit-identical scores, so the selection has to fall back on the index."""
    t = wl.steps[0]
    for s in wl.samples:
        for off, n in ((s.off_2d, s.n_2d), (s.off_3d, s.n_3d)):
            rows = s.seq_off + off + np.arange(n)
            src = s.seq_off + off + (np.arange(n) // group) * group
            for name in ("hidden", "q", "k", "v"):
                getattr(t, name)[rows] = getattr(t, name)[src]


@pytest.mark.parametrize("mode", [W.MODE_FIXED, W.MODE_ADAPTIVE])
@pytest.mark.parametrize("sizes", [((200, 77), (300, 500)), ((900, 1000), (1100, 130))])   # <= 1024 and <= 2048 tokens
@pytest.mark.parametrize("group", [8, 4096])                                                  # runs of 8; everything equal
def test_step_with_equal_scores_straddling_the_budget(mode, sizes, group):
    wl = W.small_workload(91, batch=2, D=256, H=2, d=64, dtype="bf16", mode=mode, n_txt=(9, 20), n_2d=sizes[0],
                          n_3d=sizes[1], keep=(0.37, 0.21), keep_fixed=(0.33, 0.41))
    _duplicate_visual_rows(wl, group)
    ctx = mvla.context_for(wl)
    out, refs = run_and_check_step(ctx, wl, 0, _fresh_states(wl))     # includes the exact stage-wise check
    ahat = out.ahat.cpu().numpy()
    assert len(np.unique(ahat)) < 0.6 * len(ahat), "the case was meant to hold many equal scores"
    ctx.close()


def test_step_leaves_the_bytes_behind_its_outputs_alone():
    # stands in for a memory checker: capacity-sized output buffers are filled with a pattern, and whatever
    # lies behind the rows / list entries the step reports must still hold it afterwards
    wl = W.small_workload(93, batch=3, D=256, H=4, d=128, dtype="bf16", n_txt=(5, 19, 33), n_2d=(70, 130, 260),
                          n_3d=(150, 37, 300), keep=(0.4, 0.3, 0.55))
    ctx = mvla.context_for(wl)
    dev = device_tensors(wl)
    for flags in (0, mvla.FLAG_INPUTS_STABLE):
        out = ctx.alloc_outputs(wl.samples, extras=True)
        for t in (out.out_hidden, out.out_k, out.out_v):
            t.view(torch.int16).fill_(0x5A5A)
        out.kept_idx.fill_(-77)
        ctx.prune_step(0, wl.samples, wl.mode, dev["q"], dev["k"], dev["v"], dev["hidden"], flags=flags | mvla.FLAG_RESET_STATE,
                       out=out)
        torch.cuda.synchronize()
        n = out.total_kept
        assert 0 < n < out.kept_idx.numel() and int(out.out_offsets[-1]) == n
        assert bool((out.kept_idx[n:] == -77).all()), "list entries past the total were written"
        assert bool((out.kept_idx[:n] >= 0).all())
        for t in (out.out_hidden, out.out_k, out.out_v):
            assert bool((t[n:].view(torch.int16) == 0x5A5A).all()), "rows past the total were written"
    ctx.close()


def test_a_bounded_wait_that_runs_out_is_reported_and_sticky():
    # the wait is the one the row-copying CTAs use for a kept-list word; here it polls a word nothing sets,
    # with a limit of 200 us: the kernel ends by itself, the status word holds the error
    wl = W.small_workload(95, batch=1, D=256, H=2, d=64, dtype="bf16", n_txt=(5,), n_2d=(70,), n_3d=(150,))
    dev = device_tensors(wl)
    ctx = mvla.context_for(wl)
    ctx.prune_step(0, wl.samples, wl.mode, dev["q"], dev["k"], dev["v"], dev["hidden"])     # healthy before
    torch.cuda.synchronize()
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    ctx.selftest_wait_timeout(200)
    t1.record()
    torch.cuda.synchronize()
    assert 0.15 < t0.elapsed_time(t1) < 50.0, "the wait must end by itself after about its limit"
    for call in (lambda: ctx.prune_step(0, wl.samples, wl.mode, dev["q"], dev["k"], dev["v"], dev["hidden"]),
                 lambda: ctx.salience(wl.samples, dev["q"], dev["k"])):
        with pytest.raises(mvla.MvlaError) as e:
            call()
        assert e.value.code == mvla.ERR_TIMEOUT                       # sticky: every later call reports it
    ctx.close()
    ctx2 = mvla.context_for(wl)                                       # a fresh context works
    out, refs = run_and_check_step(ctx2, wl, 0, _fresh_states(wl))
    with pytest.raises(mvla.MvlaError) as e:
        ctx2.selftest_wait_timeout(0)                                 # the limit must be 1 us .. 1 s
    assert e.value.code == mvla.ERR_INVALID_ARG
    ctx2.close()


# ------------------------------------------------------------------ reuse of the previous action step's logits
@pytest.mark.parametrize("drift,T", [("all", 16), ("visual_local", 8)])
def test_action_iteration_reusing_the_previous_steps_logits(drift, T):
    # every step is judged against the FULL oracle on the step's own inputs: with a truthful mask the reuse
    # must not be visible in the results
    wl = W.config5_action_iteration(T=T, drift=drift)
    ctx = mvla.context_for(wl, logit_cache=1)
    states = _fresh_states(wl)
    per_step = []
    for t in range(T):
        before = ctx.logit_cache_stats()
        run_and_check_step(ctx, wl, t, states, flags=mvla.FLAG_RESET_STATE if t == 0 else 0,
                           changed_rows=wl.extra["changed_rows"][t] if t > 0 else None)
        after = ctx.logit_cache_stats()
        per_step.append((after[0] - before[0], after[1] - before[1]))
    assert per_step[0] == (10, 0)                                     # 2 image + 8 point tiles, nothing to reuse yet
    assert all(c + r == 10 for c, r in per_step)
    if drift == "visual_local":                                       # one run of 131 rows: two or three tiles change
        assert all(1 <= c <= 3 for c, r in per_step[1:])
    ctx.close()


def test_a_mask_that_hides_a_change_reuses_the_stale_logits():
    # shows that the cache is what is read: with a mask that claims nothing changed, step 2 returns step 1's scores
    wl = W.config5_action_iteration(T=2, D=256, H=4, d=64, n_txt=20, n_2d=150, n_3d=300, drift="visual_local")
    ctx = mvla.context_for(wl, logit_cache=1)
    wl.steps[1].k[:40] *= np.float32(-2.0)                            # a change no tolerance can hide (exact in bf16)
    dev0, dev1 = device_tensors(wl, 0), device_tensors(wl, 1)
    out0 = ctx.prune_step(0, wl.samples, wl.mode, dev0["q"], dev0["k"], dev0["v"], dev0["hidden"], flags=mvla.FLAG_RESET_STATE)
    attn0 = out0.attn.clone()
    lie = np.zeros(wl.samples[0].seq_len, dtype=np.uint8)
    out1 = ctx.prune_step(0, wl.samples, wl.mode, dev1["q"], dev1["k"], dev1["v"], dev1["hidden"], changed_rows=lie)
    torch.cuda.synchronize()
    assert torch.equal(out1.attn, attn0)
    t1 = wl.steps[1]
    truth = oracle.salience(t1.q, t1.k, wl.n_heads, wl.head_dim, wl.samples[0])
    got = out1.attn.cpu().numpy()
    assert (np.abs(got - truth) > 20 * SALIENCE_RTOL * np.abs(truth)).sum() >= 20, "the stale logits were not what was used"
    # and with the truthful mask the same step is right
    ctx.prune_step(0, wl.samples, wl.mode, dev0["q"], dev0["k"], dev0["v"], dev0["hidden"], flags=mvla.FLAG_RESET_STATE)
    out2 = ctx.prune_step(0, wl.samples, wl.mode, dev1["q"], dev1["k"], dev1["v"], dev1["hidden"],
                          changed_rows=wl.extra["changed_rows"][1] | (np.arange(wl.samples[0].seq_len) < 40))
    torch.cuda.synchronize()
    assert_salience_close(out2.attn.cpu().numpy(), truth)
    assert ctx.logit_cache_stats()[1] >= 5                            # step 2 reused all 2 + 3 tiles of step 1
    ctx.close()


@pytest.mark.parametrize("n_txt,n_2d,n_3d", [(40, 700, 900), (64, 512, 640), (17, 1500, 500), (48, 100, 60)])
def test_step_with_two_threads_per_key_in_every_shape_of_the_scoring_kernel(n_txt, n_2d, n_3d):
    # more than 16 text queries: the scoring kernel of the fused step runs with two threads per key, half of the
    # queries each; 33-64 queries use 64 tensor-memory columns (the second half partly empty at 40 and 48), more
    # than 1024 visual tokens put two key tiles on a CTA
    wl = W.small_workload(97, batch=1, D=128, H=2, d=64, dtype="bf16", n_txt=(n_txt,), n_2d=(n_2d,), n_3d=(n_3d,),
                          keep=(0.4,), steps=2)
    ctx = mvla.context_for(wl)
    states = _fresh_states(wl)
    for t in range(2):
        run_and_check_step(ctx, wl, t, states)
    ctx.close()
