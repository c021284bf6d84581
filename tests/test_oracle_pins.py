"""Pins for the fp64 CPU oracle: closed forms, invariants, brute force on tiny
inputs, special cases that reduce to a library routine, and the constants the
paper prints.  None of these re-type the oracle's own loops; each is chosen so
that a plausible slip (a dropped scale, a wrong stride, a transposed operand,
a wrong branch) fails at least one of them."""
import itertools
import math
import os

import numpy as np
import pytest
from scipy.special import softmax as scipy_softmax

import oracle
from paper_2604_09244_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def S(n_txt, n_2d, n_3d, *, seq_off=0, text_first=False, **kw):
    if text_first:
        return W.Sample(seq_off=seq_off, off_txt=0, n_txt=n_txt, off_2d=n_txt, n_2d=n_2d,
                        off_3d=n_txt + n_2d, n_3d=n_3d, **kw)
    return W.layout_2d_3d_txt(seq_off, n_txt, n_2d, n_3d, **kw)


def paper_constants():
    out = {}
    with open(os.path.join(GOLDEN, "paper_constants.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = [float(v) for v in vals]
    return out


# ---------------------------------------------------------------- salience
def test_salience_single_query_single_head_is_library_softmax():
    rng = np.random.default_rng(0)
    d, nv = 16, 9
    s = S(1, 4, 5)
    x = rng.standard_normal((s.seq_len, 1, d)).astype(np.float32)
    a = oracle.salience(x, x, 1, d, s)
    logits = (x[s.off_txt, 0].astype(np.float64) @ x[:nv, 0].astype(np.float64).T) / math.sqrt(d)
    np.testing.assert_allclose(a, scipy_softmax(logits), rtol=1e-13, atol=0)


def test_salience_two_keys_closed_form_sigmoid():
    # one head, one query, two keys: a_0 = sigmoid(q.(k0-k1)/sqrt(d)); pins the 1/sqrt(d) scale and the sign
    d = 4
    s = S(1, 1, 1)
    q = np.zeros((3, 1, d), np.float32)
    k = np.zeros((3, 1, d), np.float32)
    q[2, 0] = [1.0, 2.0, -1.0, 0.5]
    k[0, 0] = [0.5, 0.25, 1.0, -2.0]
    k[1, 0] = [-1.0, 0.5, 0.0, 1.0]
    delta = float(np.dot(q[2, 0], k[0, 0] - k[1, 0])) / 2.0
    a = oracle.salience(q, k, 1, d, s)
    assert a[0] == pytest.approx(1.0 / (1.0 + math.exp(-delta)), rel=1e-14)
    assert a[1] == pytest.approx(1.0 / (1.0 + math.exp(delta)), rel=1e-14)


def test_salience_head_and_query_mean_and_strides():
    # two heads, two queries, two keys, d=2; every (head, query) pair has its own closed-form
    # sigmoid; the expected mean is assembled by hand.  A wrong head/row stride mixes them up.
    d, H = 2, 2
    s = S(2, 1, 1)
    q = np.zeros((4, H, d), np.float32)
    k = np.zeros((4, H, d), np.float32)
    k[0, 0] = [1, 0]; k[1, 0] = [0, 1]      # head 0 keys
    k[0, 1] = [2, 2]; k[1, 1] = [-1, 3]     # head 1 keys
    q[2, 0] = [3, 1]; q[3, 0] = [0, -2]     # head 0 queries (text rows 2, 3)
    q[2, 1] = [1, 1]; q[3, 1] = [0.5, -1]   # head 1 queries
    # garbage in the visual rows' queries and the text rows' keys must not matter
    q[0] = 99; q[1] = -77; k[2] = 55; k[3] = -33
    sig = lambda x: 1.0 / (1.0 + math.exp(-x))
    r2 = math.sqrt(2.0)
    deltas = [(3 - 1) / r2, (0 - (-2)) / r2,             # head 0: q.k0 - q.k1
              ((2 + 2) - (-1 + 3)) / r2, ((1 - 2) - (-0.5 - 3)) / r2]
    expect0 = sum(sig(x) for x in deltas) / 4.0
    a = oracle.salience(q, k, H, d, s)
    assert a[0] == pytest.approx(expect0, rel=1e-14)
    assert a[1] == pytest.approx(1.0 - expect0, rel=1e-13)


@pytest.mark.parametrize("text_first", [False, True])
def test_salience_invariants(text_first):
    rng = np.random.default_rng(1)
    H, d = 3, 8
    s = S(5, 7, 11, seq_off=4, text_first=text_first)
    rows = s.seq_off + s.seq_len + 3
    q = rng.standard_normal((rows, H, d)).astype(np.float32)
    k = rng.standard_normal((rows, H, d)).astype(np.float32)
    a = oracle.salience(q, k, H, d, s)
    assert a.shape == (18,)
    assert a.sum() == pytest.approx(1.0, abs=1e-14)          # each softmax row sums to one
    assert (a > 0).all()
    # adding the same vector to every key of a head shifts each query's logits by a constant
    k2 = k.copy()
    k2[:, 1, :] += rng.standard_normal(d).astype(np.float32).astype(np.float64).astype(np.float32)
    np.testing.assert_allclose(oracle.salience(q, k2, H, d, s), a, rtol=1e-5)
    # permuting the 3D keys permutes their scores
    perm = rng.permutation(s.n_3d)
    k3 = k.copy()
    base = s.seq_off + s.off_3d
    k3[base:base + s.n_3d] = k[base + perm]
    a3 = oracle.salience(q, k3, H, d, s)
    np.testing.assert_allclose(a3[s.n_2d:], a[s.n_2d:][perm], rtol=1e-13)
    np.testing.assert_allclose(a3[:s.n_2d], a[:s.n_2d], rtol=1e-13)


def test_salience_layout_independent_of_segment_order():
    # the same tokens laid out [2D|3D|text] and [text|2D|3D] give the same scores
    rng = np.random.default_rng(2)
    H, d = 2, 4
    sa, sb = S(3, 4, 6), S(3, 4, 6, text_first=True)
    q = rng.standard_normal((13, H, d)).astype(np.float32)
    k = rng.standard_normal((13, H, d)).astype(np.float32)
    order = np.r_[10:13, 0:10]           # rows of layout a in layout b's order
    np.testing.assert_array_equal(oracle.salience(q, k, H, d, sa),
                                  oracle.salience(q[order], k[order], H, d, sb))


def test_salience_uniform_cases():
    rng = np.random.default_rng(3)
    H, d = 2, 8
    s = S(3, 5, 6)
    q = rng.standard_normal((s.seq_len, H, d)).astype(np.float32)
    k = rng.standard_normal((s.seq_len, H, d)).astype(np.float32)
    k_same = k.copy()
    k_same[:11] = k[0]                                        # identical keys
    np.testing.assert_allclose(oracle.salience(q, k_same, H, d, s), 1.0 / 11, rtol=1e-15)
    np.testing.assert_allclose(oracle.salience(np.zeros_like(q), k, H, d, s), 1.0 / 11, rtol=1e-15)


def test_salience_dominant_key_is_one_hot():
    H, d = 1, 4
    s = S(2, 3, 3)
    q = np.ones((s.seq_len, H, d), np.float32)
    k = np.zeros((s.seq_len, H, d), np.float32)
    k[4] = 100.0                                              # 3D token 1 (visual index 4)
    a = oracle.salience(q, k, H, d, s)
    assert a[4] == pytest.approx(1.0, abs=1e-12)
    assert np.delete(a, 4).max() < 1e-12


def test_salience_bruteforce_python_loops():
    # explicit loops in pure Python with math.fsum, on a tiny ragged case with a sequence offset
    rng = np.random.default_rng(4)
    H, d = 2, 3
    s = S(2, 2, 3, seq_off=2)
    rows = s.seq_off + s.seq_len
    q = rng.standard_normal((rows, H, d)).astype(np.float32)
    k = rng.standard_normal((rows, H, d)).astype(np.float32)
    vis = [s.seq_off + s.off_2d + j for j in range(s.n_2d)] + [s.seq_off + s.off_3d + j for j in range(s.n_3d)]
    txt = [s.seq_off + s.off_txt + i for i in range(s.n_txt)]
    expect = [0.0] * len(vis)
    for h, i in itertools.product(range(H), txt):
        e = [math.exp(math.fsum(float(q[i, h, c]) * float(k[j, h, c]) for c in range(d)) / math.sqrt(d))
             for j in vis]
        tot = math.fsum(e)
        for jj in range(len(vis)):
            expect[jj] += e[jj] / tot / (H * len(txt))
    np.testing.assert_allclose(oracle.salience(q, k, H, d, s), expect, rtol=1e-13)


def test_segments_in_any_order_3d_text_2d():
    # layout [3D | text | 2D]: the visual numbering is still 2D first, then 3D; brute force in Python
    rng = np.random.default_rng(14)
    H, d, D = 2, 3, 5
    s = W.Sample(seq_off=1, off_3d=0, n_3d=4, off_txt=4, n_txt=2, off_2d=6, n_2d=3)
    rows = s.seq_off + s.seq_len + 1
    q = rng.standard_normal((rows, H, d)).astype(np.float32)
    k = rng.standard_normal((rows, H, d)).astype(np.float32)
    hid = rng.standard_normal((rows, D)).astype(np.float32)
    vis = [s.seq_off + s.off_2d + j for j in range(s.n_2d)] + [s.seq_off + s.off_3d + j for j in range(s.n_3d)]
    txt = [s.seq_off + s.off_txt + i for i in range(s.n_txt)]
    expect = [0.0] * len(vis)
    for h, i in itertools.product(range(H), txt):
        e = [math.exp(math.fsum(float(q[i, h, c]) * float(k[j, h, c]) for c in range(d)) / math.sqrt(d)) for j in vis]
        tot = math.fsum(e)
        for jj in range(len(vis)):
            expect[jj] += e[jj] / tot / (H * len(txt))
    np.testing.assert_allclose(oracle.salience(q, k, H, d, s), expect, rtol=1e-13)
    np.testing.assert_allclose(oracle.l1norm(hid, D, s), [np.abs(hid[r].astype(np.float64)).sum() for r in vis], rtol=1e-14)
    z = np.array([5.0, 1.0, 3.0, 2.0, 9.0, 4.0, 8.0])       # 2D: 5 1 3   3D: 2 9 4 8
    got = oracle.select(z, s, 2, 2)
    assert got.tolist() == sorted([6 + 0, 6 + 2, 0 + 1, 0 + 3, 4, 5])


# ---------------------------------------------------------------- L1 norms, indicators
def test_salience_grouped_key_heads_equal_repeated_keys():
    # grouped-query attention is plain attention on keys repeated per group (numpy's repeat is the definition)
    rng = np.random.default_rng(41)
    H, Hkv, d = 6, 2, 8
    for text_first in (False, True):
        s = S(3, 5, 7, seq_off=2, text_first=text_first)
        rows = s.seq_off + s.seq_len
        q = rng.standard_normal((rows, H, d)).astype(np.float32)
        k = rng.standard_normal((rows, Hkv, d)).astype(np.float32)
        a = oracle.salience_gqa(q, k, H, Hkv, d, s)
        np.testing.assert_allclose(a, oracle.salience(q, np.repeat(k, H // Hkv, axis=1), H, d, s), rtol=1e-14)
        assert a.sum() == pytest.approx(1.0, rel=1e-13)
    np.testing.assert_array_equal(oracle.salience_gqa(q, np.repeat(k, 3, axis=1), H, H, d, s),
                                  oracle.salience(q, np.repeat(k, 3, axis=1), H, d, s))


def test_l1norm_closed_forms():
    s = S(2, 3, 4, seq_off=1)
    D = 6
    hidden = np.zeros((s.seq_off + s.seq_len, D), np.float32)
    for j in range(7):
        hidden[s.seq_off + j] = (j + 1) * 0.5 * np.array([1, -1, 1, -1, 1, -1], np.float32)
    hidden[s.seq_off + 7:] = 1000.0                          # text rows: never read
    hidden[0] = -1000.0                                      # another sample's row
    n = oracle.l1norm(hidden, D, s)
    np.testing.assert_allclose(n, D * 0.5 * np.arange(1, 8), rtol=0, atol=0)


def test_indicators_closed_forms():
    n2, n3 = 6, 10
    x = oracle.indicators(np.full(16, 1 / 16), None, n2, n3)
    assert x[3] == pytest.approx(n3 / 16, rel=1e-15) and x[2] == pytest.approx(n2 / 16, rel=1e-15)
    assert x[0] == 0.5 and x[1] == 0.5
    # constant rows: 2D norm c, 3D norm s*c  ->  M^S1_3D = s/(1+s), whatever the token counts
    for sc in (0.05, 0.136, 0.30, 1.0, 4.0):
        l1 = np.r_[np.full(n2, 3.0), np.full(n3, 3.0 * sc)]
        x = oracle.indicators(np.full(16, 1 / 16), l1, n2, n3)
        assert x[1] == pytest.approx(sc / (1 + sc), rel=1e-14)
        assert x[0] + x[1] == pytest.approx(1.0, abs=1e-15)
    # attention share uses the sum (not the mean) over tokens
    a = np.r_[np.full(n2, 0.1), np.full(n3, 0.04)]
    assert oracle.indicators(a, None, n2, n3)[3] == pytest.approx(0.4, rel=1e-14)


def test_table1_pairs_sum_to_one_like_the_indicator_pair():
    # Table 1 prints M^S1_2D and M^S1_3D as complementary percentages; the oracle's pair is too.
    c = paper_constants()
    for a, b in zip(c["ms1_2d_percent"], c["ms1_3d_percent"]):
        assert a + b == pytest.approx(100.0, abs=0.011)


# ---------------------------------------------------------------- state update (Eqs. 8, 9)
def run_updates(xs, k=7, beta=0.85):
    xhat = np.zeros_like(np.asarray(xs[0], dtype=np.float64))
    out = []
    for t, x in enumerate(xs, start=1):
        xhat = oracle.state_update(t, k, beta, np.asarray(x, dtype=np.float64), xhat)
        out.append(xhat.copy())
    return out


def test_state_update_impulse_closed_form():
    c = paper_constants()
    beta, k = c["beta"][0], int(c["window_k"][0])
    assert (beta, k) == (0.85, 7)
    hist = run_updates([[1.0]] + [[0.0]] * 8, k=k, beta=beta)
    for t in range(1, 7):
        assert hist[t - 1][0] == pytest.approx(1.0 / t, rel=1e-14)      # Eq. 8 = running mean
    assert hist[6][0] == pytest.approx(0.85 / 6, rel=1e-14)             # t = 7 = k uses Eq. 9
    assert hist[7][0] == pytest.approx(0.85 ** 2 / 6, rel=1e-14)
    assert hist[8][0] == pytest.approx(0.85 ** 3 / 6, rel=1e-14)


def test_state_update_mean_then_geometric():
    rng = np.random.default_rng(5)
    xs = rng.uniform(0, 1, size=(12, 3))
    k, beta = 5, 0.6
    hist = run_updates(list(xs), k=k, beta=beta)
    for t in range(1, k):
        np.testing.assert_allclose(hist[t - 1], xs[:t].mean(axis=0), rtol=1e-13)
    base = xs[:k - 1].mean(axis=0)
    for t in range(k, 13):
        expect = beta ** (t - k + 1) * base + (1 - beta) * sum(beta ** (t - s) * xs[s - 1] for s in range(k, t + 1))
        np.testing.assert_allclose(hist[t - 1], expect, rtol=1e-13)
    const = run_updates([[0.3, 0.7]] * 10)
    for h in const:
        np.testing.assert_allclose(h, [0.3, 0.7], rtol=1e-15)


# ---------------------------------------------------------------- gates
def test_gate_truth_table_and_boundaries():
    c = paper_constants()
    p = oracle.c_params(tau_2d=c["tau_2d"][0], tau_3d=c["tau_3d"][0], eps_3d=0.02)
    both = oracle.SET_2D | oracle.SET_3D
    cases = [  # (M^S1_3D, M^S2_3D) -> (C^S1, C^S2, C_final)
        (0.05, 0.50, (oracle.SET_2D, both, oracle.SET_2D)),
        (0.12, 0.50, (both, both, both)),
        (0.30, 0.50, (oracle.SET_3D, both, oracle.SET_3D)),
        (0.05, 0.01, (oracle.SET_2D, oracle.SET_2D, oracle.SET_2D)),
        (0.12, 0.01, (both, oracle.SET_2D, oracle.SET_2D)),
        (0.30, 0.01, (oracle.SET_3D, oracle.SET_2D, oracle.SET_2D)),   # empty intersection -> C^S2
        (0.08, 0.02, (both, both, both)),                              # exactly at tau_2d / eps: inclusive middle
        (0.20, 0.50, (both, both, both)),                              # exactly at tau_3d
    ]
    for s1, s2, expect in cases:
        got = oracle.gates([1 - s1, s1, 1 - s2, s2], p)
        assert got[:3] == expect, (s1, s2, got)
    assert oracle.gates([0.92, 0.08, 0.5, 0.5], p)[3] == 1             # flagged as near a threshold
    assert oracle.gates([0.88, 0.12, 0.5, 0.5], p)[3] == 0


def test_gate_on_table1_values_with_paper_defaults():
    # Table 1's printed M^S1_3D shares under the printed default thresholds (Sec. 4.1 rule)
    c = paper_constants()
    p = oracle.c_params(tau_2d=c["tau_2d"][0], tau_3d=c["tau_3d"][0])
    both = oracle.SET_2D | oracle.SET_3D
    got = [oracle.gates([1 - v / 100, v / 100, 0.5, 0.5], p)[0] for v in c["ms1_3d_percent"]]
    expect = [both] * 10 + [oracle.SET_3D, both, both, oracle.SET_2D, oracle.SET_2D]
    assert got == expect


# ---------------------------------------------------------------- budgets
def test_round_half_up():
    r = oracle.lib().oracle_round_half_up
    assert [r(0.5), r(1.5), r(2.5), r(2.4999), r(0.0), r(102.4), r(153.6)] == [1, 2, 3, 2, 0, 102, 154]


def test_budget_fixed_single_frame_values():
    s = S(32, 256, 512, keep_2d=0.40, keep_3d=0.30)
    assert oracle.budget_fixed(s) == (102, 154)
    assert oracle.budget_fixed(S(1, 10, 10, keep_2d=1.5, keep_3d=0.0)) == (10, 0)


def test_budget_adaptive_invariants():
    c = paper_constants()
    p = oracle.c_params(floor_ratio=c["floor_ratio"][0])
    both = oracle.SET_2D | oracle.SET_3D
    rng = np.random.default_rng(6)
    for _ in range(400):
        n2, n3 = int(rng.integers(1, 300)), int(rng.integers(1, 300))
        keep = float(np.round(rng.uniform(0.05, 1.0), 3))
        s = S(4, n2, n3, keep_total=keep)
        B = oracle.budget_total(s)
        assert B == min(n2 + n3, math.floor(keep * (n2 + n3) + 0.5))
        for cf, w in ((both, float(rng.uniform())), (oracle.SET_2D, 0.7), (oracle.SET_3D, 0.1)):
            k2, k3, _ = oracle.budget_adaptive(s, p, w, cf)
            assert k2 + k3 == B
            assert 0 <= k2 <= n2 and 0 <= k3 <= n3
            kmin2 = min(math.ceil(0.10 * n2), (B * n2) // (n2 + n3))
            kmin3 = min(math.ceil(0.10 * n3), (B * n3) // (n2 + n3))
            assert k2 >= kmin2 and k3 >= kmin3
            if cf == oracle.SET_2D:
                assert k3 == max(kmin3, B - n2)         # 3D gets only its floor
            if cf == oracle.SET_3D:
                assert k2 == max(kmin2, B - n3)


def test_budget_adaptive_uniform_attention_equal_ratios():
    p = oracle.c_params()
    both = oracle.SET_2D | oracle.SET_3D
    s = S(32, 256, 1024, keep_total=0.30)
    B = oracle.budget_total(s)
    assert B == 384
    k2, k3, near = oracle.budget_adaptive(s, p, 1024 / 1280, both)
    assert (k2, k3) == (77, 307)                       # rhu(384*0.8) = 307: both modalities keep ~30 %
    assert near == 0
    assert oracle.budget_adaptive(S(1, 10, 10, keep_total=0.5), p, 0.55, both)[2] == 1   # 10*0.55 = 5.5


# ---------------------------------------------------------------- select
def brute_select(z, s, k2, k3):
    kept = []
    for off, n, base, k in ((s.off_2d, s.n_2d, 0, k2), (s.off_3d, s.n_3d, s.n_2d, k3)):
        order = sorted(range(n), key=lambda j: (-z[base + j], j))
        kept += [off + j for j in order[:k]]
    kept += [s.off_txt + i for i in range(s.n_txt)]
    return sorted(kept)


@pytest.mark.parametrize("text_first", [False, True])
def test_select_against_full_sort_with_ties(text_first):
    rng = np.random.default_rng(7)
    for trial in range(200):
        n2, n3, nt = int(rng.integers(0, 12)), int(rng.integers(1, 12)), int(rng.integers(1, 4))
        s = S(nt, n2, n3, text_first=text_first)
        z = rng.integers(0, 4, size=n2 + n3).astype(np.float64)    # many exact ties
        k2, k3 = int(rng.integers(0, n2 + 1)), int(rng.integers(0, n3 + 1))
        got = oracle.select(z, s, k2, k3)
        assert got.tolist() == brute_select(z, s, k2, k3)
        assert len(got) == nt + k2 + k3
        assert (np.diff(got) > 0).all()


def test_select_all_equal_keeps_first_indices():
    s = S(2, 6, 5)
    got = oracle.select(np.ones(11), s, 3, 2)
    assert got.tolist() == [0, 1, 2, 6, 7, 11, 12]


def test_select_kept_dominate_dropped():
    rng = np.random.default_rng(8)
    s = S(3, 40, 50)
    z = rng.standard_normal(90)
    got = set(oracle.select(z, s, 13, 21).tolist())
    for off, n, base in ((0, 40, 0), (40, 50, 40)):
        kept = [z[base + j] for j in range(n) if off + j in got]
        drop = [z[base + j] for j in range(n) if off + j not in got]
        assert min(kept) >= max(drop)
    assert all(90 + i in got for i in range(3))


# ---------------------------------------------------------------- compaction
def test_compact_is_ordered_byte_copy():
    rng = np.random.default_rng(9)
    src = rng.integers(0, 2 ** 16, size=(20, 7), dtype=np.uint16)
    kept = np.array([0, 3, 4, 9], dtype=np.int32)
    out = oracle.compact(src, 5, kept)
    assert out.tobytes() == src[5 + kept].tobytes()


# ---------------------------------------------------------------- whole step
@pytest.mark.parametrize("cfg", ["config1"])
def test_whole_step_invariants(cfg):
    wl = W.by_name(cfg)
    s = wl.samples[0]
    st = oracle.State(s.n_vis)
    r = oracle.run_workload_step(wl, 0, [st])[0]
    B = oracle.budget_total(s)
    assert r.t == 1 and r.k_2d + r.k_3d == B == 96
    kept = r.kept_idx
    assert (np.diff(kept) > 0).all()                                  # order-preserving subsequence
    in2 = ((kept >= s.off_2d) & (kept < s.off_2d + s.n_2d)).sum()
    in3 = ((kept >= s.off_3d) & (kept < s.off_3d + s.n_3d)).sum()
    txt = ((kept >= s.off_txt) & (kept < s.off_txt + s.n_txt)).sum()
    assert (in2, in3, txt) == (r.k_2d, r.k_3d, s.n_txt)
    assert r.attn.sum() == pytest.approx(1.0, abs=1e-13)
    np.testing.assert_allclose(r.z[:s.n_2d].mean(), 1.0, rtol=1e-13)   # per-modality mean one
    np.testing.assert_allclose(r.z[s.n_2d:].mean(), 1.0, rtol=1e-13)
    # boosted tokens (hidden x4) attract attention: all of them survive a 50 % prune
    assert set(wl.extra["boosted"].tolist()) <= set(kept.tolist())
    # the stored fixture was written by tests/golden/make_golden.py from the oracle alone
    gold = np.loadtxt(os.path.join(GOLDEN, "config1_kept_idx.txt"), dtype=np.int64)
    assert kept.tolist() == gold.tolist()


def test_cold_start_keeps_everything_then_prunes():
    wl = W.small_workload(11, batch=1, steps=3, cold_start=1, n_txt=(4,), n_2d=(20,), n_3d=(30,),
                          keep=(0.4,), D=64, H=2, d=32)
    s = wl.samples[0]
    st = oracle.State(s.n_vis)
    r1 = oracle.run_workload_step(wl, 0, [st])[0]
    assert r1.kept_idx.tolist() == list(range(s.seq_len))            # Alg. 1: t == 1 returns all tokens
    np.testing.assert_array_equal(r1.ahat, r1.attn)                  # and the state is initialised
    r2 = oracle.run_workload_step(wl, 1, [st])[0]
    assert r2.t == 2 and len(r2.kept_idx) == s.n_txt + 20
    np.testing.assert_allclose(r2.ahat, 0.5 * (r1.attn + r2.attn), rtol=1e-14)


# ---------------------------------------------------------------- Alg. 1 over several steps
def multistep_worked():
    out = {}
    with open(os.path.join(GOLDEN, "alg1_multistep_worked.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = np.array([float(v) for v in vals])
    return out


def test_ranking_uses_the_predicted_scores_hand_worked():
    # Alg. 1 stage 1 feeds the later stages: the kept tokens follow X^_t (Eq. 8, then Eq. 9), which here
    # ranks the tokens the other way round from the step's own scores.
    g = multistep_worked()
    s = S(1, 2, 2, keep_2d=0.5, keep_3d=0.5)
    p = oracle.c_params(window_k=3, beta=0.85, cold_start_full_keep=0)
    st = oracle.State(4)
    r1 = oracle.decide_step(g["R_a1"], None, s, p, oracle.MODE_FIXED, st)
    assert r1.kept_idx.tolist() == g["R_kept1"].astype(int).tolist() and (r1.k_2d, r1.k_3d, r1.t) == (1, 1, 1)
    r2 = oracle.decide_step(g["R_a2"], None, s, p, oracle.MODE_FIXED, st)
    np.testing.assert_allclose(r2.ahat, g["R_ahat2"], rtol=1e-14)
    np.testing.assert_allclose(r2.z, g["R_z2"], rtol=1e-14)
    assert r2.kept_idx.tolist() == g["R_kept2"].astype(int).tolist()
    assert np.argmax(g["R_a2"][:2]) == 1 and np.argmax(g["R_a2"][2:]) == 1      # the step alone says rows 1, 3
    r3 = oracle.decide_step(g["R_a3"], None, s, p, oracle.MODE_FIXED, st)
    np.testing.assert_allclose(r3.ahat, g["R_ahat3_ema"], rtol=1e-14)
    assert r3.kept_idx.tolist() == g["R_kept3"].astype(int).tolist() and r3.t == 3


def _case_g(g):
    j = np.arange(10)
    a1 = np.concatenate([(j + 1) * (1 - g["G_share1"][0]) / 55, (10 - j) * g["G_share1"][0] / 55])
    a2 = np.concatenate([(10 - j) * (1 - g["G_share2"][0]) / 55, (j + 1) * g["G_share2"][0] / 55])
    n1 = np.repeat(g["G_norm1"], 10)
    n2 = np.repeat(g["G_norm2"], 10)
    return a1, a2, n1, n2


def test_gates_and_budget_use_the_predicted_indicators_hand_worked():
    # Sec. 4.1 / 4.2 / 4.4 and the budget split act on M^ (Alg. 1 stages 2-4), with the defaults of Sec. 5.4
    g = multistep_worked()
    a1, a2, n1, n2 = _case_g(g)
    s = S(1, 10, 10, keep_total=0.5)
    p = oracle.c_params(cold_start_full_keep=0)
    st = oracle.State(20)
    r1 = oracle.decide_step(a1, n1, s, p, oracle.MODE_ADAPTIVE, st)
    assert [r1.c_s1, r1.c_s2, r1.c_final] == g["G_sets1"].astype(int).tolist()
    assert [r1.k_2d, r1.k_3d] == g["G_k1"].astype(int).tolist()
    assert r1.kept_idx.tolist() == g["G_kept1"].astype(int).tolist()
    r2 = oracle.decide_step(a2, n2, s, p, oracle.MODE_ADAPTIVE, st)
    np.testing.assert_allclose(r2.mhat, g["G_mhat2"], rtol=1e-12)
    np.testing.assert_allclose(r2.x, [0.7, 0.3, 0.38, 0.62], rtol=1e-12)          # the step's own indicators
    assert [r2.c_s1, r2.c_s2, r2.c_final] == g["G_sets2"].astype(int).tolist()
    assert [r2.k_2d, r2.k_3d] == g["G_k2"].astype(int).tolist()
    assert r2.kept_idx.tolist() == g["G_kept2"].astype(int).tolist()
    assert not r2.near_gate and not r2.near_half


def test_whole_step_feeds_scores_and_norms_into_the_decisions():
    # The same two steps through oracle_prune_step.  One head, one query q = (sqrt(d), 0, ...): the logit of
    # key j is its first component, so keys (ln a_j, 0, ...) make the softmax return a_j itself; a constant
    # hidden row c has the L1 norm D |c|.
    g = multistep_worked()
    d = D = 4
    s = S(1, 10, 10, keep_total=0.5)
    p = oracle.c_params(cold_start_full_keep=0)
    st = oracle.State(20)
    for a, nrm, kept, ks in zip(_case_g(g)[:2], _case_g(g)[2:], ("G_kept1", "G_kept2"), ("G_k1", "G_k2")):
        q = np.zeros((21, 1, d), np.float32)
        k = np.zeros((21, 1, d), np.float32)
        q[20, 0, 0] = 2.0
        k[:20, 0, 0] = np.log(a)
        k[:20, 0, 1:] = 7.0                                   # orthogonal to q: must not matter
        hidden = np.zeros((21, D), np.float32)
        hidden[:20] = (nrm / D)[:, None] * np.array([1, -1, 1, -1])
        r = oracle.prune_step(q, k, hidden, 1, d, D, s, p, oracle.MODE_ADAPTIVE, st)
        np.testing.assert_allclose(r.attn, a, rtol=1e-6)
        np.testing.assert_allclose(r.l1, nrm, rtol=1e-6)
        assert [r.k_2d, r.k_3d] == g[ks].astype(int).tolist()
        assert r.kept_idx.tolist() == g[kept].astype(int).tolist()
    np.testing.assert_allclose(st.c.mhat[:], g["G_mhat2"], rtol=1e-6)


# ---------------------------------------------------------------- reuse of the previous step's logits
def _drifting_case(seed=3):
    rng = np.random.default_rng(seed)
    H, d = 2, 8
    s = S(3, 5, 6, seq_off=2)                                  # visual rows 2..12, text rows 13..15
    rows = s.seq_off + s.seq_len
    q0 = rng.standard_normal((rows, H, d)).astype(np.float32)
    k0 = rng.standard_normal((rows, H, d)).astype(np.float32)
    return H, d, s, rows, q0, k0, rng


def test_cached_salience_with_a_truthful_mask_is_the_plain_salience():
    H, d, s, rows, q, k, rng = _drifting_case()
    cache = oracle.LogitCache(H, s)
    a, n = oracle.salience_cached(q, k, H, d, s, None, cache)                  # nothing cached yet: everything computed
    assert n == 11 and np.array_equal(a, oracle.salience(q, k, H, d, s))
    for step in range(4):
        changed = np.zeros(rows, np.uint8)
        vis = s.seq_off + rng.choice(11, size=3, replace=False)
        changed[vis] = 1
        k = k.copy(); q = q.copy()
        k[vis] += rng.standard_normal((3, H, d)).astype(np.float32)
        q[vis] += 1.0                                           # queries of visual rows are never read
        a, n = oracle.salience_cached(q, k, H, d, s, changed, cache)
        assert n == 3
        assert np.array_equal(a, oracle.salience(q, k, H, d, s))               # same arithmetic, same bits
    # a changed text row: every logit has that query in it -> everything is recomputed
    changed = np.zeros(rows, np.uint8)
    changed[s.seq_off + s.off_txt + 1] = 1
    q = q.copy(); q[s.seq_off + s.off_txt + 1] *= -2.0
    a, n = oracle.salience_cached(q, k, H, d, s, changed, cache)
    assert n == 11 and np.array_equal(a, oracle.salience(q, k, H, d, s))


def test_cached_salience_really_uses_the_cache():
    # a key that changed but is reported unchanged keeps its OLD logits: the result is the plain salience of
    # the inputs in which that key still has its old row -- and not that of the current inputs
    H, d, s, rows, q, k_old, rng = _drifting_case(5)
    cache = oracle.LogitCache(H, s)
    oracle.salience_cached(q, k_old, H, d, s, None, cache)
    k_new = k_old.copy()
    moved = s.seq_off + np.array([1, 7])
    k_new[moved] += 2.0
    changed = np.zeros(rows, np.uint8)
    changed[moved[0]] = 1                                        # key 7 changed too, but the mask hides it
    a, n = oracle.salience_cached(q, k_new, H, d, s, changed, cache)
    k_mixed = k_new.copy()
    k_mixed[moved[1]] = k_old[moved[1]]
    assert n == 1
    assert np.array_equal(a, oracle.salience(q, k_mixed, H, d, s))
    assert np.abs(a - oracle.salience(q, k_new, H, d, s)).max() > 1e-3
