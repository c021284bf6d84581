"""Pins for the patch-by-patch statement of Alg. 1 in the CPU oracle (mvla_patch_oracle.c): vectors
and rule tables worked out by hand (tests/golden/), invariants of the orthogonal decomposition,
library routines (scipy softmax, numpy least squares, scikit-learn's Lloyd iteration from the same
start) and brute-force consistency of the whole step."""
import itertools
import math
import os

import numpy as np
import pytest
from scipy.special import softmax as scipy_softmax

import oracle
from paper_2604_09244_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
BOTH = oracle.SET_2D | oracle.SET_3D


def S(n_txt, n_patch, *, seq_off=0, text_first=False):
    if text_first:
        return W.Sample(seq_off=seq_off, off_txt=0, n_txt=n_txt, off_2d=n_txt, n_2d=n_patch,
                        off_3d=n_txt + n_patch, n_3d=n_patch)
    return W.layout_2d_3d_txt(seq_off, n_txt, n_patch, n_patch)


# ---------------------------------------------------------------- attention matrix
@pytest.mark.parametrize("text_first", [False, True])
def test_attention_rows_are_library_softmax_and_mean_is_the_salience(text_first):
    rng = np.random.default_rng(3)
    H, d, s = 3, 8, S(4, 5, seq_off=2, text_first=text_first)
    rows = s.seq_off + s.seq_len
    q = rng.standard_normal((rows, H, d)).astype(np.float32)
    k = rng.standard_normal((rows, H, d)).astype(np.float32)
    alpha = oracle.attention(q, k, H, d, s)
    assert alpha.shape == (H, 4, 10)
    np.testing.assert_allclose(alpha.sum(axis=2), 1.0, rtol=1e-14)
    vis = np.r_[s.seq_off + s.off_2d + np.arange(5), s.seq_off + s.off_3d + np.arange(5)]
    for h, i in itertools.product(range(H), range(4)):
        logits = (k[vis, h].astype(np.float64) @ q[s.seq_off + s.off_txt + i, h].astype(np.float64)) / math.sqrt(d)
        np.testing.assert_allclose(alpha[h, i], scipy_softmax(logits), rtol=1e-13)
    np.testing.assert_allclose(alpha.mean(axis=(0, 1)), oracle.salience(q, k, H, d, s), rtol=1e-13)


# ---------------------------------------------------------------- Eq. 3-4
def test_ortho_decompose_hand_worked_vector():
    # a2 = (1,1,1), a3 = (1,0,0): projection coefficient 1/3; ortho = (2/3, -1/3, -1/3), L1 norm 4/3
    para, ortho = oracle.ortho_decompose([1, 1, 1], [1, 0, 0])
    np.testing.assert_allclose(para, [1 / 3] * 3, rtol=1e-15)
    np.testing.assert_allclose(ortho, [2 / 3, -1 / 3, -1 / 3], rtol=1e-15)


def test_ortho_decompose_invariants_and_least_squares():
    rng = np.random.default_rng(5)
    for n in (1, 2, 7, 64):
        a2, a3 = rng.random(n), rng.random(n)
        para, ortho = oracle.ortho_decompose(a2, a3)
        np.testing.assert_allclose(para + ortho, a3, rtol=1e-14)
        assert abs(np.dot(ortho, a2)) <= 1e-14 * n
        c = np.linalg.lstsq(a2[:, None], a3, rcond=None)[0][0]          # library routine: best multiple of a2
        np.testing.assert_allclose(para, c * a2, rtol=1e-12)
    # parallel vectors: nothing is unique to 3D; disjoint supports: everything is; a2 = 0: ortho = a3
    a2 = rng.random(9)
    np.testing.assert_allclose(oracle.ortho_decompose(a2, 2.5 * a2)[1], 0.0, atol=1e-15)
    p, o = oracle.ortho_decompose([1, 2, 0, 0], [0, 0, 3, 4])
    np.testing.assert_array_equal(o, [0, 0, 3, 4])
    np.testing.assert_array_equal(p, [0, 0, 0, 0])
    np.testing.assert_array_equal(oracle.ortho_decompose([0, 0], [1, 2])[1], [1, 2])


# ---------------------------------------------------------------- Eq. 3-1, P2D, P3D per patch
def test_patch_indicators_hand_worked():
    # two patches, three (head, query) rows; columns = [2D p0, 2D p1, 3D p0, 3D p1]
    alpha = np.array([[1.0, 0.2, 1.0, 0.0],
                      [1.0, 0.0, 0.0, 0.3],
                      [1.0, 0.0, 0.0, 0.1]])
    l1 = np.array([3.0, 1.0, 1.0, 3.0])
    x = oracle.patch_indicators(alpha, l1)
    # patch 0: a2 = (1,1,1), a3 = (1,0,0): norms 3 and 1, ortho norm 4/3
    np.testing.assert_allclose(x[0], [0.75, 0.25, 3 / 4, (4 / 3) / 4], rtol=1e-15)
    # patch 1: disjoint supports: ortho = a3; norms 0.2 and 0.4
    np.testing.assert_allclose(x[1], [0.25, 0.75, 1 / 3, 2 / 3], rtol=1e-14)


def test_patch_indicators_invariants():
    rng = np.random.default_rng(11)
    rows, P = 12, 6
    alpha = rng.random((rows, 2 * P))
    l1 = rng.random(2 * P) + 0.1
    x = oracle.patch_indicators(alpha, l1)
    np.testing.assert_allclose(x[:, 0] + x[:, 1], 1.0, rtol=1e-14)
    # 3D token's vector a multiple of the 2D token's: no unique 3D information
    alpha2 = alpha.copy()
    alpha2[:, P:] = 0.5 * alpha2[:, :P]
    x2 = oracle.patch_indicators(alpha2, l1)
    np.testing.assert_allclose(x2[:, 3], 0.0, atol=1e-15)
    np.testing.assert_allclose(x2[:, 2], 1 / 1.5, rtol=1e-14)
    # scaling a patch's two vectors together changes nothing (shares)
    alpha3 = alpha.copy()
    alpha3[:, 2] *= 7.0
    alpha3[:, P + 2] *= 7.0
    np.testing.assert_allclose(oracle.patch_indicators(alpha3, l1), x, rtol=1e-13)
    # swapping two patches swaps their rows
    perm = np.arange(P); perm[[1, 4]] = perm[[4, 1]]
    xp = oracle.patch_indicators(alpha[:, np.r_[perm, P + perm]], l1[np.r_[perm, P + perm]])
    np.testing.assert_allclose(xp, x[perm], rtol=1e-15)


# ---------------------------------------------------------------- 1-D K-Means
def _golden_kmeans():
    out = {}
    with open(os.path.join(GOLDEN, "kmeans1d_worked.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                key, *vals = line.split()
                out[key] = [float(v) for v in vals]
    return out


@pytest.mark.parametrize("case", ["A", "B", "C"])
def test_kmeans_hand_worked_cases(case):
    g = _golden_kmeans()
    labels, centre, rounds, _ = oracle.kmeans1d(g[f"{case}_points"])
    assert labels.tolist() == [int(v) for v in g[f"{case}_labels"]]
    np.testing.assert_allclose(centre, g[f"{case}_centres"], rtol=1e-14)
    assert rounds == int(g[f"{case}_rounds"][0])


def test_kmeans_matches_scikit_learn_lloyd_from_the_same_start():
    from sklearn.cluster import KMeans
    rng = np.random.default_rng(17)
    for trial in range(6):
        v = np.concatenate([rng.normal(0.5, 0.2, 40), rng.normal(2.0, 0.3, 25), rng.normal(6.0, 1.0, 8)])
        rng.shuffle(v)
        init = np.array([[v.min()], [v.mean()], [v.max()]])
        km = KMeans(n_clusters=3, init=init, n_init=1, algorithm="lloyd", tol=0.0, max_iter=300).fit(v[:, None])
        labels, centre, rounds, margin = oracle.kmeans1d(v, 300)
        assert margin > 1e-9                                   # no point sits on a boundary: the result is unique
        assert np.array_equal(labels, km.labels_)
        np.testing.assert_allclose(centre, km.cluster_centers_[:, 0], rtol=1e-12)


def test_kmeans_fixed_point_and_edge_cases():
    rng = np.random.default_rng(19)
    v = rng.random(200) ** 3
    labels, centre, rounds, _ = oracle.kmeans1d(v, 100)
    assert rounds < 100
    assert (np.diff(centre) >= 0).all()
    for c in range(3):
        np.testing.assert_allclose(centre[c], v[labels == c].mean(), rtol=1e-13)
    assert np.array_equal(labels, np.argmin(np.abs(v[:, None] - centre[None, :]), axis=1))
    # one assignment round only
    l1, c1, r1, _ = oracle.kmeans1d([0, 1, 2, 5], 1)
    assert r1 == 1 and l1.tolist() == [0, 0, 1, 2]
    np.testing.assert_allclose(c1, [0.5, 2, 5])          # a round = assignment, then the centres move
    # all points equal: every distance ties, everything stays with the lowest centre
    l2, c2, r2, m2 = oracle.kmeans1d([0.3] * 5)
    assert l2.tolist() == [0] * 5 and m2 == 0.0


# ---------------------------------------------------------------- rules
LABELS = {"bg": oracle.LABEL_BG, "rob": oracle.LABEL_ROB, "obj": oracle.LABEL_OBJ}


def test_rule_table_worked_from_alg1():
    p = oracle.c_patch_params()                               # the paper's defaults
    n = 0
    with open(os.path.join(GOLDEN, "alg1_patch_rules.txt")) as f:
        for line in f:
            if not line.strip() or line.startswith("#"):
                continue
            tok = line.split()
            lab = LABELS[tok[0]]
            s1, m2, m3, mu2, mu3, u = (float(t) for t in tok[1:7])
            c1e, c2e, cfe, k2e, k3e = (int(t) for t in tok[7:12])
            c1 = oracle.patch_c_s1(s1, p.tau_2d, p.tau_3d)
            c2 = oracle.patch_c_s2(lab, m2, m3, mu2, mu3, u, p)
            cf = oracle.patch_fuse(c1, c2)
            assert (c1, c2, cf) == (c1e, c2e, cfe), line
            assert (int(bool(cf & oracle.SET_2D)), int(bool(cf & oracle.SET_3D))) == (k2e, k3e), line   # Eq. 10
            n += 1
    assert n == 23


def test_fusion_truth_table():
    # Sec. 4.4: empty semantic set discards; else the intersection; an empty intersection keeps C_S2
    expect = {(1, 1): 1, (1, 2): 2, (1, 3): 1, (2, 1): 1, (2, 2): 2, (2, 3): 2, (3, 1): 1, (3, 2): 2, (3, 3): 3}
    for c1 in (1, 2, 3):
        assert oracle.patch_fuse(c1, 0) == 0
        for c2 in (1, 2, 3):
            assert oracle.patch_fuse(c1, c2) == expect[(c1, c2)]


# ---------------------------------------------------------------- stages 1-4 together
def _small_case():
    s = S(2, 4)                                               # rows: 2D 0-3, 3D 4-7, text 8-9
    a = np.array([0.005, 0.01, 0.02, 0.5, 0.005, 0.01, 0.18, 0.4])      # patch masses 0.01 0.02 0.2 0.9
    x = np.array([[0.88, 0.12, 0.5, 0.2],
                  [0.95, 0.05, 0.5, 0.2],
                  [0.75, 0.25, 0.7, 0.1],
                  [0.75, 0.25, 0.9, 0.3]])
    u = np.array([0.5, 0.95, 0.0, 0.0])
    return s, a, x, u


def test_patch_select_hand_worked_step():
    # labels (golden case B): bg bg rob obj.  mu_2D = 0.65, mu_3D = 0.2.
    # p0: bg, u = 0.5 < 0.9 -> discarded.  p1: bg, u = 0.95 -> {2D,3D}; M^S1_3D = 0.05 < 0.08 -> {2D}: keep 2D.
    # p2: rob, 0.1 <= 0.2 and 0.7 > 0.65 -> {2D}; M^S1_3D = 0.25 > 0.20 -> {3D}; conflict -> {2D}: keep 2D.
    # p3: obj, 3D share 0.3 not near zero -> {2D,3D}; C_S1 = {3D} -> keep 3D.
    s, a, x, u = _small_case()
    st = oracle.PatchState(4)
    r = oracle.patch_select(a, x, u, s, oracle.c_patch_params(cold_start_full_keep=0), st)
    assert r.labels.tolist() == [0, 0, 1, 2]
    assert r.cand.tolist() == [[3, 0, 0], [1, 3, 1], [2, 1, 1], [2, 3, 2]]
    assert r.kept_idx.tolist() == [1, 2, 7, 8, 9]
    assert (r.k_2d, r.k_3d, r.t) == (2, 1, 1)
    assert r.mu_2d == pytest.approx(0.65) and r.mu_3d == pytest.approx(0.2)
    np.testing.assert_array_equal(st.xhat, x)                 # X^_1 = X_1


def test_patch_select_cold_start_then_running_mean_then_ema():
    s, a, x, u = _small_case()
    p = oracle.c_patch_params(window_k=3, beta=0.85)
    st = oracle.PatchState(4)
    r1 = oracle.patch_select(a, x, u, s, p, st)
    assert r1.kept_idx.tolist() == list(range(10))            # t = 1: full unpruned tokens
    assert (r1.cand[:, 2] == BOTH).all()
    x2 = x[::-1].copy()
    r2 = oracle.patch_select(a, x2, u, s, p, st)              # t = 2 < k: Eq. 8, the mean of X_1, X_2
    np.testing.assert_allclose(st.xhat, (x + x2) / 2, rtol=1e-15)
    assert len(r2.kept_idx) < 10
    x3 = np.full_like(x, 0.25)
    r3 = oracle.patch_select(a, x3, u, s, p, st)              # t = 3 = k: Eq. 9
    np.testing.assert_allclose(st.xhat, 0.85 * (x + x2) / 2 + 0.15 * x3, rtol=1e-15)
    assert st.t == 3
    # the baselines are means of the SMOOTHED shares: 0.85 * 0.65 + 0.15 * 0.25 and 0.85 * 0.2 + 0.15 * 0.25
    assert r3.mu_2d == pytest.approx(0.59, rel=1e-13) and r3.mu_3d == pytest.approx(0.2075, rel=1e-13)


def test_patch_select_invariants_random():
    rng = np.random.default_rng(23)
    for text_first in (False, True):
        P, nt = 37, 5
        s = S(nt, P, text_first=text_first)
        a = rng.random(2 * P) ** 4
        x = rng.random((P, 4))
        x[:, 1] *= 0.3
        u = rng.random(P)
        st = oracle.PatchState(P)
        r = oracle.patch_select(a, x, u, s, oracle.c_patch_params(cold_start_full_keep=0), st)
        kept = r.kept_idx
        assert (np.diff(kept) > 0).all()
        assert set(range(s.off_txt, s.off_txt + nt)) <= set(kept.tolist())
        m2 = np.isin(s.off_2d + np.arange(P), kept)
        m3 = np.isin(s.off_3d + np.arange(P), kept)
        np.testing.assert_array_equal(m2, (r.cand[:, 2] & oracle.SET_2D) != 0)      # Eq. 10
        np.testing.assert_array_equal(m3, (r.cand[:, 2] & oracle.SET_3D) != 0)
        assert (r.k_2d, r.k_3d) == (m2.sum(), m3.sum()) and len(kept) == nt + m2.sum() + m3.sum()
        assert r.n_label.sum() == P
        assert ((r.cand[:, 1] == 0) == (r.cand[:, 2] == 0)).all()   # discarded exactly when the semantic set is empty
        # background patches survive only with u >= 0.9
        bg = r.labels == oracle.LABEL_BG
        np.testing.assert_array_equal(r.cand[bg, 1] != 0, u[bg] >= 0.9)


def test_patch_step_is_the_composition_of_its_parts():
    wl = W.patch_workload(31, batch=1, D=64, H=2, d=16, n_txt=(3,), n_patch=(9,), dtype="fp32")
    s, t = wl.samples[0], wl.steps[0]
    p = oracle.patch_params_of(wl)
    u = wl.extra["rand_u"][0][:9]
    r = oracle.patch_step(t.q, t.k, t.hidden, 2, 16, 64, s, u, p, oracle.PatchState(9))
    alpha = oracle.attention(t.q, t.k, 2, 16, s)
    np.testing.assert_allclose(r.attn, oracle.salience(t.q, t.k, 2, 16, s), rtol=1e-13)
    x = oracle.patch_indicators(alpha.reshape(-1, 18), oracle.l1norm(t.hidden, 64, s))
    np.testing.assert_allclose(r.x, x, rtol=1e-15)
    r2 = oracle.patch_select(r.attn, x, u, s, p, oracle.PatchState(9))
    assert np.array_equal(r.kept_idx, r2.kept_idx) and np.array_equal(r.cand, r2.cand)


def test_patch_rules_use_the_predicted_indicators_hand_worked():
    # Alg. 1 stages 2-4 read X^_t (Eq. 8 at t = 2, Eq. 9 at t = 3 = k); every named patch is built so
    # that its predicted share and the step's own share fall on opposite sides of a threshold.
    g = {}
    with open(os.path.join(GOLDEN, "alg1_multistep_worked.txt")) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                key, *vals = line.split()
                g[key] = np.array([float(v) for v in vals])
    s, a, _, u = _small_case()
    p = oracle.c_patch_params(window_k=3, beta=0.85, cold_start_full_keep=0)
    st = oracle.PatchState(4)
    for t in (1, 2, 3):
        r = oracle.patch_select(a, g[f"P_x{t}"].reshape(4, 4), u, s, p, st)
        assert r.t == t and r.labels.tolist() == [0, 0, 1, 2]
        assert r.cand.reshape(-1).tolist() == g[f"P_cand{t}"].astype(int).tolist(), t
        assert r.kept_idx.tolist() == g[f"P_kept{t}"].astype(int).tolist(), t
        if t > 1:
            assert [r.mu_2d, r.mu_3d] == pytest.approx(g[f"P_mu{t}"].tolist(), rel=1e-13)
    np.testing.assert_allclose(st.xhat[1], g["P_xhat3_p1"], rtol=1e-13)
