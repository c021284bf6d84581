"""Do the pins bite?  Each case plants one plausible mistake in a COPY of the oracle's C source (on the
CPU, in a temporary directory), builds it, runs the pin tests against the mutated library and demands
that at least one of them fails.  The oracle in the repository is never touched."""
import os
import subprocess

import pytest

import oracle
import test_oracle_pins as pins

import test_patch_oracle_pins as patch_pins

ODIR = os.path.dirname(oracle.__file__)
FILES = ("mvla_oracle.c", "mvla_oracle.h", "mvla_patch_oracle.c", "mvla_patch_oracle.h")

PIN_TESTS = [getattr(pins, n) for n in dir(pins) if n.startswith("test_")]
PATCH_PIN_TESTS = [getattr(patch_pins, n) for n in dir(patch_pins) if n.startswith("test_")]

MUTATIONS = {
    "logit scale dropped": ("logit[j] = acc / sqrt((double)d);", "logit[j] = acc;"),
    "logit sign flipped": ("acc += (double)qi[c] * (double)kj[c];", "acc -= (double)qi[c] * (double)kj[c];"),
    "query head offset wrong": ("+ s->off_txt + i) * row + (int64_t)h * d;", "+ s->off_txt + i) * row + (int64_t)h;"),
    "key row ignores the sample offset": ("const float *kj = k + ((int64_t)s->seq_off + vis_row(s, j)) * krow",
                                          "const float *kj = k + ((int64_t)vis_row(s, j)) * krow"),
    "grouped key head taken modulo": ("(int64_t)(h / group) * d;", "(int64_t)(h % n_kv_heads) * d;"),
    "key row stride of the query tensor": ("const int64_t krow = (int64_t)n_kv_heads * d;", "const int64_t krow = (int64_t)H * d;"),
    "mean over heads only": ("a_out[j] = acc / ((double)H * (double)nt);", "a_out[j] = acc / ((double)H);"),
    "softmax denominator over 2D keys only": ("for (int32_t j = 0; j < nv; ++j) den += exp(logit[j] - mx);",
                                              "for (int32_t j = 0; j < s->n_2d; ++j) den += exp(logit[j] - mx);"),
    "3D tokens read from the 2D segment": ("return j < s->n_2d ? s->off_2d + j : s->off_3d + (j - s->n_2d);",
                                          "return j < s->n_2d ? s->off_2d + j : s->off_2d + j;"),
    "norm without the absolute value": ("acc += fabs((double)r[c]);", "acc += (double)r[c];"),
    "attention share uses 2D in the numerator": ("x[3] = a3 / (a2 + a3);", "x[3] = a2 / (a2 + a3);"),
    "norm share from sums, not means": ("const double m3 = n_3d > 0 ? s3 / n_3d : 0.0;", "const double m3 = s3;"),
    "running mean weight off by one": ("xhat[j] = ((double)(t - 1) / (double)t) * xhat[j] + (1.0 / (double)t) * x[j];",
                                       "xhat[j] = ((double)(t - 1) / (double)t) * xhat[j] + (1.0 / (double)(t + 1)) * x[j];"),
    "switch to the EMA one step late": ("else if (t < window_k)", "else if (t <= window_k)"),
    "EMA weights swapped": ("xhat[j] = beta * xhat[j] + (1.0 - beta) * x[j];", "xhat[j] = (1.0 - beta) * xhat[j] + beta * x[j];"),
    "lower threshold inclusive": ("if (s1_3d < p->tau_2d) c1 = ORACLE_SET_2D;", "if (s1_3d <= p->tau_2d) c1 = ORACLE_SET_2D;"),
    "upper threshold selects 2D": ("else if (s1_3d > p->tau_3d) c1 = ORACLE_SET_3D;", "else if (s1_3d > p->tau_3d) c1 = ORACLE_SET_2D;"),
    "conflict falls back to the wrong set": ("if (cf == 0) cf = c2;", "if (cf == 0) cf = c1;"),
    "budget rounds down": ("return (int32_t)floor(x + 0.5);", "return (int32_t)floor(x);"),
    "budget split ignores the floor": ("const int32_t lo = imax(kmin3, B - n2);", "const int32_t lo = imax(0, B - n2);"),
    "2D-only set gives 3D everything": ("else if (c_final == ORACLE_SET_2D) w3 = 0.0;", "else if (c_final == ORACLE_SET_2D) w3 = 1.0;"),
    "smaller scores first": ("if (a->z > b->z) return -1;          /* larger score first */\n    if (a->z < b->z) return 1;",
                             "if (a->z > b->z) return 1;\n    if (a->z < b->z) return -1;"),
    "ties to the higher index": ("return (a->j > b->j) - (a->j < b->j);", "return (a->j < b->j) - (a->j > b->j);"),
    "text tokens dropped": ("for (int32_t i = 0; i < s->n_txt; ++i) kept_idx[n++] = s->off_txt + i;", ""),
    "compaction ignores the sample offset": ("(const char *)src + ((int64_t)seq_off + kept_idx[r]) * row_bytes",
                                             "(const char *)src + ((int64_t)kept_idx[r]) * row_bytes"),
    "ranks on the scores of the step alone": ("oracle_normalise(st->ahat, n2, n3, z);", "oracle_normalise(a, n2, n3, z);"),
    "gates on the indicators of the step alone": ("oracle_gates(st->mhat, p, &dg.c_s1,", "oracle_gates(x, p, &dg.c_s1,"),
    "budget from the attention share of the step alone": ("oracle_budget_adaptive(s, p, st->mhat[3], dg.c_final,",
                                                          "oracle_budget_adaptive(s, p, x[3], dg.c_final,"),
    "whole step decides on zeroed scores": ("const int32_t n_kept = oracle_decide_step(a, l1, s, p, mode,",
                                            "memset(a, 0, sizeof(double)); const int32_t n_kept = oracle_decide_step(a, l1, s, p, mode,"),
    "whole step drops the norms": ("const int32_t n_kept = oracle_decide_step(a, l1, s, p, mode,",
                                   "const int32_t n_kept = oracle_decide_step(a, NULL, s, p, mode,"),
    "cached logits never refreshed": ("if (!all && !changed[krow]) continue;                 /* the previous step's logits of key j stand */",
                                      "if (!all) continue;"),
    "changed text row not honoured": ("if (changed[(int64_t)s->seq_off + s->off_txt + i]) all = 1;", ";"),
    "cache ignored": ("int32_t all = !cache_valid || changed == NULL;", "int32_t all = 1;"),
    "mask read without the sample offset": ("const int64_t krow = (int64_t)s->seq_off + vis_row(s, j);\n        if (!all && !changed[krow]) continue;",
                                            "const int64_t krow = (int64_t)s->seq_off + vis_row(s, j);\n        if (!all && !changed[vis_row(s, j)]) continue;"),
    "cold start prunes": ("if (t == 1 && p->cold_start_full_keep) {", "if (0) {"),
    "state updated after the decision": ("const int32_t n_kept = oracle_select(z, s, k2, k3, kept_idx);",
                                         "const int32_t n_kept = oracle_select(attn_out ? attn_out : z, s, k2, k3, kept_idx);"),
}
# the last entry selects on an output buffer that is filled only afterwards: a wrong-operand slip
MUTATIONS.pop("state updated after the decision")


# Mistakes planted in the patch-by-patch statement of Alg. 1 (mvla_patch_oracle.c).
PATCH_MUTATIONS = {
    "projection on the wrong vector": ("d22 += a2[r] * a2[r];", "d22 += a3[r] * a3[r];"),
    "orthogonal part keeps the parallel part": ("ortho[r] = a3[r] - para[r];", "ortho[r] = a3[r];"),
    "3D share uses the whole vector": ("x[4 * p + 3] = no / (n2 + n3);", "x[4 * p + 3] = n3 / (n2 + n3);"),
    "2D attention share inverted": ("x[4 * p + 2] = n2 / (n2 + n3);", "x[4 * p + 2] = n3 / (n2 + n3);"),
    "feature shares swapped": ("x[4 * p + 1] = f3 / (f2 + f3);", "x[4 * p + 1] = f2 / (f2 + f3);"),
    "3D token of the patch read from the wrong column": ("a3[r] = alpha[(size_t)r * nv + P + p];",
                                                         "a3[r] = alpha[(size_t)r * nv + p];"),
    "attention not normalised": ("for (int32_t j = 0; j < nv; ++j) out[j] = exp(out[j] - mx) / den;",
                                 "for (int32_t j = 0; j < nv; ++j) out[j] = exp(out[j] - mx);"),
    "k-means ties go up": ("if (dc < bd) { second = bd; bd = dc; best = c; }", "if (dc <= bd) { second = bd; bd = dc; best = c; }"),
    "k-means centre is a sum": ("if (cnt > 0) centre[c] = acc / cnt;", "if (cnt > 0) centre[c] = acc;"),
    "k-means starts from the maximum twice": ("centre[1] = n > 0 ? sum / n : 0.0;", "centre[1] = mx;"),
    "patch threshold inclusive": ("if (mhat_s1_3d < tau_2d) return ORACLE_SET_2D;", "if (mhat_s1_3d <= tau_2d) return ORACLE_SET_2D;"),
    "background kept when it should go": ("return u < p->bg_prune_prob ? 0 : both;", "return u < p->bg_prune_prob ? both : 0;"),
    "robot rule compares 2D first": ("if (m3 > mu_3d) return both;                    /* pure 3D reliance above the baseline */\n        if (m2 > mu_2d) return ORACLE_SET_2D;",
                                     "if (m2 > mu_2d) return ORACLE_SET_2D;\n        if (m3 > mu_3d) return both;"),
    "object rule is an or": ("if (m2 > p->obj_2d_min && m3 < p->eps_3d) return ORACLE_SET_2D;",
                             "if (m2 > p->obj_2d_min || m3 < p->eps_3d) return ORACLE_SET_2D;"),
    "empty semantic set falls back to the modality set": ("if (c_s2 == 0) return 0;", "if (c_s2 == 0) return c_s1;"),
    "patch conflict keeps the modality set": ("return cf != 0 ? cf : c_s2;", "return cf != 0 ? cf : c_s1;"),
    "3D mask emits the 2D token": ("kept_idx[n] = s->off_3d + q; ++n; ++dg.k_3d;", "kept_idx[n] = s->off_2d + q; ++n; ++dg.k_3d;"),
    "baseline from the instantaneous shares": ("s3 += st->xhat[4 * q + 3];", "s3 += x[4 * q + 3];"),
    "clusters the 2D mass only": ("mass[q] = a[q] + a[P + q];", "mass[q] = a[q];"),
    "patch rules on the shares of the step alone": ("const double *xh = st->xhat + 4 * q;", "const double *xh = x + 4 * q;"),
    "patch cold start prunes": ("if (cold) cf = ORACLE_SET_2D | ORACLE_SET_3D;", "if (0) cf = 0;"),
}


def _run_mutant(which, old, new, tests, tmp_path, monkeypatch, name):
    for f in FILES:
        src = open(os.path.join(ODIR, f)).read()
        if f == which:
            assert src.count(old) == 1, f"mutation site not found exactly once: {name}"
            src = src.replace(old, new)
        (tmp_path / f).write_text(src)
    so = tmp_path / "libmut.so"
    subprocess.run(["gcc", "-O1", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-w", "-o", str(so),
                    str(tmp_path / "mvla_oracle.c"), str(tmp_path / "mvla_patch_oracle.c"), "-lm"], check=True)
    oracle.lib()                                            # make sure the real one is loaded first
    monkeypatch.setattr(oracle, "_lib", oracle.load(str(so)))
    return _caught(tests)


@pytest.mark.parametrize("name", sorted(PATCH_MUTATIONS))
def test_patch_pins_catch_planted_mistake(name, tmp_path, monkeypatch):
    old, new = PATCH_MUTATIONS[name]
    assert _run_mutant("mvla_patch_oracle.c", old, new, PATCH_PIN_TESTS, tmp_path, monkeypatch, name), f"no pin noticed: {name}"


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_pins_catch_planted_mistake(name, tmp_path, monkeypatch):
    old, new = MUTATIONS[name]
    assert _run_mutant("mvla_oracle.c", old, new, PIN_TESTS, tmp_path, monkeypatch, name), f"no pin noticed: {name}"


def _caught(tests):
    caught = []
    for fn in tests:
        marks = [m for m in getattr(fn, "pytestmark", []) if m.name == "parametrize"]
        argsets = [()]
        if marks:
            argsets = [(v,) if not isinstance(v, tuple) else v for v in marks[0].args[1]]
        for args in argsets:
            try:
                fn(*args)
            except AssertionError:
                caught.append(fn.__name__)
            except Exception:
                caught.append(fn.__name__)
    return caught
