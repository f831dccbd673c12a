"""Do the pins bite? Each case plants one plausible mistake in a copy of the oracle's C source (a
dropped factor, a wrong sign or index, swapped operands, a wrong comparison), builds it, and runs
tests/test_oracle_pins.py against that build: some pin must fail. The unchanged source, built the same
way, must pass. Nothing here touches the CUDA library."""
import os
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "speca_oracle.c")
PY_SRC = os.path.join(ROOT, "oracle", "speca_oracle.py")

# (name, text to find, replacement, which occurrence (0-based), how many occurrences the source has)
MUTANTS = [
    ("update_wrong_sign", "c[i + 1] = (c[i] - old_i) / gap[i];", "c[i + 1] = (old_i - c[i]) / gap[i];", 0, 1),
    ("update_divides_by_span_in_taylor_basis", "(basis == ORACLE_NEWTON ? t_hist[i] : t_hist[0])", "t_hist[i]", 0, 1),
    ("update_newton_divides_by_last_gap", "(basis == ORACLE_NEWTON ? t_hist[i] : t_hist[0])", "t_hist[0]", 0, 1),
    ("update_forgets_the_new_top_plane", "for (int i = 0; i <= v_new; ++i)\n            store_elem(",
     "for (int i = 0; i < v_new; ++i)\n            store_elem(", 0, 1),
    ("forecast_drops_the_factorial", "w[i] = pow(x, (double)i) / fact;", "w[i] = pow(x, (double)i);", 0, 2),
    ("forecast_offset_has_wrong_sign", "        double x = t_target - t_hist[0];\n        double fact = 1.0;",
     "        double x = t_hist[0] - t_target;\n        double fact = 1.0;", 0, 1),
    ("forecast_reads_an_undefined_plane", "int v = n_refs - 1 < m ? n_refs - 1 : m;", "int v = n_refs < m ? n_refs : m;", 0, 2),
    ("forecast_skips_the_top_order", "for (int i = 1; i <= v; ++i)\n            s += load_elem(", "for (int i = 1; i < v; ++i)\n            s += load_elem(", 0, 2),
    ("newton_nodes_all_at_the_last_reference", "w[i] = w[i - 1] * (t_target - t_hist[i - 1]);", "w[i] = w[i - 1] * (t_target - t_hist[0]);", 0, 2),
    ("adams_bashforth_wrong_coefficient", "{23.0 / 12, -16.0 / 12, 5.0 / 12, 0}", "{23.0 / 12, -16.0 / 12, 4.0 / 12, 0}", 0, 1),
    ("adams_bashforth_wrong_fourth_order_coefficient", "37.0 / 24, -9.0 / 24}", "37.0 / 24, -8.0 / 24}", 0, 1),
    ("adams_bashforth_backward_difference_sign", "hp *= -h;", "hp *= h;", 0, 1),
    ("summed_forecast_keeps_only_the_last_entry", "acc[j] += s;", "acc[j] = s;", 0, 1),
    ("summed_forecast_drops_the_factorial", "w[i] = pow(x, (double)i) / fact;", "w[i] = pow(x, (double)i);", 1, 2),
    ("summed_adams_bashforth_wrong_coefficient", "static const double gam[4] = {1.0, 1.0 / 2, 5.0 / 12, 3.0 / 8};\n", "static const double gam[4] = {1.0, 1.0 / 2, 5.0 / 12, 1.0 / 3};\n", 0, 1),
    ("bf16_store_truncates", "nearbyint(ldexp(v, 7 - lead))", "trunc(ldexp(v, 7 - lead))", 0, 1),
    ("store_rounds_the_double_directly", "float r = (float)v; /* the binary32 register that holds the result */",
     "double r = v;", 0, 1),
    ("error_normalised_by_the_forecast", "num += (p - f) * (p - f);\n        den += f * f;", "num += (p - f) * (p - f);\n        den += p * p;", 0, 1),
    ("error_without_the_square_root", "return sqrt(num) / (sqrt(den) + eps);", "return num / (sqrt(den) + eps);", 0, 1),
    ("error_epsilon_under_the_root", "return sqrt(num) / (sqrt(den) + eps);", "return sqrt(num) / sqrt(den + eps);", 0, 1),
    ("l1_without_absolute_value", "num += fabs(p - f);", "num += (p - f);", 0, 1),
    ("linf_takes_the_minimum", "if (d > num) num = d;", "if (d < num) num = d;", 0, 1),
    ("cosine_similarity_instead_of_distance", "return 1.0 - dot / (sqrt(pp) * sqrt(ff) + eps);", "return dot / (sqrt(pp) * sqrt(ff) + eps);", 0, 1),
    ("two_stage_l2_swaps_its_sums", "if (metric == 0) return sqrt(s[0]) / (sqrt(s[1]) + eps);", "if (metric == 0) return sqrt(s[1]) / (sqrt(s[0]) + eps);", 0, 1),
    ("two_stage_linf_adds_instead_of_maximising", "if (d > a0) a0 = d;", "a0 += d;", 0, 1),
    ("update_ignores_the_warm_up", "int v_new = n_refs < m ? n_refs : m;", "int v_new = m;", 0, 1),
    ("bf16_subnormals_rounded_like_normals", "if (lead < -126) lead = -126;", "if (lead < -300) lead = -300;", 0, 1),
    ("bf16_nan_becomes_infinity", "if (isnan(v)) return 0x7FC0u;", "if (isnan(v)) return 0x7F80u;", 0, 1),
    ("l1_normalised_by_the_forecast", "num += fabs(p - f);\n        den += fabs(f);", "num += fabs(p - f);\n        den += fabs(p);", 0, 1),
    ("linf_hides_a_nan", "if (bad) return NAN;", "", 0, 1),
    ("two_stage_l1_normalised_by_the_forecast", "a0 += fabs(p - f);\n            a1 += fabs(f);", "a0 += fabs(p - f);\n            a1 += fabs(p);", 0, 1),
    ("two_stage_linf_hides_a_nan", "if (bad) a0 = a1 = NAN;", "", 0, 1),
    ("summed_forecast_base_added_twice", "for (int64_t j = 0; j < n; ++j) acc[j] += load_elem(src, dtype, j);",
     "for (int64_t j = 0; j < n; ++j) acc[j] += 2.0 * load_elem(src, dtype, j);", 0, 1),
    ("history_wrong_sign", "c[i + 1] = (c[i] - d[i]) / gap;", "c[i + 1] = (d[i] - c[i]) / gap;", 0, 1),
    ("history_taylor_divides_by_span", "double gap = t_hist[k] - (basis == ORACLE_NEWTON ? t_hist[k + 1 + i] : t_hist[k + 1]);",
     "double gap = t_hist[k] - t_hist[k + 1 + i];", 0, 1),
    ("history_newton_divides_by_last_gap", "double gap = t_hist[k] - (basis == ORACLE_NEWTON ? t_hist[k + 1 + i] : t_hist[k + 1]);",
     "double gap = t_hist[k] - t_hist[k + 1];", 0, 1),
    ("history_starts_from_the_newest", "d[0] = load_elem(hist[v], dtype, j);\n    for (int k = v - 1; k >= 0; --k) {",
     "d[0] = load_elem(hist[0], dtype, j);\n    for (int k = v - 1; k >= 0; --k) {", 0, 1),
    ("history_sum_keeps_only_the_last_entry", "acc[j] += history_forecast_elem(", "acc[j] = history_forecast_elem(", 0, 1),
    ("history_drops_the_factorial", "s += d[i] * pow(x, (double)i) / fact;", "s += d[i] * pow(x, (double)i);", 0, 1),
    ("history_newton_nodes_shifted", "w *= t_target - t_hist[i - 1];", "w *= t_target - t_hist[i];", 0, 1),
    ("history_adams_bashforth_wrong_coefficient", "static const double gam[4] = {1.0, 1.0 / 2, 5.0 / 12, 3.0 / 8}; /* Adams-Bashforth, collected by plane */",
     "static const double gam[4] = {1.0, 1.0 / 2, 5.0 / 12, 1.0 / 3};", 0, 1),
    ("history_keeps_only_low_orders", "for (int i = 0; i <= v - k; ++i) d[i] = c[i];", "for (int i = 0; i < v - k; ++i) d[i] = c[i];", 0, 1),
    ("accept_is_strict", "return err <= tau ? 1 : 0;", "return err < tau ? 1 : 0;", 0, 1),
    ("threshold_decays_the_wrong_way", "pow(beta, (T - t) / T)", "pow(beta, t / T)", 0, 1),
    ("speedup_forgets_the_verification_cost", "1.0 / (1.0 - alpha + alpha * gamma)", "1.0 / (1.0 - alpha)", 0, 1),
]


# The same for the Python half of the oracle (per-sample state, masks, the continuation rule).
PY_MUTANTS = [
    ("continuation_allows_one_step_too_many", "count[b] < k_max", "count[b] <= k_max", 0, 1),
    ("continuation_counts_inactive_samples", "        if active[b]:\n            if accept_flags[b]:", "        if True:\n            if accept_flags[b]:", 0, 1),
    ("continuation_keeps_rejected_samples", "keep[b] = 1 if (accept_flags[b] and count[b] < k_max) else 0", "keep[b] = 1 if count[b] < k_max else 0", 0, 1),
    ("group_survives_if_any_member_does", "ok = all(keep[g + i] for i in range(group))", "ok = any(keep[g + i] for i in range(group))", 0, 1),
    ("update_ignores_the_sample_mask", "                elif mask[b]:\n                    update_segment(", "                else:\n                    update_segment(", 0, 1),
    ("history_update_ignores_the_sample_mask", "if mask[b] and self.layout == LAYOUT_HISTORY:", "if self.layout == LAYOUT_HISTORY:", 0, 1),
    ("commit_advances_every_sample", "            if mask[b]:\n                self.t_hist[b] =", "            if True:\n                self.t_hist[b] =", 0, 1),
    ("commit_appends_instead_of_prepending", "([float(t_ref[b])] + self.t_hist[b])[: self.m + 1]", "(self.t_hist[b] + [float(t_ref[b])])[: self.m + 1]", 0, 1),
    ("reset_keeps_the_count", "                self.n_refs[b] = 0\n", "                pass\n", 0, 1),
    ("forecast_ignores_the_active_mask", "if (active is None or active[b]) and self.n_refs[b] >= 1:\n                if self.layout == LAYOUT_HISTORY:",
     "if self.n_refs[b] >= 1:\n                if self.layout == LAYOUT_HISTORY:", 0, 1),
    ("verify_scores_inactive_samples", "if (active is None or active[b]) and self.n_refs[b] >= 1:\n                err[b] =",
     "if self.n_refs[b] >= 1:\n                err[b] =", 0, 1),
    ("verify_compares_fresh_with_itself", "err[b] = rel_err(metric, self.dtype, pred[b], fresh[b], self.eps)",
     "err[b] = rel_err(metric, self.dtype, fresh[b], fresh[b], self.eps)", 0, 1),
    ("history_appends_instead_of_prepending", "self.hist[e][b] = ([f[b].copy()] + kept)[: self.m + 1]", "self.hist[e][b] = (kept + [f[b].copy()])[: self.m + 1]", 0, 1),
    ("history_survives_a_reset", "kept = self.hist[e][b] if self.n_refs[b] >= 1 else []   # a reset sample starts over", "kept = self.hist[e][b]", 0, 1),
    ("history_keeps_one_feature_too_few", "self.hist[e][b] = ([f[b].copy()] + kept)[: self.m + 1]", "self.hist[e][b] = ([f[b].copy()] + kept)[: self.m]", 0, 1),
    ("summed_forecast_skips_the_base", "            if base is not None:\n", "            if False:\n", 0, 1),
]


def mutate(src: str, old: str, new: str, which: int, count: int) -> str:
    assert src.count(old) == count, "the oracle source changed: %r occurs %d times, expected %d" % (old, src.count(old), count)
    pos = -1
    for _ in range(which + 1):
        pos = src.index(old, pos + 1)
    return src[:pos] + new + src[pos + len(old):]


def build_and_run_pins(workdir: str, name: str, source: str):
    c_path = os.path.join(workdir, name + ".c")
    so_path = os.path.join(workdir, name + ".so")
    with open(c_path, "w") as fh:
        fh.write(source)
    subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fno-fast-math", "-ffp-contract=off", "-shared", "-fPIC", "-std=c99",
                           "-o", so_path, c_path, "-lm"])
    env = dict(os.environ, SPECA_ORACLE_LIB=so_path, OMP_NUM_THREADS="2")
    res = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_oracle_pins.py"), "-x", "-q",
                          "-p", "no:cacheprovider"], cwd=ROOT, env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT,
                         text=True, timeout=600)
    return res.returncode, res.stdout


def run_pins_on_python_variant(workdir: str, name: str, source: str):
    """A private copy of the few files the pins need, with the oracle's Python module replaced."""
    top = os.path.join(workdir, name)
    os.makedirs(os.path.join(top, "oracle"))
    os.makedirs(os.path.join(top, "tests"))
    open(os.path.join(top, "oracle", "__init__.py"), "w").close()
    with open(os.path.join(top, "oracle", "speca_oracle.py"), "w") as fh:
        fh.write(source)
    for f in ("__init__.py", "conftest.py", "test_oracle_pins.py"):
        shutil.copy(os.path.join(ROOT, "tests", f), os.path.join(top, "tests", f))
    shutil.copytree(os.path.join(ROOT, "tests", "golden"), os.path.join(top, "tests", "golden"))
    from oracle import speca_oracle
    env = dict(os.environ, SPECA_ORACLE_LIB=speca_oracle.build(), OMP_NUM_THREADS="2")
    env["PYTHONPATH"] = ROOT   # for the workload shapes one pin reads; the copy's own folder comes first
    res = subprocess.run([sys.executable, "-m", "pytest", os.path.join(top, "tests", "test_oracle_pins.py"), "-x", "-q",
                          "-p", "no:cacheprovider", "--rootdir", top], cwd=top, env=env, stdout=subprocess.PIPE,
                         stderr=subprocess.STDOUT, text=True, timeout=600)
    return res.returncode, res.stdout


def test_every_mistake_planted_in_the_python_half_fails_a_pin(tmp_path):
    src = open(PY_SRC).read()
    jobs = [("unchanged", src)] + [(name, mutate(src, old, new, which, count)) for name, old, new, which, count in PY_MUTANTS]
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 2)) as pool:
        results = list(pool.map(lambda job: run_pins_on_python_variant(str(tmp_path), job[0], job[1]), jobs))
    rc, out = results[0]
    assert rc == 0, "the unchanged oracle fails its own pins in the private copy:\n" + out[-2000:]
    survivors = [name for (name, _), (rc, _) in zip(jobs[1:], results[1:]) if rc == 0]
    assert not survivors, "no pin notices: %s" % ", ".join(survivors)
    for (name, _), (rc, out) in zip(jobs[1:], results[1:]):
        assert rc == 1 and " failed" in out, "%s: pytest ended with %d\n%s" % (name, rc, out[-800:])


def test_every_planted_mistake_fails_a_pin(tmp_path):
    src = open(SRC).read()
    jobs = [("unchanged", src)] + [(name, mutate(src, old, new, which, count)) for name, old, new, which, count in MUTANTS]
    assert len({name for name, _ in jobs}) == len(jobs)
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 2)) as pool:
        results = list(pool.map(lambda job: build_and_run_pins(str(tmp_path), job[0], job[1]), jobs))
    rc, out = results[0]
    assert rc == 0, "the unchanged oracle fails its own pins:\n" + out[-2000:]
    survivors = [name for (name, _), (rc, _) in zip(jobs[1:], results[1:]) if rc == 0]
    assert not survivors, "no pin notices: %s" % ", ".join(survivors)
    # the failures are pin failures, not build or collection errors
    for (name, _), (rc, out) in zip(jobs[1:], results[1:]):
        assert rc == 1 and " failed" in out, "%s: pytest ended with %d\n%s" % (name, rc, out[-800:])
