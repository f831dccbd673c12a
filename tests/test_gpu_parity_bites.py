"""Does the parity gate bite? The GPU parity tests compare the CUDA library with the oracle; here a
mistake is planted in a copy of the ORACLE's C source (never in the CUDA path), and a few of those
parity tests are run against that build: they must fail. A tolerance loose enough to hide a dropped
factorial, a wrong sign or a wrong norm would show up here as a planted mistake that still passes."""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

import pytest

from tests.test_oracle_mutants import MUTANTS, SRC, mutate

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
TABLES = ["tests/test_gpu_parity.py", "-k", "tiny_config or verify_entry_spanning or masks_leave"]
METRICS = ["tests/test_gpu_metrics.py", "-k", "many_tiles"]
SUMS = ["tests/test_gpu_sum.py", "-k", "matches_oracle"]
BASES = ["tests/test_gpu_parity.py", "-k", "ragged_shapes and (3-1-0-3 or 3-1-1-3 or 3-2-0-3 or 3-2-1-3)"]   # order 3, Newton and Adams-Bashforth
# which parity tests must notice which planted mistake
CASES = {
    "update_wrong_sign": TABLES,
    "update_divides_by_span_in_taylor_basis": TABLES,
    "update_newton_divides_by_last_gap": BASES,
    "update_forgets_the_new_top_plane": TABLES,
    "forecast_drops_the_factorial": TABLES,
    "forecast_offset_has_wrong_sign": TABLES,
    "forecast_skips_the_top_order": TABLES,
    "newton_nodes_all_at_the_last_reference": BASES,
    "adams_bashforth_wrong_coefficient": BASES,
    "summed_forecast_keeps_only_the_last_entry": SUMS,
    "bf16_store_truncates": ["tests/test_gpu_parity.py", "-k", "verify_entry_spanning or model_shaped"],
    "error_normalised_by_the_forecast": TABLES,
    "error_without_the_square_root": TABLES,
    "l1_without_absolute_value": METRICS,
    "linf_takes_the_minimum": METRICS,
    "cosine_similarity_instead_of_distance": METRICS,
}


def run_parity(workdir, name, source, selection):
    so_path = os.path.join(workdir, name + ".so")
    if source is not None:
        c_path = os.path.join(workdir, name + ".c")
        with open(c_path, "w") as fh:
            fh.write(source)
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fno-fast-math", "-ffp-contract=off", "-shared", "-fPIC", "-std=c99",
                               "-o", so_path, c_path, "-lm"])
    env = dict(os.environ, SPECA_ORACLE_LIB=so_path, OMP_NUM_THREADS="4")
    res = subprocess.run([sys.executable, "-m", "pytest"] + selection + ["-x", "-q", "-m", "gpu", "-p", "no:cacheprovider"],
                         cwd=ROOT, env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True, timeout=900)
    return res.returncode, res.stdout


def test_parity_tests_fail_on_a_mistaken_oracle(tmp_path):
    src = open(SRC).read()
    by_name = {name: (old, new, which, count) for name, old, new, which, count in MUTANTS}
    # the unchanged source, built the same way, passes every selection used below
    selections = []
    for sel in CASES.values():
        if sel not in selections:
            selections.append(sel)
    run_parity(str(tmp_path), "unchanged", src, ["tests/test_gpu_parity.py", "-k", "tiny_config"])  # builds unchanged.so
    jobs = [("unchanged", None, sel) for sel in selections] + \
           [(name, mutate(src, *by_name[name]), sel) for name, sel in CASES.items()]
    with ThreadPoolExecutor(max_workers=6) as pool:
        results = list(pool.map(lambda j: run_parity(str(tmp_path), j[0], j[1], j[2]), jobs))
    for (name, _, sel), (rc, out) in zip(jobs, results):
        if name == "unchanged":
            assert rc == 0, "parity selection %r fails on the unchanged oracle:\n%s" % (sel, out[-1500:])
        else:
            assert rc == 1 and " failed" in out, "planted mistake %s goes unnoticed by %r (exit %d)\n%s" % (name, sel, rc, out[-800:])
