"""The C ABI on its own: a C program (tests/c_abi/gpu_roundtrip.c) that uses only speca.h and the CUDA
runtime -- no Python, no torch in its process -- runs reference steps, a forecast, the verification and
the continuation rule on the GPU and writes its results to a file; this test regenerates the program's
inputs (a 32-bit linear congruential generator) and compares the file with the oracle."""
import os
import subprocess
import types

import numpy as np
import pytest

from oracle import speca_oracle as O

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
TIMES = [[1.00, 0.99, 1.01], [0.93, 0.92, 0.95], [0.90, 0.0, 0.91]]
MASK2 = [1, 0, 1]
TARGET = [0.86, 0.88, 0.87]


def lcg_values(state, n):
    """n values of the program's generator, continuing from `state`; returns (float32 array, state)."""
    out = np.empty(n, dtype=np.float64)
    for i in range(n):
        state = (state * 1664525 + 1013904223) & 0xFFFFFFFF
        out[i] = (state >> 8) / 8388608.0 - 1.0
    return out.astype(np.float32), state


@pytest.fixture(scope="module")
def exe(tmp_path_factory):
    from paper_2509_11628_b200 import build
    lib = build.build()
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    out = str(tmp_path_factory.mktemp("c_abi") / "gpu_roundtrip")
    subprocess.check_call(["gcc", "-std=c11", "-Wall", "-Wextra", "-Werror", "-I", os.path.join(ROOT, "include"),
                           "-I", os.path.join(cuda, "include"), os.path.join(ROOT, "tests", "c_abi", "gpu_roundtrip.c"),
                           "-L", os.path.dirname(lib), "-lspeca", "-L", os.path.join(cuda, "lib64"), "-lcudart_static",
                           "-ldl", "-lpthread", "-lrt", "-Wl,-rpath," + os.path.dirname(lib), "-o", out])
    return out


@pytest.mark.parametrize("fused", [False, True])     # True: the last reference step and the forecast as one call
@pytest.mark.parametrize("basis", [O.TAYLOR, O.NEWTON, O.ADAMS_BASHFORTH])
def test_c_program_matches_oracle(exe, tmp_path, basis, fused):
    from tests import gpu_util as U
    path = str(tmp_path / "out.bin")
    res = subprocess.run([exe, path, str(basis)] + (["fused"] if fused else []), stdout=subprocess.PIPE,
                         stderr=subprocess.STDOUT, text=True, timeout=120)
    assert res.returncode == 0 and res.stdout.strip().endswith("ok"), res.stdout
    raw = open(path, "rb").read()
    B, ne, m, basis_got, n_steps = np.frombuffer(raw, np.int32, 5)
    assert (B, ne, m, basis_got, n_steps) == (3, 3, 2, basis, 3)
    shapes = np.frombuffer(raw, np.int32, 2 * ne, 20).reshape(ne, 2)
    elems = [int(n) * int(d) for n, d in shapes]
    off = 20 + 8 * ne
    fresh = np.frombuffer(raw, np.float32, B * elems[-1], off).reshape(B, -1)
    off += 4 * B * elems[-1]
    got = []
    for e in range(ne):
        got.append(np.frombuffer(raw, np.float32, B * elems[e], off).reshape(B, -1))
        off += 4 * B * elems[e]
    err = np.frombuffer(raw, np.float32, B, off); off += 4 * B
    accept = np.frombuffer(raw, np.uint8, B, off); off += B
    nxt = np.frombuffer(raw, np.uint8, B, off); off += B
    cnt = np.frombuffer(raw, np.int32, B, off); off += 4 * B
    n_active = int(np.frombuffer(raw, np.int32, 1, off)[0]); off += 4
    assert off == len(raw)

    cpu = O.OracleCache(elems, B, m, O.F32, basis)
    state = 2509
    for step in range(n_steps):
        feats = []
        for e in range(ne):
            v, state = lcg_values(state, B * elems[e])
            feats.append(v.reshape(B, -1))
        cpu.update(feats, TIMES[step], MASK2 if step == 2 else None)
        cpu.commit_step()
    assert cpu.n_refs == [3, 2, 3]
    view = types.SimpleNamespace(cpu=cpu, m=m, basis=basis)
    for e in range(ne):
        want = cpu.forecast_entry(e, TARGET)
        for b in range(B):
            scale = U.term_scale(cpu.planes[e][b], U.Pair.forecast_weights(view, b, TARGET[b]))
            U.assert_close_storage(got[e][b], want[b], O.F32, scale, "entry %d sample %d" % (e, b))
    tau = [float(np.float32(0.05))] * B
    e_want, a_want, _ = cpu.verify(fresh, TARGET, tau)
    for b in range(B):
        assert abs(float(err[b]) - e_want[b]) <= U.ERR_TOL * max(1.0, e_want[b]), (b, err[b], e_want[b])
    assert err[0] < 1e-5 and 0.001 < err[1] < 0.05 < err[2]          # the three noise levels the program adds
    assert accept.tolist() == [int(a) for a in a_want] == [1, 1, 0]
    want_act, want_cnt, want_idx = O.select_adaptive([int(a) for a in a_want], 4, 1, [0] * B, [1] * B)
    assert nxt.tolist() == want_act and cnt.tolist() == want_cnt and n_active == len(want_idx)
