"""The C interface used from plain C: tests/c_abi/restore_prefix.c includes only include/bsr.h and
the CUDA runtime.  On CPU it must compile as C11 and link against the built library; on a GPU it
runs a seeded case end to end and everything it writes is compared with the oracle."""
import os
import shutil
import subprocess

import numpy as np
import pytest

from harness import Case, run_oracle
from oracle import bsr_oracle as O
from paper_2608_17826_b200 import build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "tests", "c_abi", "restore_prefix.c")
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


def _compile(out_dir):
    lib = build.build()
    exe = os.path.join(str(out_dir), "restore_prefix")
    cmd = ["gcc", "-std=c11", "-Wall", "-Werror", "-O1", "-I", os.path.join(ROOT, "include"),
           "-I", os.path.join(CUDA, "include"), SRC, "-o", exe,
           "-L", os.path.dirname(lib), "-lbsr", "-L", os.path.join(CUDA, "lib64"), "-lcudart",
           "-Wl,-rpath," + os.path.dirname(lib), "-Wl,-rpath," + os.path.join(CUDA, "lib64")]
    res = subprocess.run(cmd, capture_output=True, text=True)
    assert res.returncode == 0, res.stderr
    return exe


@pytest.mark.skipif(shutil.which("gcc") is None, reason="no C compiler")
def test_c_caller_compiles_as_c11_and_links(tmp_path):
    assert os.path.exists(_compile(tmp_path))


@pytest.mark.gpu
@pytest.mark.parametrize("layout_name,R,N,W", [("tiny", 2, 21, 4), ("hetero", 2, 5, 2)])
def test_c_caller_restores_a_prefix_bit_exactly(tmp_path, layout_name, R, N, W):
    layout = {"tiny": synth.tiny_layout, "hetero": synth.hetero_layout}[layout_name]()
    case = Case(layout, R, N, seed=1700 + N, reg_id=9)
    ora = run_oracle(case, W)
    assert ora["status"] == O.OK
    d = str(tmp_path)
    with open(os.path.join(d, "case.txt"), "w") as f:
        f.write(f"{R} {N} {W} {case.G} {len(layout.tensors)} {case.salt} {case.reg_id}\n")
        for g in range(case.G):
            f.write(f"{layout.block_tokens[g]} {case.pools[g]}\n")
        for g, e in layout.tensors:
            f.write(f"{g} {e}\n")
    case.tok[: N * 256].astype("<i4").tofile(os.path.join(d, "tokens.bin"))
    for r in range(R):
        np.concatenate([case.payload[(r, i)] for i in range(N)]).tofile(os.path.join(d, f"payload_r{r}.bin"))
        np.array([case.cks[(r, i)] for i in range(N)], dtype="<u8").tofile(os.path.join(d, f"ck_r{r}.bin"))
        for g in range(case.G):
            np.asarray(case.tables[r][g], dtype="<i4").tofile(os.path.join(d, f"table_r{r}_g{g}.bin"))
    exe = _compile(tmp_path)
    res = subprocess.run([exe, d], capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stdout + res.stderr
    n_hit, exposed, peak = (int(x) for x in open(os.path.join(d, "result.txt")).read().split())
    assert n_hit == exposed == ora["exposed"] == N
    assert peak == ora["stats"].peak_staging_bytes[0] == min(N, W) * case.reg.slot_bytes
    assert np.array_equal(np.fromfile(os.path.join(d, "keys.bin"), dtype="<u8"), ora["keys"])
    assert np.array_equal(np.fromfile(os.path.join(d, "bitmap.bin"), dtype="<u8"),
                          np.asarray(ora["req"].bitmap()).ravel())
    for r in range(R):
        for l in range(len(layout.tensors)):
            got = np.fromfile(os.path.join(d, f"paged_r{r}_l{l}.bin"), dtype=np.uint8)
            assert np.array_equal(got, ora["paged"][r][l].ravel()), (r, l)
