"""The bulk install kernel's stage recycling, made observable.

The product build streams about ten 16 KiB tiles through each shared-memory stage of a CTA, so a
stage handed back to the loader too early (while its store is still reading it, or before the
checksum warps are done with it) has few chances to show.  A second build of the same source with
three 1 KiB stages, one lagging store and at most 32 CTAs per launch recycles every stage hundreds
of times per CTA; the byte-for-byte parity cases of the bulk kernel are run against that build in
a child process (the binding loads the library named by BSR_LIBRARY)."""
import os
import subprocess
import sys

import pytest

from conftest import ROOT

pytestmark = pytest.mark.gpu

CASES = ("test_bulk_install_kernel_matches_oracle or test_bulk_install_kernel_detects_corruption "
         "or test_more_tiles_per_chunk_than_ctas_in_the_grid or test_many_pipeline_shapes_give_the_same_bytes "
         "or test_install_launches_carry_the_configured_number_of_chunks or test_bounded_wait_inside or test_spans_of_several_short_runs or test_stores_of_long_runs_followed")


def test_bulk_kernel_parity_cases_on_the_small_stage_build():
    from paper_2608_17826_b200 import build
    lib = build.build_stress()
    env = dict(os.environ, BSR_LIBRARY=lib)
    out = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_gpu_parity.py"),
                          "-m", "gpu", "-x", "-q", "-k", CASES], capture_output=True, text=True, env=env,
                         cwd=ROOT, timeout=1500)
    assert out.returncode == 0, out.stdout[-3000:] + out.stderr[-1000:]
    assert " passed" in out.stdout and "failed" not in out.stdout
