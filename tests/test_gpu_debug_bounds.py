"""The build with address checks in the kernels (-DLQ_DEBUG_BOUNDS: every global or shared-memory access whose index
derives from a caller's size, stride, group or block offset is checked against the buffers the entry point was given; a
miss is recorded in the status word as LQ_ERR_INVALID_ARG and the access skipped) runs the tiny, ragged and odd-shaped
cases of the parity suite: they must pass as they do with the normal build, which also means that no access fell outside
-- the tests read the status word after every call.  Stands in for a memory checker on shapes far from the tile sizes."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CASES = ("tiny_and_ragged or stage1_hessian or stage1_token_major or stage1_empty or stage2_prepare or stage2_dead or "
         "stage3_nonuniform or stage3_grouped or stage3_weighted or stage3_degenerate or stage3_affine or stage4 or lazy_refit or pack_codes or "
         "activation_order or act_order or record or stack_of_layers or chained_affine or noalloc")


def test_parity_cases_under_the_bounds_checking_build():
    if os.environ.get("LQ_LIBRARY_VARIANT") == "debug":
        pytest.skip("already inside the debug run")
    env = dict(os.environ, LQ_LIBRARY_VARIANT="debug")
    cmd = [sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "-p", "no:cacheprovider", "-k", CASES,
           os.path.join(ROOT, "tests", "test_gpu_parity.py"), os.path.join(ROOT, "tests", "test_gpu_record.py"),
           os.path.join(ROOT, "tests", "test_zz_no_alloc.py")]
    out = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    tail = "\n".join(out.stdout.splitlines()[-25:])
    assert out.returncode == 0, tail
    assert " passed" in tail and "failed" not in tail, tail
