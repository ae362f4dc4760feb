"""The checked build of the library (-DSPECS_DEBUG) on the GPU.

It stands in for a memory checker: every kernel tests the indices of its global-memory accesses and
raises SPECS_DEV_BOUNDS instead of touching memory outside its buffers, and it carries the plain
CUDA-core scoring engine as a second GPU implementation.  The parity tests that exercise tile edges,
ragged tails, the second scoring pass and the device-detected conditions are run again on it, in a
child process (the library is chosen when the binding is first imported), and must pass with a clean
status word -- which their own fixtures assert.
"""
import os
import subprocess
import sys

import pytest

from paper_2506_15733_b200 import binding, build

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_default_build_has_neither_the_checks_nor_the_simt_engine():
    if binding.debug_build():
        pytest.skip("this process runs the checked build")
    ctx = binding.Context(0)
    with pytest.raises(binding.SpecsError) as e:
        ctx.set_engine(binding.ENGINE_SIMT)
    assert e.value.status == 2
    ctx.close()


def test_parity_subset_on_the_checked_build():
    if binding.debug_build():
        pytest.skip("already inside the checked build")
    assert os.path.exists(build.LIB_PATH_DEBUG), "build the checked library: python -m paper_2506_15733_b200.build --debug"
    env = dict(os.environ, SPECS_B200_DEBUG="1")
    select = ("tiny or edge or empty or multi_wave or out_of_range or rescore or one_large or buffers or host_steps "
              "or fused or garbage or random_shapes or vocab_sharded")
    res = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_gpu_parity.py"), "-m", "gpu",
                          "-x", "-q", "-k", select], cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    tail = res.stdout[-2000:] + res.stderr[-2000:]
    assert res.returncode == 0, tail
    assert " passed" in res.stdout and "failed" not in res.stdout, tail
