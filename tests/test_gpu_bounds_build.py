"""The index-check build of the library (-DLQ_DEBUG_BOUNDS): the kernels check every index that comes from the
host's bookkeeping against the extent of the store it goes to; a failing check sets bit 2 of the status word and
skips the access.  (A stand-in for a memory checker.)  The small parity cases must run through it with a clean
status word, and a deliberately wrong index must be caught."""
import os
import subprocess
import sys

import pytest

from paper_2503_19950_b200 import build

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def bounds_env():
    env = dict(os.environ)
    env["LOGQUANT_LIBRARY"] = build.build(bounds=True)
    return env


def test_small_parity_cases_pass_under_the_index_checks(bounds_env):
    # run_case asserts a zero status word at its end: no check may fire on a correct run
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
           os.path.join(ROOT, "tests", "test_gpu_parity.py"), os.path.join(ROOT, "tests", "test_gpu_umma.py"),
           "-k", "config1 or shapes_and_edge_cases or four_bit_cache or left_padded or one_launch"]
    res = subprocess.run(cmd, env=bounds_env, cwd=ROOT, capture_output=True, text=True, timeout=1500)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-2000:]
    assert " passed" in res.stdout


_CATCH = r"""
import torch
from paper_2503_19950_b200 import LogQuantCache, binding, synth
assert "bounds" in binding._LIB_PATH
c = LogQuantCache(1, 1, 8, 2, 32, 32, max_tokens=256)
k, v = synth.keys_values(3, 1, 2, 40, 128, "cuda")
c.append(0, k[:, :, :20].contiguous(), v[:, :, :20].contiguous())
before = {key: val.copy() for key, val in c.export(0).items()}
assert c.kernel_status() == 0
c.debug_bad_slot_next_append()
c.append(0, k[:, :, 20:].contiguous(), v[:, :, 20:].contiguous())
torch.cuda.synchronize()
assert c.kernel_status() == 4, c.kernel_status()
assert c.check_guards() == 0
print("caught")
"""


def test_a_wrong_slot_is_caught_by_the_index_checks(bounds_env):
    res = subprocess.run([sys.executable, "-c", _CATCH], env=bounds_env, cwd=ROOT, capture_output=True, text=True,
                         timeout=600)
    assert res.returncode == 0 and "caught" in res.stdout, res.stdout[-2000:] + res.stderr[-2000:]


def test_the_normal_build_refuses_the_hook():
    from paper_2503_19950_b200 import LogQuantCache, LogQuantError, binding
    if os.environ.get("LOGQUANT_LIBRARY"):
        pytest.skip("running against another build of the library")
    c = LogQuantCache(1, 1, 8, 2, 32, 32, max_tokens=64)
    with pytest.raises(LogQuantError) as e:
        c.debug_bad_slot_next_append()
    assert e.value.status == binding.LQ_ERR_UNSUPPORTED
    c.close()
