"""The checked build of the library (libkvsched_checked.so, -DKVSCHED_CHECKED): every index a kernel
derives from data or from its own arithmetic is range-checked before use, an index that leaves its
array is recorded and replaced by 0, and the host call reports SCHED_E_INTERNAL.  It stands in for a
memory checker: the small-instance parity tests are run once more against it, in a child process
(the library is chosen when the binding is first loaded), and must pass unchanged -- which also
means that no index was ever out of range.  The check itself is shown to fire on an out-of-range
value through a probe call that accesses nothing."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
pytestmark = pytest.mark.gpu

SMALL_CASES = ("small_random or paper_example or long_waits or every_simulator_shape or shared_memory_timelines or "
               "full_neighbourhood_tiny or random_small_instances or sorted_f_matches or sorted_f_example1 or "
               "local_swap_matches or quantile_greedy or online_policies_match or amin_small or tiny_backlog_all_solvers or "
               "policy_sweep_small or odd_sizes or start_times_checker or local_search_tiny or local_search_random or "
               "sampled_and_resume or bounds_checked_on_the_device or 8_byte_aligned")

_PROBE = r"""
import sys
sys.path.insert(0, sys.argv[1])
import torch
from paper_2508_06133_b200 import binding as kv
torch.cuda.set_device(0)
assert kv.CHECKED and kv.LIB_PATH.endswith("libkvsched_checked.so")
assert kv.build_flags() & kv.BUILD_CHECKED
kv.debug_check_index(0, 10)
kv.debug_check_index(9, 10)
for bad in (10, -1, 1 << 35):
    try:
        kv.debug_check_index(bad, 10)
    except kv.SchedError as e:
        assert e.code == kv.E_INTERNAL, e.code
        assert "site 9999" in kv.load().sched_last_cuda_error().decode()
    else:
        raise SystemExit("index %d was not reported" % bad)
kv.debug_check_index(3, 10)          # the record was cleared: in-range indices pass again
print("checked-probe-ok")
"""


def _env():
    env = dict(os.environ)
    env["KVSCHED_CHECKED"] = "1"
    return env


def test_checked_build_reports_an_index_outside_its_array():
    lib = os.path.join(ROOT, "paper_2508_06133_b200", "libkvsched_checked.so")
    assert os.path.exists(lib), "checked library not built: python -m paper_2508_06133_b200.build --checked"
    r = subprocess.run([sys.executable, "-c", _PROBE, ROOT], env=_env(), capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "checked-probe-ok" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]


def test_small_parity_cases_pass_on_the_checked_build():
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_gpu_parity.py"), "-m", "gpu",
                        "-x", "-q", "-p", "no:cacheprovider", "-k", SMALL_CASES],
                       env=_env(), capture_output=True, text=True, timeout=3000, cwd=ROOT)
    tail = r.stdout[-3000:] + r.stderr[-2000:]
    assert r.returncode == 0, tail
    assert " passed" in r.stdout and "failed" not in r.stdout, tail


def test_the_normal_build_is_not_the_checked_one():
    from paper_2508_06133_b200 import binding as kv
    if kv.CHECKED:
        pytest.skip("this session itself runs on the checked build")
    assert kv.build_flags() == 0
    with pytest.raises(kv.SchedError) as e:
        kv.debug_check_index(0, 1)
    assert e.value.code == kv.E_UNSUPPORTED
