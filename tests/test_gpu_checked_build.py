"""The bounds-checked build of the library (`python -m paper_2508_05700_b200.build --checked`, every
kernel index tested against its array, violations reported through MFET_DEV_BOUNDS): the tiny
hand-computed cases, the random shapes, the staging windows, the host-table path, dedup, backward
and the guard-band tests run on it in a child process and must pass with no bit set (the tests
themselves assert a clean error word after every call)."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_parity_and_guard_tests_pass_on_the_bounds_checked_build():
    from paper_2508_05700_b200 import build
    lib = build.build(checked=True)
    env = dict(os.environ, MFET_LIBRARY=lib)
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
           "tests/test_gpu_random_shapes.py", "tests/test_gpu_canaries.py", "tests/test_gpu_backward.py",
           "tests/test_gpu_parity.py", "-k",
           "random_shape or canaries or guard or checked_build_reports or backward or tiny_bags or staging_windows or "
           "host_table_path or dedup_bit_exact or cache_probe or int4_host or facets_concat or 2_to_32"]
    r = subprocess.run(cmd, cwd=ROOT, env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True, timeout=1500)
    tail = r.stdout[-3000:]
    assert r.returncode == 0, tail
    assert " passed" in tail and "checked_build_reports" not in tail.split("short test summary")[-1], tail
