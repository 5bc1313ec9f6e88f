"""The small-shape parity suite under the checked build of the library (-DRABIT_CHECKED): every index that addresses
memory in the decode kernels (table-driven and f16 GEMV) is compared with its range first, a violation sets the layer's status word and
skips the access.  This stands in for a memory checker: the suite must pass with a clear status word.  The checked library
is a separate file (librabit_checked.so) selected through RABIT_LIBRARY, so it runs in a child process."""
import importlib.util
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_small_shapes_pass_under_the_checked_build():
    spec = importlib.util.spec_from_file_location("_rabit_build", os.path.join(ROOT, "paper_2602_05367_b200", "build.py"))
    build = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(build)
    lib = build.LIB_CHECKED
    sources = [os.path.join(build.CSRC, f) for f in os.listdir(build.CSRC)]
    if not os.path.exists(lib) or any(os.path.getmtime(f) > os.path.getmtime(lib) for f in sources):
        build.build(checked=True)
    env = dict(os.environ, RABIT_LIBRARY=lib)
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", os.path.join(ROOT, "tests", "test_gpu_parity.py"),
           os.path.join(ROOT, "tests", "test_gpu_group.py"), "-k", "small_shapes or structured or outlier or repeated or group"]
    proc = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=1200)
    assert proc.returncode == 0, proc.stdout[-3000:] + proc.stderr[-2000:]
    assert " passed" in proc.stdout
