"""The parity suite once more on the checking build of the library.

libxnor_check.so is libxnor.so compiled with -DXNOR_BOUNDS_CHECK: the tensor-core BinConv kernel
then compares every shared-memory address its producers compute (weight stages, patch planes,
the raw input rows) and every global index its epilogue stores to with the extent of the buffer,
skips an access that fails and records it, and xnor_check_device reports XNOR_ERR_BOUNDS.  The
parity tests call xnor_check_device after every convolution, so running them against that
build fails on the first address outside its buffer (together with the guard words around the
output buffers this stands in for a memory checker).  A subprocess, because a process loads
one build of the library."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.gpu
def test_parity_suite_on_the_checking_build():
    from paper_1603_05279_b200 import build as b
    lib = b.build(bounds_check=True)
    assert os.path.exists(lib)
    env = dict(os.environ, XNOR_LIB=os.path.basename(lib))
    probe = subprocess.run([sys.executable, "-c",
                            "import paper_1603_05279_b200 as X; print(X.xnor_built_with_bounds_check())"],
                           cwd=ROOT, env=env, capture_output=True, text=True)
    assert probe.returncode == 0 and probe.stdout.strip() == "1", probe.stderr
    files = ["tests/test_gpu_parity.py", "tests/test_gpu_fused.py", "tests/test_gpu_options.py",
             "tests/test_gpu_timed_paths.py::test_every_sweep_point",
             "tests/test_gpu_timed_paths.py::test_layers_at_full_batch_without_acc_out"]
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider"] + files,
                       cwd=ROOT, env=env, capture_output=True, text=True)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-1000:]
