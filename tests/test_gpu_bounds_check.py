"""The bounds-check build of the library (-DRELAY_BOUNDS_CHECK): a subset of the small-shape parity tests runs against it in a
child process; every test there ends with a poll of the device error word, so an address computed outside a call's
tensors anywhere in the memory-bound or SIMT kernels fails the run (the access itself is skipped, nothing faults)."""
import os
import subprocess
import sys

import pytest

from paper_1810_00952_b200 import binding as B

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def child(code_or_args, use_pytest=True):
    env = dict(os.environ, RELAY_B200_LIB=B.CHECK_LIB_PATH)
    cmd = [sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", *code_or_args] if use_pytest else [sys.executable, "-c", code_or_args]
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)


def test_check_build_exists_and_reports_a_failed_check():
    assert os.path.exists(B.CHECK_LIB_PATH), "build it with `python -m paper_1810_00952_b200.build --check`"
    r = child("import torch\n"
              "from paper_1810_00952_b200 import binding as B\n"
              "torch.zeros(1, device='cuda:0')\n"
              "B.relay_debug_bounds_probe()\n"
              "try:\n    B.relay_poll_status()\n    print('no report')\n"
              "except B.RelayError as e:\n    print(e.status_name, '|', e)\n"
              "B.relay_poll_status(); print('cleared')\n", use_pytest=False)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "ERR_CUDA" in r.stdout and "bounds check" in r.stdout and "cleared" in r.stdout, r.stdout + r.stderr
    with pytest.raises(B.RelayError) as e:            # the ordinary build carries no checks
        B.relay_debug_bounds_probe()
    assert e.value.status_name == "ERR_UNSUPPORTED"


def test_small_shape_parity_subset_passes_with_bounds_checks():
    r = child(["tests/test_gpu_ewise.py", "tests/test_gpu_ewise_vm.py", "tests/test_gpu_dense.py", "-k",
               "not full_size and not fixed_unit and not ragged_edges and not sampled"])
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
