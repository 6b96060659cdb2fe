"""The debug-bounds build of the library (every global-memory address a kernel computes is checked
against the buffers of its call and an outside address is skipped and reported, never accessed):
what stands in for a memory checker on machines where none can be run.  The build is exercised in a
child process, because a process loads one library: the child runs the parity tests of the tiny
configuration and of the ragged and unaligned shapes against the debug library, where every test
ends with sbp_check_device_errors() (tests/conftest.py)."""
import os
import subprocess
import sys

import pytest
import torch
from conftest import ROOT

import paper_2110_15032_b200 as sbp

pytestmark = pytest.mark.gpu

# config 1 (all six signatures, the chain, boxing on the results), ragged / unaligned / strided shapes
# of every operator; the full-size cases stay with the normal build (the checks cost 10-50x)
SELECT = ("config1 or ragged or unaligned or degenerate or edges or windows or view or nd_every_axis or "
          "to_partial or cast_fused or disjoint_2d or disjoint_3d or embedding_parity or hidden_axis or "
          "backward_parity or xent_parity or static_scratch or fused_classifier_ragged or two_axis_boxing")


@pytest.fixture(scope="module")
def debug_library():
    from paper_2110_15032_b200.build import build
    return build(debug_bounds=True)


def _child(debug_library, args, timeout=1500):
    env = dict(os.environ, SBP_B200_LIBRARY=debug_library)
    return subprocess.run([sys.executable] + args, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_debug_bounds_build_reports_a_refused_address_without_touching_it(debug_library):
    assert not sbp.sbp_debug_bounds_enabled()          # this process runs the normal build
    code = (
        "import torch, paper_2110_15032_b200 as sbp\n"
        "assert sbp.sbp_debug_bounds_enabled()\n"
        "buf = torch.zeros(64, dtype=torch.uint8, device='cuda')\n"
        "sbp.sbp_selftest_debug_bounds(buf[:32])\n"
        "torch.cuda.synchronize()\n"
        "try:\n"
        "    sbp.sbp_check_device_errors()\n"
        "    raise SystemExit('no report')\n"
        "except sbp.SbpError as e:\n"
        "    assert e.name == 'SBP_ERR_BOUNDS', e.name\n"
        "sbp.sbp_check_device_errors()\n"                                  # reported once, then clear
        "assert buf[0].item() == 1 and int(buf[1:].sum().item()) == 0\n"   # the refused byte was not written
        "print('ok')\n")
    r = _child(debug_library, ["-c", code])
    assert r.returncode == 0 and r.stdout.strip().endswith("ok"), r.stdout[-2000:] + r.stderr[-2000:]
    with pytest.raises(sbp.SbpError) as e:              # the normal build has no such self-test
        sbp.sbp_selftest_debug_bounds(torch.zeros(8, dtype=torch.uint8, device="cuda"))
    assert e.value.name == "SBP_ERR_UNSUPPORTED"


def test_parity_tests_of_small_and_ragged_shapes_pass_under_the_debug_bounds_build(debug_library):
    r = _child(debug_library, ["-m", "pytest", "tests", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
                               "--deselect", "tests/test_debug_bounds_gpu.py", "-k", SELECT])
    tail = r.stdout[-3000:] + r.stderr[-2000:]
    assert r.returncode == 0, tail
    last = r.stdout.strip().splitlines()[-1]
    assert " passed" in last and "failed" not in last, tail
    assert int(last.split(" passed")[0].split()[-1]) >= 150, last     # the selection really selected
