"""The checking build of the library (-DLPMM_DEBUG: guard zones behind every arena sub-buffer, per-tile index checks
that report through the device status word) over the shape zoo, every schedule and every quantizer variant. It runs in
a process of its own because a process binds to one build of the library."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))


def test_shape_zoo_under_the_checking_build():
    out = subprocess.run([sys.executable, os.path.join(HERE, "checking_build_script.py")], capture_output=True, text=True,
                         timeout=900)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    assert out.stdout.strip().splitlines()[-1].startswith("OK "), out.stdout[-2000:]
