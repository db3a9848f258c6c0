"""The checked build of the library (range-checked indices, status word instead of a trap): the cases of
tests/checked_cases.py run in a process of their own, because the library is chosen when the binding is
imported (TIGA_CHECKED=1)."""
import os
import subprocess
import sys

import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))


def test_checked_build_flags_bad_indices_and_stays_quiet_on_good_ones():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    lib = os.path.join(os.path.dirname(HERE), "paper_2609_24802_b200", "libtiga_checked.so")
    assert os.path.exists(lib), "libtiga_checked.so is missing: python -m paper_2609_24802_b200.build"
    env = dict(os.environ, TIGA_CHECKED="1")
    res = subprocess.run([sys.executable, os.path.join(HERE, "checked_cases.py")], env=env, capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-4000:]
    assert "all cases passed" in res.stdout


def test_normal_build_reports_no_checks():
    from paper_2609_24802_b200 import api
    assert not api.is_checked_build()
    assert api.checked_status() == 0
