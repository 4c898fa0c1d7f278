"""The alternative kernels (warp-specialised, fused single-role) against the oracle.

The variant is chosen once per process from the HPCTOPK_VARIANT environment variable, so each
one runs in a child process."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.mark.parametrize("variant", ["0", "100", "2"])
def test_variant_matches_oracle(variant):
    env = dict(os.environ, HPCTOPK_VARIANT=variant)
    out = subprocess.run([sys.executable, os.path.join(HERE, "variant_check.py")], env=env, capture_output=True,
                         text=True, timeout=600)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    assert "variant ok" in out.stdout
