"""The alternative kernels against the oracle: warp-specialised (0), fused single-role (100),
another launch shape (2), and the single kernel for every call shape (4; the default takes the
three-kernel pipeline for calls of more than 512 rows).

The variant is chosen once per process from an environment variable, so each one runs in a child
process."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.mark.parametrize("variant", ["0", "100", "2", "4"])
def test_variant_matches_oracle(variant):
    env = dict(os.environ, HPCTOPK_VARIANT=variant)
    out = subprocess.run([sys.executable, os.path.join(HERE, "variant_check.py")], env=env, capture_output=True,
                         text=True, timeout=600)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    assert "variant ok" in out.stdout
