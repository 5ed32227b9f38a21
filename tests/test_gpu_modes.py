"""The library's environment switches select other launch forms of the same kernels: resident grids
whose blocks loop over rows and prefetch through shared-memory rings (FS_PERSISTENT=1), the
register-resident cluster kernel (FS_CLUSTER_REGS=1), launches without programmatic dependent
launch (FS_PDL=0), the L2 prefetch off or a whole generation ahead (FS_PREFETCH_PCT=0 / 100), the first wave of a one-shot
grid started all at once (FS_LAG_BW=0). Each form gets the same oracle parity sweep, in a child process
because the switches are read once per process."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.mark.parametrize("env", [
    {},
    {"FS_PERSISTENT": "1"},
    {"FS_CLUSTER_REGS": "1"},
    {"FS_PERSISTENT": "1", "FS_CLUSTER_REGS": "1"},
    {"FS_PDL": "0"},
    {"FS_PREFETCH_PCT": "0"},
    {"FS_PREFETCH_PCT": "100"},
    {"FS_LAG_BW": "0"},
], ids=lambda e: ",".join(f"{k}={v}" for k, v in e.items()) or "default")
def test_parity_in_every_launch_form(env):
    full = dict(os.environ)
    for k in ("FS_PERSISTENT", "FS_CLUSTER_REGS", "FS_PDL", "FS_PREFETCH_PCT", "FS_LAG_BW"):
        full.pop(k, None)
    full.update(env)
    out = subprocess.run([sys.executable, os.path.join(HERE, "mode_check.py")], env=full, capture_output=True,
                         text=True, timeout=900)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    assert "mode_check ok" in out.stdout
