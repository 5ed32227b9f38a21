"""The library's environment switches select other launch forms of the same kernels: launches without
programmatic dependent launch (FS_PDL=0), no prefetch ahead of the dependency wait (FS_EARLY_PF=0), rows that are not a multiple of 16 bytes on the element-wise kernel only (FS_SHIFT=0), the L2 prefetch off or a whole generation ahead (FS_PREFETCH_PCT=0 / 100),
the first wave of a one-shot grid started all at once (FS_LAG_BW=0), a device simulated without cluster launch or
with little shared memory (FS_SIM_NO_CLUSTER=1, FS_SIM_SMEM_OPTIN), pointer validation and logging (FS_CHECK=1,
FS_LOG=1). Each form gets the same oracle parity sweep, in a child process because the switches are read once per
process."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.mark.parametrize("env", [
    {},
    {"FS_SIM_NO_CLUSTER": "1"},
    {"FS_SIM_SMEM_OPTIN": "65536"},
    {"FS_CHECK": "1", "FS_LOG": "1"},
    {"FS_PDL": "0"},
    {"FS_EARLY_PF": "0"},
    {"FS_SHIFT": "0"},
    {"FS_PREFETCH_PCT": "0"},
    {"FS_PREFETCH_PCT": "100"},
    {"FS_LAG_BW": "0"},
], ids=lambda e: ",".join(f"{k}={v}" for k, v in e.items()) or "default")
def test_parity_in_every_launch_form(env):
    full = dict(os.environ)
    for k in [k for k in full if k.startswith("FS_")]:
        full.pop(k)
    full.update(env)
    out = subprocess.run([sys.executable, os.path.join(HERE, "mode_check.py")], env=full, capture_output=True,
                         text=True, timeout=900)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    assert "mode_check ok" in out.stdout
