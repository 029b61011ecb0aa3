"""The stand-alone hardware probes compile for sm_100a (they are run by hand on a GPU machine, see their module docstring)."""
import os
import subprocess
import tempfile

import pytest

from paper_2609_22335_b200 import probes


@pytest.mark.parametrize("name", probes.PROBES)
def test_probe_compiles(name):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    if not os.path.exists(nvcc):
        pytest.skip("nvcc not found")
    with tempfile.TemporaryDirectory() as tmp:
        r = subprocess.run([nvcc, "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-o", os.path.join(tmp, name),
                            os.path.join(probes.HERE, name + ".cu")], capture_output=True, text=True)
        assert r.returncode == 0, r.stderr[-2000:]


def test_unknown_probe_is_rejected():
    with pytest.raises(ValueError):
        probes.run("no_such_probe")
