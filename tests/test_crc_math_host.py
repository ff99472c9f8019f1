"""The checksum arithmetic of the GPU kernels, run on the CPU (the helpers are host/device
functions) and compared with the bit-serial definitions and with the oracle's CRC-64."""
import os
import shutil
import subprocess

import numpy as np
import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def checker(tmp_path_factory):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    if not os.path.exists(nvcc) and shutil.which("nvcc") is None:
        pytest.skip("nvcc not available")
    exe = str(tmp_path_factory.mktemp("crc") / "crc_math_check")
    subprocess.check_call([nvcc, "-O2", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a",
                           "-I", os.path.join(ROOT, "include"),
                           "-I", os.path.join(ROOT, "paper_2607_28633_b200", "csrc"),
                           os.path.join(ROOT, "tests", "native", "crc_math_check.cu"), "-o", exe])
    return exe


@pytest.mark.parametrize("run,runs,layers", [(576, 45, 3), (1024, 33, 2), (16, 7, 1), (48, 100, 4),
                                             (256, 64, 1), (1024, 1, 5)])
def test_device_checksum_arithmetic_on_the_host(checker, run, runs, layers):
    out = subprocess.run([checker, str(run), str(runs), str(layers)], capture_output=True, text=True,
                         timeout=300)
    assert out.returncode == 0, out.stdout + out.stderr
    tag, r, n, l, crc = out.stdout.split()
    assert tag == "ok" and (int(r), int(n), int(l)) == (run, runs, layers)
    msg = ((7 * np.arange(run * runs * layers, dtype=np.int64) + 3) % 256).astype(np.uint8)
    assert int(crc, 16) == oracle.crc64(msg.tobytes())
