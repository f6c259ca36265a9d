"""The L2-stream microbenchmark behind the roofline argument of the two tile kernels: compiles
tests/microbench/l2_streams.cu with nvcc, runs it and prints its table (gathers of 1 KB query pieces with
cp.async, fp32 vector reductions, and the two together).  The numbers are the ceiling the key-block-major
attention kernel is compared with; the test only checks that the benchmark runs and reports sane rates."""
import os
import shutil
import subprocess

import pytest

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))


def test_l2_stream_microbenchmark_runs_and_reports(tmp_path):
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    exe = str(tmp_path / "l2_streams")
    subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3",
                    os.path.join(HERE, "microbench", "l2_streams.cu"), "-o", exe], check=True)
    out = subprocess.run([exe], check=True, capture_output=True, text=True, timeout=300).stdout
    print(out)
    rates = {}
    for line in out.splitlines():
        if " TB/s" in line:
            name = line[:44].strip()
            rates[name] = float(line.split(" ms")[1].split("TB/s")[0])
    assert len(rates) == 13 and all(0.5 < r < 20.0 for r in rates.values()), rates


def test_tma_row_box_microbenchmark_runs_and_reports(tmp_path):
    """The same query gather through the copy engine (tests/microbench/tma_rows.cu): one TMA box of 4 adjacent rows x
    128 bytes per (token, slab) instead of 16-byte cp.async copies.  Prints the table; checks that it ran, that no
    bounded wait ran out and that the rates are sane."""
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    exe = str(tmp_path / "tma_rows")
    subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3",
                    os.path.join(HERE, "microbench", "tma_rows.cu"), "-o", exe], check=True)
    out = subprocess.run([exe], check=True, capture_output=True, text=True, timeout=300).stdout
    print(out)
    assert "ran out" not in out and "error" not in out
    rates = [float(line.split(" ms")[1].split("TB/s")[0]) for line in out.splitlines() if " TB/s" in line]
    assert len(rates) == 5 and all(0.5 < r < 20.0 for r in rates), rates
