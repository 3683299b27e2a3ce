"""Host-side check of the multiply-and-shift division the kernels use for divisors fixed at launch
(ratio, group size): exact for every non-negative int below 2^31.  Compiles the library's own header with g++."""
import shutil
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
CUDA_INC = Path("/usr/local/cuda/include")

SRC = r"""
#include <cstdio>
#include <cstdint>
#include "ug_common.cuh"
int main() {
  long long bad = 0;
  const int ds[] = {1, 2, 3, 4, 5, 7, 8, 12, 16, 31, 32, 33, 100, 127, 128, 129, 640, 1000, 4096, 4097, 16384, 65535,
                    65536, 1000003, (1 << 30) - 1, 1 << 30, 0x7fffffff};
  for (int d : ds) {
    const ug::FastDiv f = ug::make_fastdiv(d);
    uint32_t x = 12345u;
    for (int i = 0; i < 400000; ++i) {
      x = x * 1664525u + 1013904223u;
      const int n = i < 100000 ? i : (int)(x >> 1);
      bad += ug::fdiv(f, n) != n / d;
    }
    const int edge[] = {0, d - 1, d, d < 0x7fffffff ? d + 1 : d, 0x7fffffff, 0x7ffffffe};
    for (int n : edge) bad += ug::fdiv(f, n) != n / d;
  }
  std::printf("%lld\n", bad);
  return bad != 0;
}
"""


@pytest.mark.skipif(shutil.which("g++") is None or not CUDA_INC.exists(), reason="needs g++ and the CUDA headers")
def test_fastdiv_is_exact(tmp_path):
    src = tmp_path / "fastdiv.cpp"
    src.write_text(SRC)
    exe = tmp_path / "fastdiv"
    subprocess.check_call(["g++", "-O1", "-std=c++17", "-I", str(CUDA_INC), "-I", str(ROOT / "include"),
                           "-I", str(ROOT / "paper_2509_15763_b200" / "csrc"), str(src), "-o", str(exe)])
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0 and out.stdout.strip() == "0", out.stdout + out.stderr
