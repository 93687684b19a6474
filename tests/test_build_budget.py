"""Register budget of the dominant kernel, checked at build time (nvcc cross-compiles without a
GPU): four CTAs of 128 threads per SM need at most 128 registers per thread, and the all-node
variants for 64 elements per thread may spill a few words at most (with 2-byte logits their CTAs
leave almost no L1 for spill traffic: a variant that spilled 48 bytes lost 15 %)."""
import os
import re
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
NVCC = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"

PROBE = """
#include "mcsd_device.cuh"
void *f0() { return (void *)mcsd::node_kernel<MCSD_DTYPE_F32, 64, false, false>; }
void *f1() { return (void *)mcsd::node_kernel<MCSD_DTYPE_BF16, 64, false, false>; }
void *f2() { return (void *)mcsd::node_kernel<MCSD_DTYPE_F16, 64, false, false>; }
"""


@pytest.mark.skipif(not os.path.exists(NVCC), reason="nvcc not available")
def test_headline_node_kernels_fit_their_register_budget(tmp_path):
    src = tmp_path / "probe.cu"
    src.write_text(PROBE)
    cmd = [NVCC, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-Xptxas", "-v",
           "-I", os.path.join(ROOT, "include"), "-I", os.path.join(ROOT, "paper_2401_06706_b200", "csrc"),
           "-c", str(src), "-o", str(tmp_path / "probe.o")]
    out = subprocess.run(cmd, capture_output=True, text=True, check=True).stderr
    blocks = re.findall(r"Compiling entry function '(\S+node_kernelILi(\d)ELi64ELb0ELb0E\S*)'.*?(\d+) bytes spill stores, "
                        r"(\d+) bytes spill loads.*?Used (\d+) registers", out, flags=re.S)
    assert len(blocks) == 3, out
    for _, dtype, st, ld, regs in blocks:
        assert int(regs) <= 128
        limit = 16 if dtype in ("1", "2") else 32
        assert int(st) <= limit and int(ld) <= limit, (dtype, st, ld)
