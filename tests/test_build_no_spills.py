"""The product kernel's producer / issuer warps run with 56 or 72 registers after setmaxnreg; a few spilled values in
their loops cost a quarter of the throughput of the balanced kernels.  Compile the file with ptxas statistics and
require every instantiation to be spill-free."""
import os
import re
import shutil
import subprocess
import tempfile

import pytest

from paper_2609_26077_b200 import build as B


@pytest.mark.skipif(shutil.which(B.NVCC) is None and not os.path.exists(B.NVCC), reason="nvcc not available")
def test_product_kernel_has_no_register_spills():
    src = os.path.join(B.CSRC, "fmm_gemm.cu")
    with tempfile.TemporaryDirectory() as tmp:
        cmd = [B.NVCC] + B.FLAGS + ["-Xptxas", "-v", "-c", src, "-o", os.path.join(tmp, "g.o")]
        out = subprocess.run(cmd, capture_output=True, text=True)
    assert out.returncode == 0, out.stderr[-2000:]
    text = out.stderr + out.stdout
    entries = re.findall(r"Compiling entry function '([^']*fmm_gemm_kernel[^']*)'.*?\n.*?\n\s*(\d+) bytes stack frame, (\d+) bytes spill stores, (\d+) bytes spill loads", text)
    assert len(entries) >= 8, "ptxas statistics not found"
    bench = ("ILi128ELi3ELi32ELi2", "ILi256ELi1ELi32ELi2")
    bad = [(name[-60:], st, ld) for name, _, st, ld in entries if int(st) or int(ld)]
    assert not bad, f"register spills in {bad}"
    assert all(any(b in name for name, *_ in entries) for b in bench), "benchmark kernels not found"
