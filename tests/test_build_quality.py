"""Host-side guard on what the compiler made of the hot decode kernel (no GPU needed): the two token
loops of the staged kernel are sized for 640 threads per CTA (at most 102 registers per thread), and
spills inside them cost several per cent of the headline number.  ptxas reports registers and spills;
this test keeps them where the measured numbers were taken."""
import os
import re
import shutil
import subprocess
import tempfile

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")


@pytest.mark.skipif(not os.path.exists(NVCC), reason="nvcc not installed")
def test_staged_decode_kernel_has_no_spills():
    src = os.path.join(ROOT, "paper_2512_17917_b200", "csrc", "kvr_decode_staged.cu")
    with tempfile.TemporaryDirectory() as tmp:
        r = subprocess.run([NVCC, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-Xptxas", "-v",
                            "-I", os.path.join(ROOT, "include"), "-I", os.path.dirname(src), "-c", src,
                            "-o", os.path.join(tmp, "staged.o")], capture_output=True, text=True)
    assert r.returncode == 0, r.stderr[-2000:]
    blocks = re.findall(r"Compiling entry function '(\S*decode_staged_kernel\S*)'.*?\n.*?\n\s*(\d+) bytes stack frame, "
                        r"(\d+) bytes spill stores, (\d+) bytes spill loads\n.*?Used (\d+) registers", r.stderr)
    assert len(blocks) == 12, "expected the twelve instantiations (fp16 / bf16 x G = 1, 2, 4 x median / mean)"
    for name, stack, st, ld, regs in blocks:
        # a few loop-invariant words may live on the stack (set-up values that are used once per pass)
        limit = 32
        assert int(st) <= limit and int(ld) <= limit, f"{name}: {st} B spill stores, {ld} B spill loads"
        assert int(regs) <= 102, f"{name}: {regs} registers (640 threads per CTA need <= 102)"
