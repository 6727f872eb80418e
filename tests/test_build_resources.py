"""What the compiler made of the weight-streaming GEMM: every variant must leave room for two CTAs per SM (the
decode-step launches rely on two resident CTAs with a ring each) and spill nothing.  An epilogue change that blows
up the register count still passes every numerical test and silently costs 20 % of the step: this catches it on the
CPU machine (ptxas reports registers per thread at compile time)."""
import os
import re
import subprocess

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "paper_2511_21759_b200", "csrc", "gemm_tcgen05.cu")


def test_gemm_variants_fit_two_ctas_per_sm_and_spill_nothing():
    r = subprocess.run(["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-Xptxas", "-v", "-c", SRC,
                        "-o", os.devnull], capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stderr[-2000:]
    blocks = re.split(r"ptxas info\s*: Compiling entry function '", r.stderr)[1:]
    seen = 0
    for b in blocks:
        name = b.split("'", 1)[0]
        if "gemm_kernel" not in name:
            continue
        regs = int(re.search(r"Used (\d+) registers", b).group(1))
        spills = [int(x) for x in re.findall(r"(\d+) bytes spill", b)]
        seen += 1
        # 192 threads per CTA, 65536 registers per SM: two CTAs need at most 170 registers per thread
        assert regs <= 128, (name, regs)
        assert not any(spills), (name, spills)
    assert seen == 24          # 4 row-tile sizes x 3 epilogues x {single CTA, CTA pair}
