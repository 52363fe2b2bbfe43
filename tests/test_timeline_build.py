"""The optional in-kernel clock stamps (-DSPACE_TIMELINE, read by paper_2402_11809_b200.timeline) must keep
compiling: the regular build leaves them out, so nothing else would notice if they rotted."""
import os
import subprocess

import pytest

from paper_2402_11809_b200 import build

CSRC = build.CSRC


@pytest.mark.parametrize("src,symbols", [
    ("attn_tc.cu", ["space_debug_timeline_read", "space_debug_timeline_read_merge"]),
    ("verify.cu", ["space_debug_timeline_read_verify"]),
])
def test_instrumented_sources_compile_and_export_their_readers(tmp_path, src, symbols):
    obj = tmp_path / (src + ".o")
    cmd = [build._nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-Xcompiler", "-fPIC",
           "-DSPACE_TIMELINE", "-c", os.path.join(CSRC, src), "-o", str(obj)]
    res = subprocess.run(cmd, capture_output=True, text=True)
    assert res.returncode == 0, res.stderr[-2000:]
    names = subprocess.run(["nm", "-g", "--defined-only", str(obj)], capture_output=True, text=True).stdout
    for s in symbols:
        assert f" T {s}" in names, (s, names[-500:])
