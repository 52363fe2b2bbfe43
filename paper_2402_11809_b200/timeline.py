"""In-kernel clock trace of one step's kernel chain (attention, merge, verify + commit) in CUDA-graph replay.

The kernels carry optional %globaltimer stamps (compiled in with -DSPACE_TIMELINE; see csrc/attn_tc.cu and
csrc/verify.cu).  This module builds a second copy of the library with them, libspace_timeline.so, next to
the regular one, replays a graph of eight steps of a single-sequence workload and prints, in microseconds
after the attention kernel's dependency wait of the last step: when the attention blocks pass their stages
(regular groups and helper groups apart), when the merge and verify blocks become resident, when their
dependency waits return and when they finish.  What a kernel boundary costs and where a launch spends its
time cannot be seen from outside the kernels: a profiler serialises the launches.

Usage: python -m paper_2402_11809_b200.timeline [workload]      (default llama7b; needs a B200)
"""
import ctypes as C
import os
import subprocess
import sys

import numpy as np

from . import build as _build

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_TL = os.path.join(HERE, "libspace_timeline.so")


def build_timeline_library():
    srcs = [os.path.join(_build.CSRC, s) for s in _build.SOURCES]
    deps = [os.path.join(_build.CSRC, f) for f in os.listdir(_build.CSRC)]
    if os.path.exists(LIB_TL) and all(os.path.getmtime(d) <= os.path.getmtime(LIB_TL) for d in deps):
        return LIB_TL
    cmd = [_build._nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-shared",
           "-Xcompiler", "-fPIC", "-cudart", "static", "-DSPACE_TIMELINE"] + srcs + ["-o", LIB_TL]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return LIB_TL


def main(argv):
    import torch
    _build.build()
    from . import binding as B, workloads, device as H
    lib = C.CDLL(build_timeline_library())
    for name in B.EXPORTS:                                   # the same ABI: swap the library under the binding
        f, g = getattr(B.lib, name), getattr(lib, name)
        g.argtypes, g.restype = f.argtypes, f.restype
    B.lib = lib
    name = argv[1] if len(argv) > 1 else "llama7b"
    cfg = workloads.resolve(name)
    if cfg["B"] != 1:
        raise SystemExit("the trace is laid out for one sequence (regular and helper groups)")
    k = cfg["k"]
    sets = [workloads.make_step_inputs(cfg, set_index=i) for i in range(8)]
    ctx = B.Context(device=0, max_batch=1, n_q_heads=cfg["H_q"], n_kv_heads=cfg["H_kv"], head_dim=cfg["d"],
                    k_max=k, vocab=cfg["V"], s_cap=sets[0]["s_cap"])
    ds = [H.DeviceStep(cfg, x) for x in sets]

    def step(i):
        ds[i % 8].attn(ctx)
        ds[i % 8].verify_commit(ctx)

    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        for i in range(16):
            step(i)
        st.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=st):
            for i in range(8):
                step(i)
        for _ in range(10):
            g.replay()
        st.synchronize()

    def read(fn, n_blocks, points):
        buf = (C.c_ulonglong * (n_blocks * points))()
        fn.argtypes, fn.restype = [C.c_void_p, C.c_int], C.c_int
        assert fn(buf, n_blocks) == 0
        return np.array(buf[:], dtype=np.int64).reshape(n_blocks, points)

    A = read(lib.space_debug_timeline_read, 148, 16)
    M = read(lib.space_debug_timeline_read_merge, 4096, 4)
    V = read(lib.space_debug_timeline_read_verify, 4096, 8)
    t0 = A[:, 2][A[:, 2] > 0].min()                          # the attention's dependency wait returns
    us = lambda x: (np.asarray(x) - t0) / 1e3
    n_reg = (148 // cfg["H_kv"]) * cfg["H_kv"]
    names = {3: "first request", 12: "S^T issuer at its first wait", 4: "first K tile in use", 5: "first S^T ready",
             6: "first P ready", 8: "last S^T ready", 9: "last P ready", 10: "last O^T done", 11: "partial stored",
             13: "exit"}
    print(f"{name}: one step of a graph of eight, microseconds after the attention's dependency wait returned")
    for cls, sel in (("regular groups", np.arange(148) < n_reg), ("helper groups", np.arange(148) >= n_reg)):
        if not sel.any():
            continue
        print(f"  attention, {cls} ({int(sel.sum())} blocks): median / max")
        for i, nm in names.items():
            v = us(A[sel, i][A[sel, i] > 0])
            if len(v):
                print(f"    {nm:30s} {np.median(v):6.2f} / {v.max():6.2f}")
    # the stamps of the last launch of each kernel: its dependency wait returned after the attention's (t0);
    # a point a block did not pass in that launch still holds an older stamp and is left out
    M, V = M[M[:, 1] > t0], V[V[:, 1] > t0]
    after = lambda T, col: T[:, col][T[:, col] > T[:, 1].min()]
    print(f"  attention: last block out {us(A[:, 13]).max():.2f}")
    print(f"  merge ({len(M)} blocks): resident {us(M[:, 0]).min():.2f} .. {us(M[:, 0]).max():.2f}; wait returned "
          f"{us(M[:, 1]).min():.2f}; descriptor in registers {us(after(M, 2)).min():.2f} .. {us(after(M, 2)).max():.2f}; "
          f"output stored {us(after(M, 3)).min():.2f} .. {us(after(M, 3)).max():.2f}")
    fin = V[V[:, 5] > V[:, 1].min()]
    print(f"  verify + commit ({len(V)} blocks): resident {us(V[:, 0]).min():.2f} .. {us(V[:, 0]).max():.2f}; wait returned "
          f"{us(V[:, 1]).min():.2f}; logits in registers {us(V[:, 2]).min():.2f} .. {us(V[:, 2]).max():.2f}; counted in "
          f"{us(V[:, 3]).min():.2f} .. {us(V[:, 3]).max():.2f}; finishing block: rows reduced "
          f"{us(fin[:, 4]).max():.2f}, done {us(fin[:, 5]).max():.2f}")


if __name__ == "__main__":
    main(sys.argv)
