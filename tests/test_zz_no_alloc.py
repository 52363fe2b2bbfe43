"""space_verify_greedy_noalloc: greedy verification for callers that must not
allocate device memory (a process whose GPU memory is entirely owned by its own
pool, or a decode loop that cannot tolerate the synchronisation an allocation may
cause).  Its scratch is a fixed array inside the library, so it needs no context.

The test calls it through the C ABI twice in a row, on different inputs, and
checks every output against space_verify (the context-based entry point) on the
same inputs: integers exactly, probabilities to 1e-4 relative, as in the other
GPU tests.  It lives in its own file, collected last.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2402_11809_b200 import workloads

pytestmark = pytest.mark.gpu


def _outputs(ds):
    return dict(n_accept=ds.n_accept.cpu().numpy().copy(), out_tokens=ds.out_tokens.cpu().numpy().copy(),
                n_out=ds.n_out.cpu().numpy().copy(), next_cand=ds.next_cand.cpu().numpy().copy(),
                next_cand_prob=ds.next_cand_prob.cpu().numpy().copy(),
                finished=ds.finished.cpu().numpy().copy())


def _poison(ds):
    ds.n_accept.fill_(-7); ds.out_tokens.fill_(-7); ds.n_out.fill_(-7); ds.next_cand.fill_(-7)
    ds.next_cand_prob.fill_(float("nan")); ds.finished.fill_(9)


def test_noalloc_matches_space_verify_on_two_calls_in_a_row():
    from paper_2402_11809_b200 import build
    build.build()
    from paper_2402_11809_b200 import binding as B
    import gpu_harness as H

    cases = [dict(B=3, k=5, V=32000, dtype="bf16", seed=901, eos=False),
             dict(B=B.NOALLOC_MAX_BATCH, k=2, V=1003, dtype="f32", seed=902, eos=True)]
    runs = []
    for cs in cases:
        cfg = workloads.resolve("tiny", B=cs["B"], H_q=1, H_kv=1, d=64, L=(5, 40), k=cs["k"], V=cs["V"],
                                logits_dtype=cs["dtype"], sigma=2.0, p_accept=(0.6, 0.6), seed=cs["seed"])
        x = workloads.make_step_inputs(cfg)
        ctx = H.make_context(cfg, x)
        ds = H.DeviceStep(cfg, x)
        # reference: the context-based entry point
        a = ds.verify(ctx)
        torch.cuda.synchronize()
        eos = int(ds.out_tokens[0, 0]) if cs["eos"] else -1
        if cs["eos"]:
            a = ds.verify(ctx, eos_id=eos)
            torch.cuda.synchronize()
        runs.append((ctx, ds, a, _outputs(ds), eos))

    # two calls in a row through the allocation-free entry point
    for ctx, ds, a, want, eos in runs:
        _poison(ds)
        before = torch.cuda.memory_allocated()
        rc = B.lib.space_verify_greedy_noalloc(C.byref(a), C.c_void_p(torch.cuda.current_stream().cuda_stream))
        assert rc == B.OK, B.space_strerror(rc)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        got = _outputs(ds)
        for name in ("n_accept", "out_tokens", "n_out", "next_cand", "finished"):
            assert np.array_equal(got[name], want[name]), name
        np.testing.assert_allclose(got["next_cand_prob"], want["next_cand_prob"], rtol=1e-4, atol=1e-30)
    assert runs[1][3]["finished"][0] == 1 and runs[0][3]["n_accept"].max() > 0

    # sizes beyond the fixed scratch and unsupported modes are refused, not run
    ctx, ds, a, _, _ = runs[0]
    bad = B.VerifyArgs.from_buffer_copy(a); bad.batch = B.NOALLOC_MAX_BATCH + 1
    assert B.lib.space_verify_greedy_noalloc(C.byref(bad), None) == B.E_STATIC_LIMIT
    assert "NOALLOC" in B.space_strerror(B.E_STATIC_LIMIT)
    bad = B.VerifyArgs.from_buffer_copy(a); bad.mode = B.MODE_SAMPLE
    assert B.lib.space_verify_greedy_noalloc(C.byref(bad), None) == B.E_INVALID_ARG
    bad = B.VerifyArgs.from_buffer_copy(a); bad.logits = None
    assert B.lib.space_verify_greedy_noalloc(C.byref(bad), None) == B.E_INVALID_ARG
    assert B.lib.space_verify_greedy_noalloc(None, None) == B.E_INVALID_ARG
    torch.cuda.synchronize()
