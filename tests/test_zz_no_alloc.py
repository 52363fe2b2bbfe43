"""space_verify_greedy_noalloc: greedy verification for callers that must not
allocate device memory -- a serving process that has handed all of the GPU's
memory to its own pool (nothing is left for cudaMalloc), or a decode loop that
cannot take the device-wide synchronisation an allocation may cause.  Its
scratch is a fixed array inside the library image, so it needs no context.

The test calls it through the C ABI, first before any context exists in this
test and then twice in a row on different inputs, and checks every output
against the CPU oracle (oracle.verify.verify_step) and against space_verify
(the context-based entry point): integers exactly, probabilities to 1e-4
relative, as in the other GPU tests.  One case passes a logits pointer and a
row stride that are not 16-byte aligned, which takes the kernel's element-wise
path.  The driver's free-memory figure (cudaMemGetInfo, which sees every
allocation of the process, not only torch's) must not move across the calls.
It lives in its own file, collected last.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle.verify import verify_step
from paper_2402_11809_b200 import workloads

pytestmark = pytest.mark.gpu

NAMES = ("n_accept", "out_tokens", "n_out", "next_cand", "finished")


def _outputs(ds):
    return dict(n_accept=ds.n_accept.cpu().numpy().copy(), out_tokens=ds.out_tokens.cpu().numpy().copy(),
                n_out=ds.n_out.cpu().numpy().copy(), next_cand=ds.next_cand.cpu().numpy().copy(),
                next_cand_prob=ds.next_cand_prob.cpu().numpy().copy(),
                finished=ds.finished.cpu().numpy().copy())


def _poison(ds):
    ds.n_accept.fill_(-7); ds.out_tokens.fill_(-7); ds.n_out.fill_(-7); ds.next_cand.fill_(-7)
    ds.next_cand_prob.fill_(float("nan")); ds.finished.fill_(9)


def _verify_args(B, ds, logits, row_stride, eos_id):
    """space_verify_args built without a context (the marshalling needs none)."""
    p = lambda t: C.c_void_p(t.data_ptr())
    return B.VerifyArgs(batch=ds.cand.shape[0], k=ds.k, vocab=ds.cfg["V"],
                        logits_dtype=B.DTYPE_F32 if logits.dtype == torch.float32 else B.DTYPE_BF16,
                        mode=B.MODE_GREEDY, resample=B.RESAMPLE_RESIDUAL_POINTMASS, eos_id=eos_id,
                        temperature=1.0, seed=0, logits=p(logits), logits_row_stride=row_stride,
                        cand=p(ds.cand), cand_prob=p(ds.cand_prob), seq_id=None, kv_len=p(ds.kv_len),
                        n_accept=p(ds.n_accept), out_tokens=p(ds.out_tokens), n_out=p(ds.n_out),
                        next_cand=p(ds.next_cand), next_cand_prob=p(ds.next_cand_prob),
                        finished=p(ds.finished), status=p(ds.status))


def _check(got, want, what):
    for name in NAMES:
        assert np.array_equal(got[name], want[name]), f"{what}: {name}"
    np.testing.assert_allclose(got["next_cand_prob"], want["next_cand_prob"], rtol=1e-4, atol=1e-30)


def test_noalloc_matches_oracle_and_space_verify_on_two_calls_in_a_row():
    from paper_2402_11809_b200 import build
    build.build()
    from paper_2402_11809_b200 import binding as B
    import gpu_harness as H

    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    cases = [dict(B=3, k=5, V=32000, dtype="bf16", seed=901, eos=False, unaligned=False),
             dict(B=B.NOALLOC_MAX_BATCH, k=2, V=1003, dtype="f32", seed=902, eos=True, unaligned=False),
             dict(B=2, k=3, V=4099, dtype="bf16", seed=903, eos=False, unaligned=True)]
    prepared = []
    for cs in cases:
        cfg = workloads.resolve("tiny", B=cs["B"], H_q=1, H_kv=1, d=64, L=(5, 40), k=cs["k"], V=cs["V"],
                                logits_dtype=cs["dtype"], sigma=2.0, p_accept=(0.6, 0.6), seed=cs["seed"])
        x = workloads.make_step_inputs(cfg)
        ds = H.DeviceStep(cfg, x)
        logits, stride = ds.logits, cs["V"]
        if cs["unaligned"]:
            # rows V + 1 elements apart, starting one element into a buffer: neither the base
            # nor the row pitch is a multiple of 16 bytes
            n_rows = cs["B"] * x["n_q"]
            buf = torch.zeros(n_rows * (cs["V"] + 1) + 1, dtype=ds.logits.dtype, device="cuda")
            view = buf[1:].view(n_rows, cs["V"] + 1)[:, :cs["V"]]
            view.copy_(ds.logits.view(n_rows, cs["V"]))
            logits, stride = view, cs["V"] + 1
            assert logits.data_ptr() % 16 != 0
            ds._keep = buf
        r = verify_step(x["logits"], x["cand"], x["cand_prob"], cs["k"], "greedy")
        eos = int(r["out_tokens"][0, 0]) if cs["eos"] else -1
        if cs["eos"]:
            r = verify_step(x["logits"], x["cand"], x["cand_prob"], cs["k"], "greedy", eos_id=eos)
        prepared.append((cfg, x, ds, _verify_args(B, ds, logits, stride, eos), r, eos))
    torch.cuda.synchronize()

    # ---- the calls that must not allocate: before any context of this test exists ----
    cfg, x, ds, a, r, eos = prepared[0]
    rc = B.lib.space_verify_greedy_noalloc(C.byref(a), stream)     # warm-up: the first call on a device
    assert rc == B.OK, B.space_strerror(rc)                        # loads the module and looks the array up
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    got = []
    for cfg, x, ds, a, r, eos in prepared:                          # calls in a row, different inputs
        _poison(ds)
        rc = B.lib.space_verify_greedy_noalloc(C.byref(a), stream)
        assert rc == B.OK, B.space_strerror(rc)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "the allocation-free entry point changed the device's free memory"
    for cfg, x, ds, a, r, eos in prepared:
        got.append(_outputs(ds))
        _check(got[-1], r, f"noalloc vs oracle, seed {cfg['seed']}")
        assert int(ds.status.abs().sum()) == 0
    assert prepared[1][4]["finished"][0] == 1 and prepared[0][4]["n_accept"].max() > 0

    # a second round on the same inputs: the shared array keeps the last call's contents and
    # the counters must have been cleared
    for (cfg, x, ds, a, r, eos), g in zip(prepared, got):
        _poison(ds)
        rc = B.lib.space_verify_greedy_noalloc(C.byref(a), stream)
        assert rc == B.OK
        torch.cuda.synchronize()
        _check(_outputs(ds), r, "second round")

    # ---- the context-based entry point gives the same results ----
    for (cfg, x, ds, a, r, eos), g in zip(prepared, got):
        ctx = H.make_context(cfg, x)
        _poison(ds)
        rc = B.lib.space_verify(ctx._h, C.byref(a), stream)
        assert rc == B.OK, B.space_strerror(rc)
        torch.cuda.synchronize()
        _check(_outputs(ds), g, "space_verify vs noalloc")

    # sizes beyond the fixed scratch and unsupported modes are refused, not run
    a = prepared[0][3]
    bad = B.VerifyArgs.from_buffer_copy(a); bad.batch = B.NOALLOC_MAX_BATCH + 1
    assert B.lib.space_verify_greedy_noalloc(C.byref(bad), None) == B.E_STATIC_LIMIT
    assert "NOALLOC" in B.space_strerror(B.E_STATIC_LIMIT)
    bad = B.VerifyArgs.from_buffer_copy(a); bad.mode = B.MODE_SAMPLE
    assert B.lib.space_verify_greedy_noalloc(C.byref(bad), None) == B.E_INVALID_ARG
    bad = B.VerifyArgs.from_buffer_copy(a); bad.logits = None
    assert B.lib.space_verify_greedy_noalloc(C.byref(bad), None) == B.E_INVALID_ARG
    assert B.lib.space_verify_greedy_noalloc(None, None) == B.E_INVALID_ARG
    torch.cuda.synchronize()
