"""GPU parity of space_lmhead_verify (output projection fused with greedy
verification) against the float64 oracle, through the C ABI.

Integers (accepted count, emitted tokens, next candidates, row arg-maxes) must
match exactly.  The arg-max of a row is decided on fp32 accumulators of bf16
products; a row whose two largest oracle logits are closer than GAP_BAND is a
floating-point tie: a sequence that reads such a row is excluded and printed.
Row maxima: |err| <= 2e-3 (fp32 accumulation over D <= 4096 terms of size
<= ~1: rounding error ~ sqrt(D) * 2^-24 * |terms|, far below).  Probabilities
1e-3 relative (hardware exp2, sums of up to 128k terms in fp32).
"""
import numpy as np
import pytest
import torch

from paper_2402_11809_b200 import workloads
from oracle.lmhead import lmhead_verify_step

pytestmark = pytest.mark.gpu

GAP_BAND = 1e-3
MAX_TOL = 2e-3
PROB_RTOL = 1e-3


@pytest.fixture(scope="module")
def H():
    import gpu_harness
    return gpu_harness


def _run(H, cfg, x, eos_id=-1, ctx=None, pad=0):
    from paper_2402_11809_b200 import binding as B
    Bn, k, V, D = cfg["B"], cfg["k"], cfg["V"], cfg["D"]
    n_q = x["n_q"]
    own = ctx is None
    if own:
        ctx = B.Context(device=0, max_batch=Bn, n_q_heads=8, n_kv_heads=8, head_dim=64, k_max=k, vocab=V,
                        s_cap=256)
    hidden = H.to_dev(x["hidden"])
    weight = H.to_dev(x["weight"])
    if pad:                                                  # row strides larger than D
        wp = torch.full((V, D + pad), float("nan"), dtype=torch.bfloat16, device="cuda")
        wp[:, :D] = weight
        weight = wp[:, :D]
        hp = torch.full((Bn, n_q, D + pad), float("nan"), dtype=torch.bfloat16, device="cuda")
        hp[:, :, :D] = hidden
        hidden = hp[:, :, :D]
    dev = "cuda"
    o = dict(
        n_accept=torch.full((Bn,), -7, dtype=torch.int32, device=dev),
        out_tokens=torch.full((Bn, k + 1), -7, dtype=torch.int32, device=dev),
        n_out=torch.full((Bn,), -7, dtype=torch.int32, device=dev),
        next_cand=torch.full((Bn, k), -7, dtype=torch.int32, device=dev),
        next_cand_prob=torch.full((Bn, k), float("nan"), device=dev),
        finished=torch.full((Bn,), 9, dtype=torch.uint8, device=dev),
        status=torch.zeros(Bn, dtype=torch.int32, device=dev),
        row_max=torch.full((Bn, n_q), float("nan"), device=dev),
        row_argmax=torch.full((Bn, n_q), -7, dtype=torch.int32, device=dev),
    )
    a = ctx.lmhead_args(hidden, weight, H.to_dev(x["cand"]), o["n_accept"], o["out_tokens"], o["n_out"],
                        o["next_cand"], o["next_cand_prob"], o["finished"], k, eos_id=eos_id,
                        status=o["status"], row_max=o["row_max"], row_argmax=o["row_argmax"])
    n0 = ctx.launch_count
    ctx.space_lmhead_verify(a)
    torch.cuda.synchronize()
    assert ctx.launch_count == n0 + 1
    got = {key: v.cpu().numpy() for key, v in o.items()}
    if own:
        ctx.close()
    return got


def _compare(cfg, x, got, eos_id=-1, what=""):
    k = cfg["k"]
    r = lmhead_verify_step(x["hidden"], x["weight"], x["cand"], x["cand_prob"], k, eos_id=eos_id)
    assert not got["status"].any(), (what, got["status"])
    ref_max = r["logits"].max(axis=-1)
    assert np.abs(got["row_max"] - ref_max).max() <= MAX_TOL, what
    ref_arg = np.argmax(r["logits"], axis=-1)
    tie = r["row_gap"] <= GAP_BAND                           # [B, n_q]
    assert np.array_equal(got["row_argmax"][~tie], ref_arg[~tie]), what
    excluded = 0
    for b in range(cfg["B"]):
        i = int(r["n_accept"][b])
        used = [t * (k + 1) for t in range(k + 1)] + [i * (k + 1) + o for o in range(1, k + 1)]
        if tie[b, used].any():
            excluded += 1
            print(f"{what}: sequence {b} excluded (top-two gap {r['row_gap'][b, used].min():.2e} inside the band)")
            continue
        assert got["n_accept"][b] == r["n_accept"][b], (what, b)
        assert np.array_equal(got["out_tokens"][b], r["out_tokens"][b]), (what, b)
        assert got["n_out"][b] == r["n_out"][b], (what, b)
        assert np.array_equal(got["next_cand"][b], r["next_cand"][b]), (what, b)
        assert got["finished"][b] == r["finished"][b], (what, b)
        assert np.allclose(got["next_cand_prob"][b], r["next_cand_prob"][b], rtol=PROB_RTOL, atol=0), (what, b)
    assert excluded <= cfg["B"] // 4, what
    return r


@pytest.mark.parametrize("V,D,k,Bn", [
    (1000, 256, 4, 1),        # ranges shorter than 16 tokens
    (4736, 512, 5, 1),        # exactly 32 tokens per thread block
    (5000, 320, 3, 2),        # two sequences, ragged ranges
    (40000, 192, 2, 3),       # two boxes per range: a full one and a tail
    (130000, 128, 4, 2),      # four boxes per range, alternating accumulators
    (257, 72, 1, 4),          # tiny vocabulary (fewer thread blocks than SMs), D not a multiple of 64
    (33000, 128, 7, 4),       # 256 block rows: two accumulators of 128 rows, one buffer
    (100000, 64, 5, 4),       # 144 block rows and three boxes per range
])
def test_lmhead_small_shapes(H, V, D, k, Bn):
    cfg = workloads.resolve_lmhead("lmhead_tiny", V=V, D=D, k=k, B=Bn, p_accept=(0.5, 0.9))
    for s in range(2):
        x = workloads.make_lmhead_inputs(cfg, set_index=s)
        got = _run(H, cfg, x)
        _compare(cfg, x, got, what=f"V{V} D{D} k{k} B{Bn} set{s}")


def test_lmhead_exact_ties_take_the_lowest_token(H):
    # duplicated embedding rows give bit-identical logits: the lower token must win
    cfg = workloads.resolve_lmhead("lmhead_tiny", V=3000, D=128, k=3, B=2)
    x = workloads.make_lmhead_inputs(cfg)
    k = cfg["k"]
    r0 = lmhead_verify_step(x["hidden"], x["weight"], x["cand"], x["cand_prob"], k)
    top = np.argmax(r0["logits"], axis=-1)
    # copy the winner of block row 1 of sequence 0 to a later and an earlier token far away
    w = int(top[0, 1])
    lo, hi = (w + 1500) % 3000, (w + 700) % 3000
    x["weight"][lo] = x["weight"][w]
    x["weight"][hi] = x["weight"][w]
    got = _run(H, cfg, x)
    r = lmhead_verify_step(x["hidden"], x["weight"], x["cand"], x["cand_prob"], k)
    assert r["row_gap"][0, 1] == 0.0
    expect = min(w, lo, hi)
    assert int(np.argmax(r["logits"][0, 1])) == expect
    assert got["row_argmax"][0, 1] == expect


def test_lmhead_eos_padded_strides_and_bad_candidate(H):
    from paper_2402_11809_b200 import binding as B
    cfg = workloads.resolve_lmhead("lmhead_tiny", V=6000, D=256, k=4, B=2, p_accept=(1.0, 1.0))
    x = workloads.make_lmhead_inputs(cfg)
    eos = int(x["cand"][0, 1])                               # second accepted token of sequence 0
    got = _run(H, cfg, x, eos_id=eos, pad=24)
    r = _compare(cfg, x, got, eos_id=eos, what="eos")
    assert r["finished"][0] == 1 and r["n_out"][0] == 1
    x["cand"][1, 2] = cfg["V"] + 5                           # out of range: rejected and flagged
    got = _run(H, cfg, x)
    assert got["status"][1] & B.ST_BAD_CANDIDATE and not got["status"][0]
    r = lmhead_verify_step(x["hidden"], x["weight"], x["cand"], x["cand_prob"], cfg["k"])
    assert got["n_accept"][1] == r["n_accept"][1] == 2
    assert np.array_equal(got["out_tokens"], r["out_tokens"])


def test_lmhead_repeated_calls_and_argument_checks(H):
    from paper_2402_11809_b200 import binding as B
    cfg = workloads.resolve_lmhead("lmhead_tiny", V=9000, D=256, k=5, B=2)
    ctx = B.Context(device=0, max_batch=2, n_q_heads=8, n_kv_heads=8, head_dim=64, k_max=5, vocab=9000, s_cap=256)
    first = None
    for s in (0, 1, 0):                                      # the arrival counter resets itself
        x = workloads.make_lmhead_inputs(cfg, set_index=s)
        got = _run(H, cfg, x, ctx=ctx)
        _compare(cfg, x, got, what=f"repeat set{s}")
        if s == 0:
            if first is None:
                first = got
            else:
                for key in first:
                    assert np.array_equal(first[key], got[key], equal_nan=True), key   # bit-identical re-run
    x = workloads.make_lmhead_inputs(cfg)
    hidden, weight = H.to_dev(x["hidden"]), H.to_dev(x["weight"])
    z = torch.zeros(64, dtype=torch.int32, device="cuda")
    f = torch.zeros(64, device="cuda")
    u = torch.zeros(8, dtype=torch.uint8, device="cuda")
    good = lambda **kw: ctx.lmhead_args(hidden, weight, z, z, z, z, z, f, u, 5, **kw)
    a = good(); a.batch = 3
    assert B.lib.space_lmhead_verify(ctx._h, a, None) == B.E_WORKSPACE
    a = good(); a.hidden = None
    assert B.lib.space_lmhead_verify(ctx._h, a, None) == B.E_INVALID_ARG
    a = good(); a.weight_row_stride = 260
    assert B.lib.space_lmhead_verify(ctx._h, a, None) == B.E_ALIGNMENT
    a = good(); a.weight = a.weight + 2
    assert B.lib.space_lmhead_verify(ctx._h, a, None) == B.E_ALIGNMENT
    ctx.close()
    big = B.Context(device=0, max_batch=8, n_q_heads=8, n_kv_heads=8, head_dim=64, k_max=7, vocab=9000, s_cap=256)
    a = big.lmhead_args(hidden, weight, z, z, z, z, z, f, u, 7); a.batch = 5   # 5 * 64 rows > 256
    assert B.lib.space_lmhead_verify(big._h, a, None) == B.E_UNSUPPORTED
    big.close()


@pytest.mark.parametrize("name", ["lmhead_llama7b", "lmhead_batch4", "lmhead_vocab128k"])
def test_lmhead_full_size(H, name):
    cfg = workloads.resolve_lmhead(name)
    x = workloads.make_lmhead_inputs(cfg)
    got = _run(H, cfg, x)
    _compare(cfg, x, got, what=name)
