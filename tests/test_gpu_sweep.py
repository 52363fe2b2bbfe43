"""Seeded sweep over shapes for the two tensor-core attention kernels: batch,
head counts, GQA group, head_dim, k and ragged lengths drawn at random (fixed
seeds), each case against the fp64 oracle.  The shapes are chosen to cross the
boundaries of the work partition: one tile per sequence, more (sequence, head)
pairs than thread blocks, a single long sequence cut over every block, query
blocks of one or several 64/128-row pieces.  Every case runs on the contiguous cache and on
the same cache cut into pages."""
import numpy as np
import pytest
import torch

from oracle.attention import attention_step
from paper_2402_11809_b200 import workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2402_11809_b200 import build
    build.build()
    from paper_2402_11809_b200 import binding
    return binding


def _draw(seed):
    r = np.random.default_rng(1000 + seed)
    d = int(r.choice([64, 128]))
    G = int(r.choice([1, 1, 2, 4, 8]))
    H_kv = int(r.choice([1, 2, 3, 8, 16]))
    k = int(r.integers(1, 8))
    kind = seed % 4
    if kind == 0:                       # many short sequences
        Bn, L = int(r.integers(8, 25)), (0, int(r.integers(1, 200)))
    elif kind == 1:                     # one long sequence
        Bn, L = 1, (int(r.integers(2000, 6000)),) * 2
        H_kv = int(r.choice([1, 2]))
    elif kind == 2:                     # very ragged
        Bn, L = int(r.integers(2, 7)), (0, int(r.integers(500, 2500)))
    else:                               # lengths around tile boundaries
        base = 128 * int(r.integers(1, 6)) - (k + 1) ** 2
        Bn, L = int(r.integers(2, 5)), (max(0, base - 2), base + 2)
    return dict(B=Bn, H_q=H_kv * G, H_kv=H_kv, d=d, L=L, k=k, seed=seed)


@pytest.mark.parametrize("seed", list(range(24)))
def test_attention_shape_sweep(B, seed):
    import gpu_harness as H
    c = _draw(seed)
    cfg = workloads.resolve("tiny", B=c["B"], H_q=c["H_q"], H_kv=c["H_kv"], d=c["d"], L=c["L"], k=c["k"], V=64,
                            logits_dtype="f32", sigma=2.0, p_accept=(0.5, 0.5), seed=c["seed"])
    x = workloads.make_step_inputs(cfg, poison_tail=True)
    ref, ref_lse = attention_step(x["q"], x["k_cache"], x["v_cache"], x["kv_len"], c["k"], x["scale"])
    # the same caches once more as page pools behind a shuffled table, NaN wherever no key lives: the
    # result must not change (the oracle's paged form is pinned to the contiguous one on the CPU)
    xp = workloads.to_pages(x, seed=seed)
    for xi, what in ((x, "contiguous"), (xp, "paged")):
        ctx = H.make_context(cfg, xi)
        for impl in (B.ATTN_TENSOR, B.ATTN_TENSOR_ROWS):
            for rep in range(2 if what == "paged" else 1):    # (a second launch meets other timings)
                ds = H.DeviceStep(cfg, xi)
                ds.attn(ctx, impl=impl)
                torch.cuda.synchronize()
                assert int(ds.status.abs().sum()) == 0, (c, impl, what)
                H.check_attention(ds.out.cpu().numpy().astype(np.float64), ref, f"sweep {c} impl {impl} {what}")
                np.testing.assert_allclose(ds.lse.cpu().numpy(), ref_lse, rtol=0, atol=2e-3)
