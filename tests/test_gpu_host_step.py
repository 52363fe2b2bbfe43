"""space_step_host: the whole step from host buffers (copies in, attention,
verification, KV commit, copies out) against the fp64 oracle, with the whole
cache uploaded and with the cache kept on the device between calls."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle.attention import attention_step
from oracle.verify import verify_step
from oracle.commit import commit_step
from paper_2402_11809_b200 import workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2402_11809_b200 import build
    build.build()
    from paper_2402_11809_b200 import binding
    return binding


def _pinned(arr):
    return torch.from_numpy(arr.view(np.int16) if arr.dtype == np.uint16 else arr).clone().pin_memory()


def _run(B, ctx, cfg, x, pin, resident):
    k = cfg["k"]
    n_q = (k + 1) ** 2
    outs = dict(out=torch.full((cfg["B"], n_q, cfg["H_q"], cfg["d"]), float("nan")).pin_memory(),
                n_accept=torch.full((cfg["B"],), -7, dtype=torch.int32).pin_memory(),
                out_tokens=torch.zeros((cfg["B"], k + 1), dtype=torch.int32).pin_memory(),
                n_out=torch.zeros(cfg["B"], dtype=torch.int32).pin_memory(),
                next_cand=torch.zeros((cfg["B"], k), dtype=torch.int32).pin_memory(),
                next_cand_prob=torch.zeros((cfg["B"], k), dtype=torch.float32).pin_memory(),
                finished=torch.zeros(cfg["B"], dtype=torch.uint8).pin_memory(),
                status=torch.full((cfg["B"],), -1, dtype=torch.int32).pin_memory())
    h2d, d2h = C.c_int64(0), C.c_int64(0)
    hs = B.HostStepArgs(batch=cfg["B"], k=k, vocab=cfg["V"],
                        logits_dtype=B.DTYPE_F32 if cfg["logits_dtype"] == "f32" else B.DTYPE_BF16,
                        mode=B.MODE_GREEDY, resample=B.RESAMPLE_RESIDUAL_POINTMASS, eos_id=-1,
                        mask_variant=B.MASK_SAME_GROUP, scale=x["scale"], temperature=1.0, seed=0,
                        **{n: C.c_void_p(t.data_ptr()) for n, t in pin.items()},
                        **{n: C.c_void_p(t.data_ptr()) for n, t in outs.items()},
                        h2d_bytes=C.cast(C.pointer(h2d), C.c_void_p), d2h_bytes=C.cast(C.pointer(d2h), C.c_void_p),
                        cache_resident=1 if resident else 0)
    ctx.space_step_host(hs)
    torch.cuda.synchronize()
    return outs, int(h2d.value), int(d2h.value)


@pytest.mark.parametrize("k,L,H_q,H_kv", [(3, (40, 300), 4, 2), (5, (130, 131), 2, 2)])
def test_host_step_matches_oracle_full_and_resident(B, k, L, H_q, H_kv):
    import gpu_harness as H
    cfg = workloads.resolve("tiny", B=3, H_q=H_q, H_kv=H_kv, d=64, L=L, k=k, V=901, logits_dtype="bf16",
                            sigma=2.0, p_accept=(0.6, 0.6), seed=11 + k)
    x = workloads.make_step_inputs(cfg)
    n_q = (k + 1) ** 2
    ctx = B.Context(device=0, max_batch=cfg["B"], n_q_heads=H_q, n_kv_heads=H_kv, head_dim=cfg["d"], k_max=k,
                    vocab=cfg["V"], host_staging=1, s_cap=x["s_cap"])
    # oracle
    ref, _ = attention_step(x["q"], x["k_cache"], x["v_cache"], x["kv_len"], k, x["scale"])
    r = verify_step(x["logits"], x["cand"], x["cand_prob"], k, "greedy")
    Kc, Vc = x["k_cache"].copy(), x["v_cache"].copy()
    new_len, _, _ = commit_step(Kc, Vc, x["kv_len"], r["n_accept"], k)

    def fresh_pins():
        return {n: _pinned(x[n]) for n in ("q", "k_cache", "v_cache", "logits", "cand", "cand_prob", "kv_len")}

    def check(outs, pin):
        assert int(outs["status"].abs().sum()) == 0
        H.check_attention(outs["out"].numpy().astype(np.float64), ref, "host step")
        assert np.array_equal(outs["n_accept"].numpy(), r["n_accept"])
        assert np.array_equal(outs["out_tokens"].numpy(), r["out_tokens"])
        assert np.array_equal(outs["n_out"].numpy(), r["n_out"])
        assert np.array_equal(outs["next_cand"].numpy(), r["next_cand"])
        assert np.array_equal(pin["kv_len"].numpy(), new_len)
        # the rows the commit moved come back to the host cache: rows L .. new length - 1 of every
        # head (rows from the new length up to L+k come back too, but lie beyond the verified prefix
        # and are unspecified)
        got_k = pin["k_cache"].numpy().view(np.uint16)
        got_v = pin["v_cache"].numpy().view(np.uint16)
        for b in range(cfg["B"]):
            Lb, nb = int(x["kv_len"][b]), int(new_len[b])
            assert np.array_equal(got_k[b, :, Lb:nb], Kc[b, :, Lb:nb])
            assert np.array_equal(got_v[b, :, Lb:nb], Vc[b, :, Lb:nb])
            assert np.array_equal(got_k[b, :, Lb + k + 1:], Kc[b, :, Lb + k + 1:])

    pin = fresh_pins()
    outs, h2d_full, _ = _run(B, ctx, cfg, x, pin, resident=False)
    check(outs, pin)
    kv_bytes = sum(2 * (int(Lb) + n_q) * cfg["d"] * 2 * H_kv for Lb in x["kv_len"])
    assert h2d_full >= kv_bytes

    # second call, cache kept on the device: the host passes the same step again (fresh block rows,
    # the old length); only the block's rows travel and the results are the same
    pin2 = fresh_pins()
    outs2, h2d_res, _ = _run(B, ctx, cfg, x, pin2, resident=True)
    check(outs2, pin2)
    assert torch.equal(outs2["out"], outs["out"])
    block_bytes = cfg["B"] * 2 * n_q * cfg["d"] * 2 * H_kv
    assert h2d_full - h2d_res == kv_bytes - block_bytes
