"""GPU parity for the paged KV cache (the serving setting of Sec. 4.3): attention of all three
implementations and the compaction of accepted rows, through the C ABI, against oracle.paged on
page pools whose unused rows -- spare pages, pages of no sequence, the tail of every sequence's
last page -- are NaN patterns.  Same tolerances as the contiguous cache: attention within
min(2e-2, 1e-2 RMS), log-sum-exp 2e-3, cache bytes and lengths exact."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle.paged import attention_step_paged, commit_step_paged
from oracle.verify import verify_step
from oracle.bf16 import bf16_bits_to_f64
from paper_2402_11809_b200 import workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2402_11809_b200 import build
    build.build()
    from paper_2402_11809_b200 import binding
    return binding


@pytest.fixture(scope="module")
def H():
    import gpu_harness
    return gpu_harness


def _cfg(k, L, d=128, H_q=2, H_kv=2, Bn=3, V=777, seed=0):
    return workloads.resolve("tiny", B=Bn, H_q=H_q, H_kv=H_kv, d=d, L=L, k=k, V=V, logits_dtype="bf16",
                             sigma=2.0, p_accept=(0.6, 0.6), seed=seed)


IMPL = {"tensor": "ATTN_TENSOR", "rows": "ATTN_TENSOR_ROWS", "simt": "ATTN_SIMT"}


@pytest.mark.parametrize("impl", ["tensor", "rows", "simt"])
@pytest.mark.parametrize("k,L,d,H_q,H_kv,Bn", [
    (1, (0, 0), 64, 2, 2, 3),            # the block's rows only
    (3, (119, 119), 128, 2, 1, 2),       # L + n_q = 135: the block straddles two pages
    (4, (103, 103), 64, 8, 8, 2),        # L + n_q = 128: ends exactly on a page boundary
    (5, (129, 700), 128, 4, 4, 3),
    (7, (5, 900), 128, 4, 2, 3),
    (2, (10, 200), 64, 64, 64, 3),       # more (sequence, head) pairs than thread blocks: the flat cut
    (5, (2048, 2048), 128, 32, 32, 1),   # one sequence: pieces per head, helper groups, early requests
    (6, (3000, 3300), 128, 8, 1, 1),     # one sequence, grouped heads
])
def test_paged_attention(B, H, impl, k, L, d, H_q, H_kv, Bn):
    cfg = _cfg(k, L, d=d, H_q=H_q, H_kv=H_kv, Bn=Bn, seed=70 + k)
    x = workloads.to_pages(workloads.make_step_inputs(cfg), seed=k)
    if impl == "simt" and x["s_cap"] > 3000:
        pytest.skip("the SIMT cross-check keeps a sequence's scores in shared memory")
    ctx = H.make_context(cfg, x)
    ds = H.DeviceStep(cfg, x)
    ds.attn(ctx, impl=getattr(B, IMPL[impl]))
    torch.cuda.synchronize()
    ref, ref_lse = attention_step_paged(bf16_bits_to_f64(x["q"]), bf16_bits_to_f64(x["k_cache"]),
                                        bf16_bits_to_f64(x["v_cache"]), x["page_table"], x["kv_len"], k, x["scale"])
    H.check_attention(ds.out.cpu().numpy().astype(np.float64), ref, f"paged {impl} k={k} L={L}")
    np.testing.assert_allclose(ds.lse.cpu().numpy(), ref_lse, rtol=0, atol=2e-3)
    assert int(ds.status.abs().sum()) == 0


def test_paged_commit_and_verify_commit(B, H):
    for k, L in ((5, (100, 140)), (3, (240, 260)), (7, (0, 70))):      # moved rows on both sides of page boundaries
        cfg = _cfg(k, L, Bn=6, seed=90 + k)
        x = workloads.to_pages(workloads.make_step_inputs(cfg), seed=k, poison=False)
        ctx = H.make_context(cfg, x)
        r = verify_step(x["logits"], x["cand"], x["cand_prob"], k, "greedy")
        assert r["n_accept"].max() > 0
        for fused in (False, True):
            ds = H.DeviceStep(cfg, x)
            if fused:
                ds.verify_commit(ctx)
            else:
                ds.verify(ctx)
                ds.commit(ctx)
            torch.cuda.synchronize()
            kp, vp = x["k_cache"].copy(), x["v_cache"].copy()
            new_len = commit_step_paged(kp, vp, x["page_table"], x["kv_len"], r["n_accept"], k)
            assert np.array_equal(ds.kv_len_out.cpu().numpy(), new_len)
            gk, gv = H.bf16_to_bits(ds.k_cache), H.bf16_to_bits(ds.v_cache)
            if fused:
                # the single-launch form also moves the rejected candidates' rows to L+i*+1 .. L+k,
                # rows beyond the new length that nobody reads again
                for b in range(cfg["B"]):
                    for s in range(int(new_len[b]), int(x["kv_len"][b]) + k + 1):
                        pg = int(x["page_table"][b, s // 128])
                        gk[pg, :, s % 128, :] = kp[pg, :, s % 128, :]
                        gv[pg, :, s % 128, :] = vp[pg, :, s % 128, :]
            assert np.array_equal(gk, kp) and np.array_equal(gv, vp)
            assert int(ds.status.abs().sum()) == 0


def test_paged_capacity_bad_pages_and_arguments(B, H):
    k = 3
    cfg = _cfg(k, (200, 230), Bn=2, seed=5)
    x = workloads.to_pages(workloads.make_step_inputs(cfg), seed=1, poison=False)
    ctx = H.make_context(cfg, x)
    # a table entry outside the pool: flagged, nothing read or written through it
    bad = dict(x)
    bad["page_table"] = x["page_table"].copy()
    bad["page_table"][1, 0] = x["k_cache"].shape[0] + 5
    for impl in ("tensor", "rows", "simt"):
        ds = H.DeviceStep(cfg, bad)
        ds.attn(ctx, impl=getattr(B, IMPL[impl]))
        torch.cuda.synchronize()
        st = ds.status.cpu().numpy()
        assert st[1] & B.ST_BAD_PAGE and not st[0] & B.ST_BAD_PAGE, (impl, st)
        assert torch.isfinite(ds.out).all()
    # a length beyond the table's capacity: flagged, output untouched
    over = dict(x)
    over["kv_len"] = x["kv_len"].copy()
    over["kv_len"][0] = x["page_table"].shape[1] * 128 - 3
    for impl in ("tensor", "rows", "simt"):
        ds = H.DeviceStep(cfg, over)
        ds.attn(ctx, impl=getattr(B, IMPL[impl]))
        torch.cuda.synchronize()
        assert ds.status.cpu().numpy()[0] & B.ST_CAPACITY
        assert torch.isnan(ds.out[0]).all() and torch.isfinite(ds.out[1]).all()
    # arguments: a table needs its sizes, and its capacity must fit the context's
    ds = H.DeviceStep(cfg, x)
    a = ctx.attn_args(ds.q, ds.k_cache, ds.v_cache, ds.kv_len, ds.out, k, ds.scale, page_table=ds.page_table)
    for field, val in (("pages_per_seq", 0), ("n_pages", 0), ("pages_per_seq", 10 ** 6)):
        b2 = B.AttnArgs.from_buffer_copy(a)
        setattr(b2, field, val)
        assert B.lib.space_attn_step(ctx._h, C.byref(b2), None) == B.E_INVALID_ARG, field
    torch.cuda.synchronize()


def test_continuous_batching_over_a_shared_pool(B, H):
    """Sequences join and leave between steps; the pager hands their pages out of one pool and the
    step's batch is whatever slots are active.  Every step: the model's block rows go into the pool
    through the table, attention, greedy verification and the paged commit run on the GPU, and all of
    it -- attention output, accepted counts, the whole pool bit for bit, the lengths -- is compared
    with the oracle working on a host mirror of the pool."""
    k, Hh, d, V, P = 3, 2, 64, 500, 128
    n_q = (k + 1) ** 2
    n_pages, pps, slots = 9, 3, 3
    rng = np.random.default_rng(2024)
    bits = lambda shape: workloads.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    pager = B.Pager(n_pages, pps, slots)
    ctx = B.Context(device=0, max_batch=slots, n_q_heads=Hh, n_kv_heads=Hh, head_dim=d, k_max=k, vocab=V, s_cap=pps * P)
    kp = np.full((n_pages, Hh, P, d), 0x7FC0, dtype=np.uint16)     # host mirror, NaN wherever no row lives
    vp = kp.copy()
    length = {}

    def write_rows(slot, s0, n):
        t = pager.batch_table([slot])[0]
        for s in range(s0, s0 + n):
            kp[t[s // P], :, s % P, :] = bits((Hh, d))
            vp[t[s // P], :, s % P, :] = bits((Hh, d))

    def admit(L):
        s = pager.admit()
        pager.reserve(s, L)
        write_rows(s, 0, L)                                        # the prompt's rows
        length[s] = L
        return s

    a, b_ = admit(120), admit(5)
    events = {3: ("admit", 250), 5: ("release", a), 6: ("admit", 100)}
    accepted_total, reused = 0, False
    for step in range(9):
        if step in events:
            kind, arg = events[step]
            if kind == "admit":
                s_new = admit(arg)
                reused |= step == 6 and s_new == a
            else:
                pager.release(arg)
                del length[arg]
        batch = sorted(length)
        Bn = len(batch)
        for s in batch:
            pager.reserve(s, length[s] + n_q)
            write_rows(s, length[s], n_q)                          # the model's K / V rows of this step's block
        table = pager.batch_table(batch)
        L = np.array([length[s] for s in batch], dtype=np.int32)
        q = bits((Bn, n_q, Hh, d))
        logits = (rng.standard_normal((Bn, n_q, V)) * 2).astype(np.float32)
        cand = rng.integers(0, V, size=(Bn, k)).astype(np.int32)
        for i in range(Bn):
            for j in range(k):
                if rng.random() < 0.7:
                    logits[i, j * (k + 1), cand[i, j]] = 30.0      # the model agrees with this candidate
        dev = dict(kp=H.to_dev(kp), vp=H.to_dev(vp), table=H.to_dev(table), L=H.to_dev(L), q=H.to_dev(q),
                   logits=H.to_dev(logits), cand=H.to_dev(cand), cprob=torch.ones((Bn, k), device="cuda"))
        out = torch.full((Bn, n_q, Hh, d), float("nan"), device="cuda")
        status = torch.zeros(Bn, dtype=torch.int32, device="cuda")
        i32 = lambda *sh: torch.full(sh, -7, dtype=torch.int32, device="cuda")
        n_acc, toks, n_out, ncand, L_out = i32(Bn), i32(Bn, k + 1), i32(Bn), i32(Bn, k), i32(Bn)
        nprob = torch.zeros((Bn, k), device="cuda")
        fin = torch.zeros(Bn, dtype=torch.uint8, device="cuda")
        ctx.space_attn_step(ctx.attn_args(dev["q"], dev["kp"], dev["vp"], dev["L"], out, k, 0.125, status=status,
                                          page_table=dev["table"]))
        v = ctx.verify_args(dev["logits"], dev["cand"], dev["cprob"], dev["L"], n_acc, toks, n_out, ncand, nprob, fin, k,
                            status=status)
        c = ctx.commit_args(dev["kp"], dev["vp"], n_acc, dev["L"], k, kv_len_out=L_out, status=status,
                            page_table=dev["table"])
        ctx.space_verify_commit(v, c)
        torch.cuda.synchronize()
        # ---- the same step in the oracle, on the mirror ----
        ref, _ = attention_step_paged(q, kp, vp, table, L, k, 0.125)
        H.check_attention(out.cpu().numpy().astype(np.float64), ref, f"step {step}")
        r = verify_step(logits, cand, np.ones((Bn, k)), k, "greedy")
        assert np.array_equal(n_acc.cpu().numpy(), r["n_accept"])
        new_len = commit_step_paged(kp, vp, table, L, r["n_accept"], k)
        assert np.array_equal(L_out.cpu().numpy(), new_len)
        gk, gv = H.bf16_to_bits(dev["kp"]), H.bf16_to_bits(dev["vp"])
        for i in range(Bn):
            # rows L+i*+1 .. L+k lie beyond the new length; the single-launch form leaves the rejected
            # candidates' rows there (unspecified by the interface, overwritten by the next block)
            for s_ in range(int(new_len[i]), int(L[i]) + k + 1):
                gk[table[i, s_ // P], :, s_ % P, :] = kp[table[i, s_ // P], :, s_ % P, :]
                gv[table[i, s_ // P], :, s_ % P, :] = vp[table[i, s_ // P], :, s_ % P, :]
        assert np.array_equal(gk, kp) and np.array_equal(gv, vp)
        assert int(status.abs().sum()) == 0
        for i, s in enumerate(batch):
            length[s] = int(new_len[i])
        accepted_total += int(r["n_accept"].sum())
    assert accepted_total > 5 and reused          # pages and the slot of the sequence that left were used again
    assert max(length.values()) > P               # at least one sequence grew across a page boundary
    pager.close()


@pytest.mark.parametrize("name,over,heads_per_seq", [
    ("ragged16", {}, 4),                       # the transposed kernel at full size, 16 ragged sequences
    ("sampling64", {"B": 8}, 2),               # grouped heads: the row kernel, eight of the 64 sequences
])
def test_paged_step_at_full_size(B, H, name, over, heads_per_seq):
    """A whole step of a full-size configuration on a paged cache: attention on seeded (sequence, head)
    pairs against the oracle over the rows the table names, the verify + commit call's lengths and the
    whole pools after the commit against oracle.paged."""
    from oracle.attention import attention_head
    from oracle.paged import gather_cache
    cfg = workloads.resolve(name, **over)
    x = workloads.to_pages(workloads.make_step_inputs(cfg), seed=3)
    ctx = H.make_context(cfg, x)
    ds = H.DeviceStep(cfg, x)
    k = cfg["k"]
    sample = cfg["mode"] == "sample"
    ds.attn(ctx)
    ds.verify_commit(ctx, mode=B.MODE_SAMPLE if sample else B.MODE_GREEDY, temperature=cfg["temperature"], seed=cfg["seed"])
    torch.cuda.synchronize()
    assert int(ds.status.abs().sum()) == 0
    out = ds.out.cpu().numpy().astype(np.float64)
    assert np.isfinite(out).all()
    G = cfg["H_q"] // cfg["H_kv"]
    rng = np.random.default_rng(cfg["seed"])
    n_rows = x["kv_len"].astype(np.int64) + x["n_q"]
    for b in range(cfg["B"]):
        heads = sorted(rng.choice(cfg["H_q"], size=heads_per_seq, replace=False).tolist())
        L = int(x["kv_len"][b])
        kb = gather_cache(x["k_cache"], x["page_table"][b:b + 1], n_rows[b:b + 1])[0]      # [H_kv, rows, d]
        vb = gather_cache(x["v_cache"], x["page_table"][b:b + 1], n_rows[b:b + 1])[0]
        refs = np.stack([attention_head(x["q"][b, :, h], kb[h // G], vb[h // G], L, k, x["scale"])[0] for h in heads])
        H.check_attention(out[b][:, heads].transpose(1, 0, 2)[None], refs[None], f"{name} paged b={b}")
    n_acc = ds.n_accept.cpu().numpy()
    kp, vp = x["k_cache"].copy(), x["v_cache"].copy()
    new_len = commit_step_paged(kp, vp, x["page_table"], x["kv_len"], n_acc, k)
    assert np.array_equal(ds.kv_len_out.cpu().numpy(), new_len)
    gk, gv = H.bf16_to_bits(ds.k_cache), H.bf16_to_bits(ds.v_cache)
    for b in range(cfg["B"]):
        # rows beyond the new length (L+i*+1 .. L+k) are unspecified: the single-launch greedy form
        # leaves the rejected candidates' rows there
        for s_ in range(int(new_len[b]), int(x["kv_len"][b]) + k + 1):
            pg = int(x["page_table"][b, s_ // 128])
            gk[pg, :, s_ % 128, :] = kp[pg, :, s_ % 128, :]
            gv[pg, :, s_ % 128, :] = vp[pg, :, s_ % 128, :]
    assert np.array_equal(gk, kp) and np.array_equal(gv, vp)
    if not sample:
        r = verify_step(x["logits"], x["cand"], x["cand_prob"], k, "greedy")
        assert np.array_equal(n_acc, r["n_accept"])
