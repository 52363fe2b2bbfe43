"""Pins of the projection oracle (oracle/lmhead.py): the output projection that ends
the model call of Algorithm 1, followed by greedy verification.

The projection is pinned by things other than itself: entry-by-entry sums in plain
Python, a selector matrix whose product is known in closed form (catches a
transposed or mis-indexed operand), linearity, and the composition rule that a
square identity embedding turns the hidden states themselves into the logits."""
import numpy as np
import pytest

from oracle.lmhead import lm_head_logits, lmhead_verify_step, top_two_gap
from oracle.verify import verify_step
from oracle.bf16 import bf16_bits_to_f64
from paper_2402_11809_b200 import workloads


def test_projection_entry_by_entry():
    rng = np.random.default_rng(0)
    B, n_q, D, V = 2, 4, 5, 7
    h = rng.standard_normal((B, n_q, D))
    W = rng.standard_normal((V, D))
    z = lm_head_logits(h, W)
    assert z.shape == (B, n_q, V)
    for b in range(B):
        for r in range(n_q):
            for x in range(V):
                acc = 0.0
                for d in range(D):
                    acc += float(h[b, r, d]) * float(W[x, d])
                assert abs(z[b, r, x] - acc) <= 1e-12 * max(1.0, abs(acc))


def test_projection_selector_closed_form():
    # W_x = s_x * e_{perm[x]}  =>  logits[b, r, x] = s_x * h[b, r, perm[x]]
    rng = np.random.default_rng(1)
    B, n_q, D, V = 1, 9, 6, 11
    h = rng.standard_normal((B, n_q, D))
    perm = rng.integers(0, D, size=V)
    s = rng.uniform(0.5, 2.0, size=V)
    W = np.zeros((V, D))
    W[np.arange(V), perm] = s
    z = lm_head_logits(h, W)
    assert np.array_equal(z, h[:, :, perm] * s[None, None, :])


def test_projection_reads_bf16_bits_exactly_and_is_linear():
    cfg = workloads.resolve_lmhead("lmhead_tiny", V=37, D=24)
    x = workloads.make_lmhead_inputs(cfg)
    z = lm_head_logits(x["hidden"], x["weight"])
    hf, Wf = bf16_bits_to_f64(x["hidden"]), bf16_bits_to_f64(x["weight"])
    assert np.allclose(z, lm_head_logits(hf, Wf), rtol=0, atol=0)
    assert np.allclose(lm_head_logits(2.0 * hf, Wf), 2.0 * z, rtol=1e-15)
    assert np.allclose(lm_head_logits(hf, Wf[::-1]), z[:, :, ::-1], rtol=0, atol=0)


def test_identity_embedding_makes_hidden_states_the_logits():
    # D = V and W = I: the step from hidden states is the step from those logits
    rng = np.random.default_rng(2)
    k, V = 3, 50
    n_q = (k + 1) ** 2
    h = rng.standard_normal((2, n_q, V))
    cand = rng.integers(0, V, size=(2, k))
    cand[0, 0] = int(np.argmax(h[0, 0]))                       # first candidate of sequence 0 is right
    cand[0, 1] = int(np.argmax(h[0, k + 1]))                   # and the second
    r = lmhead_verify_step(h, np.eye(V), cand, np.ones((2, k)), k)
    ref = verify_step(h, cand, np.ones((2, k)), k, "greedy")
    for key in ("n_accept", "out_tokens", "n_out", "next_cand", "next_cand_prob", "finished"):
        assert np.array_equal(r[key], ref[key]), key
    assert r["n_accept"][0] >= 2


def test_planted_candidates_are_accepted_as_a_prefix():
    cfg = workloads.resolve_lmhead("lmhead_tiny")
    k = cfg["k"]
    for s in range(4):
        x = workloads.make_lmhead_inputs(cfg, set_index=s)
        r = lmhead_verify_step(x["hidden"], x["weight"], x["cand"], x["cand_prob"], k)
        for b in range(cfg["B"]):
            run = 0
            while run < k and x["planted"][b, run]:
                run += 1
            assert r["n_accept"][b] >= run                     # every planted prefix is accepted
            top = np.argmax(r["logits"][b], axis=-1)
            i = int(r["n_accept"][b])
            assert list(r["out_tokens"][b, :i]) == list(x["cand"][b, :i])
            assert r["out_tokens"][b, i] == top[i * (k + 1)]
            assert list(r["next_cand"][b]) == [top[i * (k + 1) + o] for o in range(1, k + 1)]


def test_top_two_gap():
    z = np.array([[[1.0, 5.0, 3.0, 5.0], [0.0, -1.0, 4.0, 1.5]]])
    assert np.array_equal(top_two_gap(z), np.array([[0.0, 2.5]]))


def test_identity_embedding_reduces_to_verify_step_in_sampling_mode_too():
    # W = identity: the logits are the hidden rows themselves, so the step from hidden states must
    # be verify_step on those rows -- same acceptance draws, same extra token, same new candidates --
    # for both resampling readings, with candidates that get accepted, rejected and are out of range
    rng = np.random.default_rng(11)
    k, V, Bn = 3, 24, 40
    n_q = (k + 1) ** 2
    h = rng.standard_normal((Bn, n_q, V)) * 2.0
    cand = rng.integers(0, V, size=(Bn, k))
    cand[:10, 0] = np.argmax(h[:10, 0], axis=-1)               # likely accepted
    cand[10, 1] = V + 3                                        # out of range
    P_c = np.ones((Bn, k))
    P_c[11, :] = np.inf                                        # Algorithm 1's initial state
    for resample in ("residual_pointmass", "paper_literal"):
        if resample == "paper_literal":
            P_c = np.where(np.isinf(P_c), P_c, rng.uniform(0.2, 1.0, size=P_c.shape))
        kw = dict(temperature=0.7, seed=99, seq_id=np.arange(Bn) + 5, kv_len=rng.integers(0, 50, size=Bn),
                  resample=resample)
        r = lmhead_verify_step(h, np.eye(V), cand, P_c, k, mode="sample", **kw)
        ref = verify_step(h, cand, P_c, k, "sample", **kw)
        for key in ("n_accept", "out_tokens", "n_out", "next_cand", "next_cand_prob", "finished",
                    "accept_margin", "bonus_gap", "draft_gap"):
            assert np.array_equal(r[key], ref[key]), (resample, key)
        assert r["n_accept"].max() > 0 and r["n_accept"][11] == 0
