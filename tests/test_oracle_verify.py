"""Pins for oracle.verify: greedy invariants (Sec. 3.2 / Table 1 setting),
acceptance statistics and output marginals of rejection sampling over 10^6
Philox-driven trials on a 16-token vocabulary."""
import numpy as np
import pytest

from oracle import layout
from oracle.verify import verify_step, softmax_rows, accept_uniform, gumbel_noise

INF = float("inf")


def _logits(rng, B, k, V, sigma=2.0):
    return rng.standard_normal((B, layout.n_block_rows(k), V)) * sigma


# ------------------------------------------------------------------ greedy
@pytest.mark.parametrize("k", [1, 2, 4, 5])
def test_greedy_accepts_longest_prefix_of_argmax_chain(k):
    rng = np.random.default_rng(k)
    B, V = 400, 12
    z = _logits(rng, B, k, V)
    chain = np.argmax(z[:, layout.target_rows(k), :], axis=-1)         # [B, k+1]
    cand = chain[:, :k].copy()
    # break the chain at a random place for most sequences
    cut = rng.integers(0, k + 2, size=B)
    for b in range(B):
        if cut[b] < k:
            cand[b, cut[b]] = (cand[b, cut[b]] + 1 + rng.integers(0, V - 1)) % V
    r = verify_step(z, cand, np.ones((B, k)), k, "greedy")
    for b in range(B):
        n = 0
        while n < k and cand[b, n] == chain[b, n]:
            n += 1
        assert r["n_accept"][b] == n == min(cut[b], k)
        assert r["n_out"][b] == n + 1 and 1 <= r["n_out"][b] <= k + 1       # Sec. 3.2
        assert list(r["out_tokens"][b, : n + 1]) == list(chain[b, : n + 1])
        assert all(r["out_tokens"][b, n + 1:] == -1)
        rows = layout.mask_group_rows(k, n)
        assert list(r["next_cand"][b]) == [int(np.argmax(z[b, rr])) for rr in rows]
        p = softmax_rows(z[b, rows[0]])
        assert np.isclose(r["next_cand_prob"][b, 0], p.max(), rtol=1e-12)


def test_greedy_ties_take_lowest_index_and_first_step_emits_one_token():
    k, V = 3, 8
    z = np.zeros((1, layout.n_block_rows(k), V))
    z[0, :, [2, 5]] = 1.0                                   # exact tie everywhere
    r = verify_step(z, np.array([[5, 5, 5]]), np.full((1, k), INF), k, "greedy")
    assert r["n_accept"][0] == 0 and r["out_tokens"][0, 0] == 2 and r["n_out"][0] == 1
    r = verify_step(z, np.array([[2, 2, 5]]), np.ones((1, k)), k, "greedy")
    assert r["n_accept"][0] == 2 and list(r["out_tokens"][0]) == [2, 2, 2, -1]
    assert list(r["next_cand"][0]) == [2, 2, 2]


def test_out_of_range_candidate_is_rejected():
    k, V = 2, 6
    z = _logits(np.random.default_rng(0), 1, k, V)
    for mode in ("greedy", "sample"):
        r = verify_step(z, np.array([[V + 3, 1]]), np.ones((1, k)), k, mode, seed=1)
        assert r["n_accept"][0] == 0
        r = verify_step(z, np.array([[-1, 1]]), np.ones((1, k)), k, mode, seed=1)
        assert r["n_accept"][0] == 0


def test_eos_truncates():
    k, V = 3, 10
    z = np.full((1, layout.n_block_rows(k), V), -5.0)
    for t, tok in zip(layout.target_rows(k), (4, 7, 9, 1)):
        z[0, t, tok] = 5.0
    r = verify_step(z, np.array([[4, 7, 9]]), np.ones((1, k)), k, "greedy", eos_id=9)
    assert r["n_accept"][0] == 3 and r["n_out"][0] == 2 and r["finished"][0] == 1
    assert list(r["out_tokens"][0]) == [4, 7, -1, -1]
    r = verify_step(z, np.array([[4, 7, 9]]), np.ones((1, k)), k, "greedy", eos_id=3)
    assert r["n_out"][0] == 4 and r["finished"][0] == 0


def test_planted_generator_statistics():
    # With candidates planted as the row maximum with probability p, the expected
    # accepted count is sum_{i=1..k} p^i (tiny: 1.773, llama7b: 2.689).
    from paper_2402_11809_b200 import workloads
    cfg = workloads.resolve("tiny", B=3000, V=64, L=(4, 4), H_q=1, H_kv=1, d=8)
    x = workloads.make_step_inputs(cfg)
    r = verify_step(x["logits"], x["cand"], x["cand_prob"], cfg["k"], "greedy")
    want = sum(0.7 ** i for i in range(1, 5))
    assert abs(r["n_accept"].mean() - want) < 0.08
    # accepted count equals the length of the leading run of planted candidates,
    # except when an unplanted random candidate happens to be the arg-max (1/V)
    run = np.cumprod(x["planted"], axis=1).sum(axis=1)
    assert np.mean(r["n_accept"] == run) > 0.95 and np.all(r["n_accept"] >= run)


# ---------------------------------------------------------------- sampling
N = 1_000_000
V16 = 16


def _chi2(counts, probs):
    n = counts.sum()
    keep = probs > 0
    assert counts[~keep].sum() == 0
    return float((((counts[keep] - n * probs[keep]) ** 2) / (n * probs[keep])).sum()), int(keep.sum()) - 1


def _fixed_logits(k, seed):
    rng = np.random.default_rng(seed)
    z = rng.standard_normal((1, layout.n_block_rows(k), V16)) * 1.5
    return np.broadcast_to(z, (N, layout.n_block_rows(k), V16))


def test_first_step_rejects_everything():
    # Algorithm 1 starts with P_c = +inf: nothing can be accepted, one token comes out
    k = 2
    z = _fixed_logits(k, 0)[:1000]
    r = verify_step(z, np.zeros((1000, k), dtype=int), np.full((1000, k), INF), k, "sample",
                    temperature=0.9, seed=5, seq_id=np.arange(1000))
    assert np.all(r["n_accept"] == 0) and np.all(r["n_out"] == 1)


def test_lossless_variant_reproduces_target_marginals():
    k, T, seed = 2, 0.8, 20240211
    z = _fixed_logits(k, 1)
    q = softmax_rows(z[0, layout.target_rows(k)], T)                   # [k+1, V]
    c = np.array([int(np.argsort(q[0])[-2]), int(np.argmax(q[1]))])     # fixed drafts
    cand = np.broadcast_to(c, (N, k))
    r = verify_step(z, cand, np.ones((N, k)), k, "sample", temperature=T, seed=seed,
                    seq_id=np.arange(N), kv_len=np.full(N, 11))
    # acceptance rate of a point-mass draft is q(c)
    acc1 = (r["n_accept"] >= 1).mean()
    assert abs(acc1 - q[0, c[0]]) < 5 * np.sqrt(q[0, c[0]] * (1 - q[0, c[0]]) / N)
    # first emitted token ~ q_0
    chi, dof = _chi2(np.bincount(r["out_tokens"][:, 0], minlength=V16), q[0])
    assert chi < 55.0, chi                                              # 15 dof, p ~ 1e-6
    # second emitted token, given the first candidate was accepted, ~ q_1
    sel = r["n_accept"] >= 1
    chi, dof = _chi2(np.bincount(r["out_tokens"][sel, 1], minlength=V16), q[1])
    assert chi < 55.0, chi
    sel2 = r["n_accept"] >= 2
    assert abs(sel2.sum() / sel.sum() - q[1, c[1]]) < 6 * np.sqrt(0.25 / sel.sum())
    chi, dof = _chi2(np.bincount(r["out_tokens"][sel2, 2], minlength=V16), q[2])
    assert chi < 55.0, chi
    # after a rejection the rejected token is never re-drawn
    rej0 = r["n_accept"] == 0
    assert not np.any(r["out_tokens"][rej0, 0] == c[0])
    # new candidates: arg-max of the chosen group's mask rows, probability one
    for g in range(k + 1):
        rows = layout.mask_group_rows(k, g)
        want = [int(np.argmax(z[0, rr])) for rr in rows]
        assert np.all(r["next_cand"][r["n_accept"] == g] == want)
    assert np.all(r["next_cand_prob"] == 1.0)


def test_literal_variant_matches_its_closed_form():
    # Algorithm 1 as printed: draft c ~ p, accept w.p. min(1, q/p), extra token a ~ q
    # also after a rejection.  First-token law: min(p,q)(x) + (1 - sum min(p,q)) q(x).
    k, T, seed = 1, 1.0, 99
    z = _fixed_logits(k, 2)
    q = softmax_rows(z[0, layout.target_rows(k)], T)
    rng = np.random.default_rng(7)
    p = softmax_rows(rng.standard_normal(V16) * 1.5)
    c = rng.choice(V16, size=N, p=p)
    r = verify_step(z, c[:, None], p[c][:, None], k, "sample", temperature=T, seed=seed,
                    seq_id=np.arange(N), resample="paper_literal")
    mn = np.minimum(p, q[0])
    assert abs((r["n_accept"] == 1).mean() - mn.sum()) < 5 * np.sqrt(0.25 / N)
    law = mn + (1.0 - mn.sum()) * q[0]
    chi, _ = _chi2(np.bincount(r["out_tokens"][:, 0], minlength=V16), law)
    assert chi < 55.0, chi
    # ... which is measurably not the target law (the lossless variant above is)
    chi_q, _ = _chi2(np.bincount(r["out_tokens"][:, 0], minlength=V16), q[0])
    assert chi_q > 500.0
    # sampled new candidates follow their mask row's distribution and carry its probability
    for g in (0, 1):
        sel = r["n_accept"] == g
        row = layout.mask_group_rows(k, g)[0]
        pm = softmax_rows(z[0, row], T)
        chi, _ = _chi2(np.bincount(r["next_cand"][sel, 0], minlength=V16), pm)
        assert chi < 55.0, chi
        assert np.allclose(r["next_cand_prob"][sel, 0], pm[r["next_cand"][sel, 0]])


def test_draws_are_keyed_by_seed_sequence_and_position():
    a = accept_uniform(1, np.array([0, 1, 0]), np.array([5, 5, 6]))
    assert len(set(a.tolist())) == 3
    assert accept_uniform(2, np.array([0]), np.array([5]))[0] != a[0]
    g1 = gumbel_noise(1, 1, np.array([3]), np.array([9]), 10)
    g2 = gumbel_noise(1, 2, np.array([3]), np.array([9]), 10)
    assert g1.shape == (1, 10) and not np.array_equal(g1, g2)
    # re-running a step from the same inputs reproduces it exactly (stateless RNG)
    k = 2
    z = _fixed_logits(k, 3)[:500]
    kw = dict(temperature=0.7, seed=11, seq_id=np.arange(500), kv_len=np.arange(500))
    r1 = verify_step(z, np.ones((500, k), dtype=int), np.ones((500, k)), k, "sample", **kw)
    r2 = verify_step(z, np.ones((500, k), dtype=int), np.ones((500, k)), k, "sample", **kw)
    assert all(np.array_equal(r1[x], r2[x]) for x in r1)


# ------------------------------------------------- tie diagnostics (parity bands)
def test_top2_gap_on_hand_written_rows():
    # The GPU parity tests drop a sequence whose decision sits inside a tie band; these
    # are the numbers that decide it, so they are fixed here on rows written by hand.
    from oracle.verify import _top2_gap
    s = np.array([[0.0, 3.0, 1.0, 2.5],          # clear winner: index 1, gap 0.5
                  [7.0, 7.0, 1.0, 7.0],          # exact three-way tie: lowest index, gap 0
                  [-np.inf, -2.0, -np.inf, -5.0],  # -inf entries never win: gap 3
                  [4.0, -np.inf, -np.inf, -np.inf]])  # a single finite score: gap inf
    best, gap = _top2_gap(s)
    assert best.tolist() == [1, 0, 1, 0]
    assert gap.tolist() == [0.5, 0.0, 3.0, np.inf]
    # the input is left as it was
    assert s[0, 1] == 3.0 and s[1, 0] == 7.0


def _uniform_by_hand(seed, seq, pos):
    # r of Algorithm 1 for (sequence, position): first Philox word of counter
    # (0, ACCEPT = 0, seq, pos), mapped to ((w >> 9) + 1/2) 2^-23 -- written out here,
    # Philox itself is pinned by its known-answer vectors
    from oracle.philox import philox4x32_10
    w = philox4x32_10(0, 0, seq, pos, seed & 0xFFFFFFFF, seed >> 32)[0]
    return (float(int(w) >> 9) + 0.5) * 2.0 ** -23


def test_accept_margin_on_hand_written_cases():
    k, V, T, seed, L = 2, 2, 1.0, 77, 9
    z = np.zeros((4, layout.n_block_rows(k), V))
    z[:, 0, 1] = np.log(3.0)                      # row 0: Q = (1/4, 3/4)
    z[:, layout.target_rows(k)[1], 0] = np.log(4.0)   # row of c_1: Q = (4/5, 1/5)
    cand = np.array([[1, 0]] * 4)
    seq = np.arange(4)
    r1 = np.array([_uniform_by_hand(seed, s, L + 1) for s in seq])
    r2 = np.array([_uniform_by_hand(seed, s, L + 2) for s in seq])
    P = np.ones((4, k))
    P[0, 0] = 0.75 / r1[0]                        # r*P_c == Q exactly: margin 0 (accepted, "<=")
    P[0, 1] = 2 * 0.8 / r2[0]                     # r*P_c = 2Q: margin 1, rejected
    P[1, 0] = 0.5 * 0.75 / r1[1]                  # r*P_c = Q/2: margin 1/2, accepted
    P[1, 1] = INF                                 # cannot be accepted; no floating-point decision
    P[2, 0] = 3 * 0.75 / r1[2]                    # rejected at i = 1: margin 2 ...
    P[2, 1] = 0.8 / r2[2]                         # ... and position 2 is never tested: inf
    P[3, :] = 1e-9                                # both accepted, margins ~ 1
    r = verify_step(z, cand, P, k, "sample", temperature=T, seed=seed, seq_id=seq,
                    kv_len=np.full(4, L))
    am = r["accept_margin"]
    assert r["n_accept"].tolist() == [1, 1, 0, 2]
    assert am[0, 0] < 1e-15 and abs(am[0, 1] - 1.0) < 1e-12
    assert abs(am[1, 0] - 0.5) < 1e-12 and am[1, 1] == INF
    assert abs(am[2, 0] - 2.0) < 1e-12 and am[2, 1] == INF
    assert np.all(np.abs(am[3] - 1.0) < 1e-6)
    # greedy mode takes no floating-point acceptance decision
    g = verify_step(z, cand, np.ones((4, k)), k, "greedy")
    assert np.all(g["accept_margin"] == INF) and np.all(g["bonus_gap"] == INF)


def test_bonus_gap_matches_scores_written_by_hand():
    # one sequence, three tokens: the extra token's top-two gap recomputed from
    # log Q + Gumbel noise written out explicitly
    from oracle.philox import philox4x32_10
    k, V, T, seed, L = 1, 3, 0.5, 5, 4
    z = np.zeros((1, layout.n_block_rows(k), V))
    z[0, 0] = [0.2, -0.1, 0.4]
    r = verify_step(z, np.array([[1]]), np.full((1, k), INF), k, "sample", temperature=T,
                    seed=seed, kv_len=np.array([L]), resample="paper_literal")
    assert r["n_accept"][0] == 0
    w = philox4x32_10(0, 1, 0, L + 1, seed, 0)       # tokens 0..2 share counter word 0, purpose TOKEN = 1
    u = [(float(int(w[j]) >> 9) + 0.5) * 2.0 ** -23 for j in range(3)]
    q = np.exp(z[0, 0] / T); q /= q.sum()
    score = sorted(np.log(q[j]) - np.log(-np.log(u[j])) for j in range(3))
    assert abs(r["bonus_gap"][0] - (score[2] - score[1])) < 1e-12


# --------------------------------------- Algorithm 1's initial state, odd P_c values
def test_initial_state_draws_the_first_token_from_Q_including_token_zero():
    # L_c = [0]*k, P_c = [+inf]*k (Algorithm 1): everything is rejected and the one
    # emitted token must follow Q -- token 0, the "rejected candidate", included.
    k, T, seed = 2, 0.8, 424242
    z = _fixed_logits(k, 4)
    q0 = softmax_rows(z[0, 0], T)
    r = verify_step(z, np.zeros((N, k), dtype=int), np.full((N, k), INF), k, "sample",
                    temperature=T, seed=seed, seq_id=np.arange(N), kv_len=np.full(N, 3))
    assert np.all(r["n_accept"] == 0)
    counts = np.bincount(r["out_tokens"][:, 0], minlength=V16)
    assert counts[0] > 0
    chi, _ = _chi2(counts, q0)
    assert chi < 55.0, chi


def test_acceptance_needs_a_positive_probability_and_an_in_range_token():
    k, V = 2, 6
    z = _logits(np.random.default_rng(3), 8, k, V)
    for bad_p in (0.0, -1.0, np.nan):
        for c0 in (1, V + 2, -4):
            r = verify_step(z, np.full((8, k), c0), np.full((8, k), bad_p), k, "sample",
                            seed=3, seq_id=np.arange(8))
            assert np.all(r["n_accept"] == 0), (bad_p, c0)


# ------------------------------------------------ filtered sampling (top-k, then top-p)
def test_filter_on_a_hand_written_row():
    from oracle.verify import filter_top_k_top_p
    z = np.log(np.array([[0.05, 0.5, 0.15, 0.2, 0.1]]))
    # top-k = 4 drops token 0; renormalised 0.5, 0.2, 0.15, 0.1 -> 10/19, 4/19, 3/19, 2/19
    p, m = filter_top_k_top_p(z, 1.0, 4, 1.0)
    assert np.allclose(p[0], np.array([0, 10, 3, 4, 2]) / 19.0)
    # top-p = 0.7 on top of it: 10/19 = 0.526 < 0.7 -> token 3 (4/19) is kept too, 14/19 >= 0.7 -> stop
    p, m = filter_top_k_top_p(z, 1.0, 4, 0.7)
    assert np.allclose(p[0], np.array([0, 10, 0, 4, 0]) / 14.0)
    assert abs(m[0] - min(abs(10 / 19 - 0.7), abs(14 / 19 - 0.7), abs(17 / 19 - 0.7))) < 1e-12
    # the first token is always kept; top_k beyond the vocabulary and top_p = 1 change nothing
    p, _ = filter_top_k_top_p(z, 1.0, 4, 0.01)
    assert p[0].tolist() == [0, 1, 0, 0, 0]
    p, _ = filter_top_k_top_p(z, 0.5, 99, 1.0)
    assert np.allclose(p[0], softmax_rows(z, 0.5)[0])
    # a tie at the top-k boundary goes to the lower token; temperature acts before the cut
    zt = np.array([[1.0, 3.0, 1.0, 1.0]])
    p, _ = filter_top_k_top_p(zt, 2.0, 2, 1.0)
    e = np.exp(-1.0)
    assert np.allclose(p[0], np.array([e, 1, 0, 0]) / (1 + e))


def test_filtered_sampling_is_lossless_for_the_filtered_law():
    # point-mass drafts, top-k = 5 and top-p = 0.9: the first emitted token follows the filtered Q of
    # row 0, a token outside the filter is never emitted, and a candidate outside it is never accepted
    from oracle.verify import filter_top_k_top_p
    k, T, seed, tk, tp = 2, 0.8, 77, 5, 0.9
    z = _fixed_logits(k, 5)
    qf, _ = filter_top_k_top_p(z[0, layout.target_rows(k)], T, tk, tp)       # [k+1, V]
    inside = int(np.argsort(qf[0])[-2])                                      # second most likely kept token
    outside = int(np.argmin(qf[0]))
    assert qf[0, outside] == 0.0 and 0.0 < qf[0, inside] < 1.0
    for c0 in (inside, outside):
        cand = np.broadcast_to(np.array([c0, int(np.argmax(qf[1]))]), (N, k))
        r = verify_step(z, cand, np.ones((N, k)), k, "sample", temperature=T, seed=seed, seq_id=np.arange(N),
                        kv_len=np.full(N, 2), top_k=tk, top_p=tp)
        acc = (r["n_accept"] >= 1).mean()
        assert abs(acc - qf[0, c0]) < 5 * np.sqrt(max(qf[0, c0] * (1 - qf[0, c0]), 1e-9) / N) + 1e-12
        counts = np.bincount(r["out_tokens"][:, 0], minlength=V16)
        chi, _ = _chi2(counts, qf[0])                                        # also asserts: nothing outside the filter
        assert chi < 55.0, chi
        sel = r["n_accept"] >= 1
        if sel.any():
            chi, _ = _chi2(np.bincount(r["out_tokens"][sel, 1], minlength=V16), qf[1])
            assert chi < 55.0, chi
    # without a filter the same call does emit tokens outside it
    r = verify_step(z, cand, np.ones((N, k)), k, "sample", temperature=T, seed=seed, seq_id=np.arange(N))
    assert np.bincount(r["out_tokens"][:, 0], minlength=V16)[qf[0] == 0].sum() > 0


def test_filtered_literal_reading_samples_candidates_from_the_filtered_rows():
    from oracle.verify import filter_top_k_top_p
    k, T, tk, tp = 1, 1.0, 4, 0.95
    z = _fixed_logits(k, 6)
    r = verify_step(z, np.zeros((N, k), dtype=int), np.full((N, k), INF), k, "sample", temperature=T, seed=3,
                    seq_id=np.arange(N), resample="paper_literal", top_k=tk, top_p=tp)
    pm, _ = filter_top_k_top_p(z[0, layout.mask_group_rows(k, 0)[0]], T, tk, tp)
    chi, _ = _chi2(np.bincount(r["next_cand"][:, 0], minlength=V16), pm)
    assert chi < 55.0, chi
    assert np.allclose(r["next_cand_prob"][:, 0], pm[r["next_cand"][:, 0]])
    assert np.isfinite(r["nucleus_margin"]).all()


# ------------------------------------------------ compact draft distributions, full residual resampling
def test_compact_draft_residual_on_hand_written_rows():
    from oracle.verify import compact_to_dense
    k, V = 1, 4
    z = np.full((1, layout.n_block_rows(k), V), -50.0)
    z[0, 0] = np.log(np.array([0.5, 0.3, 0.2, 1e-30]))       # Q of the root row; top-k = 3 drops token 3
    n = 4000
    zz = np.broadcast_to(z, (n,) + z.shape[1:])
    tok = np.broadcast_to(np.array([[[0, 2, -1]]]), (n, 1, 3))
    prob = np.broadcast_to(np.array([[[0.8, 0.2, 0.0]]]), (n, 1, 3))
    r = verify_step(zz, np.zeros((n, 1), dtype=int), np.full((n, 1), 0.8), k, "sample", seed=5, seq_id=np.arange(n),
                    resample="residual_draft", top_k=3, top_p=1.0, draft_tok=tok, draft_prob=prob)
    acc = r["n_accept"] == 1
    assert abs(acc.mean() - 0.5 / 0.8) < 5 * np.sqrt(0.625 * 0.375 / n)
    # residual max(0, Q - D) = (0, 0.3, 0, 0): after a rejection the extra token is token 1, always
    assert (r["out_tokens"][~acc, 0] == 1).all() and (~acc).sum() > 1000
    assert (r["out_tokens"][acc, 0] == 0).all()
    # Q(1) = 0.3, D(1) = 0: no subtraction for the winner; the runner-up has no mass
    assert np.allclose(r["bonus_cond"][~acc], 1.0)
    # a residual without mass (Q <= D everywhere) falls back to Q; here forced by P_c = +inf
    prob_q = np.broadcast_to(np.array([[[0.5, 0.2, 0.3]]]), (n, 1, 3))
    tok_q = np.broadcast_to(np.array([[[0, 2, 1]]]), (n, 1, 3))
    r = verify_step(zz, np.zeros((n, 1), dtype=int), np.full((n, 1), INF), k, "sample", seed=6, seq_id=np.arange(n),
                    resample="residual_draft", top_k=3, top_p=1.0, draft_tok=tok_q, draft_prob=prob_q)
    assert (r["n_accept"] == 0).all()
    f = np.bincount(r["out_tokens"][:, 0], minlength=V) / n
    assert np.abs(f - np.array([0.5, 0.3, 0.2, 0.0])).max() < 5 * np.sqrt(0.25 / n)
    # entries that are no distribution entries do not count
    d = compact_to_dense(np.array([[1, -1, 7, 2, 2]]), np.array([[0.5, 0.9, 0.9, np.nan, 0.25]]), 4)
    assert d.tolist() == [[0.0, 0.5, 0.25, 0.0]]
    # cancellation is reported: Q = (0.5, 0.3, 0.2), D = (0.499, 0, 0) -> the weight of token 0 is 0.001
    prob_c = np.broadcast_to(np.array([[[0.499, 0.0, 0.0]]]), (n, 1, 3))
    r = verify_step(zz, np.zeros((n, 1), dtype=int), np.full((n, 1), INF), k, "sample", seed=7, seq_id=np.arange(n),
                    resample="residual_draft", top_k=3, top_p=1.0, draft_tok=tok, draft_prob=prob_c)
    top_two_has_0 = (r["out_tokens"][:, 0] == 0) | (r["bonus_cond"] > 1.0)
    assert np.allclose(r["bonus_cond"][top_two_has_0], 0.5 / 0.001, rtol=1e-6) and top_two_has_0.any()


def test_compact_draft_lists_are_the_filtered_mask_rows():
    from oracle.verify import filter_top_k_top_p
    k, T, tk, tp = 2, 0.7, 5, 0.9
    z = _fixed_logits(k, 8)[:1000]
    n = z.shape[0]
    r = verify_step(z, np.zeros((n, k), dtype=int), np.full((n, k), INF), k, "sample", temperature=T, seed=9,
                    seq_id=np.arange(n), resample="residual_draft", top_k=tk, top_p=tp)
    for o in range(k):
        pm, _ = filter_top_k_top_p(z[0, layout.mask_group_rows(k, 0)[o]], T, tk, tp)
        t, p = r["next_draft_tok"][0, o], r["next_draft_prob"][0, o]
        kept = t >= 0
        assert abs(p.sum() - 1.0) < 1e-12 and (p[~kept] == 0).all() and (np.diff(p[kept]) <= 0).all()
        assert np.allclose(pm[t[kept]], p[kept]) and np.count_nonzero(pm) == kept.sum()
        # P_c is the list's probability of the drawn token
        c = r["next_cand"][:, o]
        assert np.allclose(r["next_cand_prob"][:, o], pm[c]) and (pm[c] > 0).all()


def test_compact_draft_residual_is_lossless_where_algorithm_1_as_printed_is_not():
    # Step A draws the candidates from the filtered mask rows of one set of logits; step B verifies them
    # against other logits.  With the residual rule the first emitted token follows the filtered Q of the
    # root row exactly, and the token after an accepted candidate the filtered Q of that candidate's row;
    # with a ~ Q after a rejection (Algorithm 1 as printed) the first token's law is
    # min(D, Q) + (1 - sum min(D, Q)) Q instead, which the same test tells apart.
    from oracle.verify import filter_top_k_top_p
    k, T, tk, tp = 2, 0.9, 5, 0.9
    zA = _fixed_logits(k, 21)
    # the verifying model agrees with the drafts in part: its target rows are the mask rows plus noise
    zb = np.array(_fixed_logits(k, 22)[0])
    zb[layout.target_rows(k)[0]] = zA[0, layout.mask_group_rows(k, 0)[0]] + 0.6 * zb[layout.target_rows(k)[0]]
    zB = np.broadcast_to(zb[None], zA.shape)
    ids = np.arange(N)
    rA = verify_step(zA, np.zeros((N, k), dtype=int), np.full((N, k), INF), k, "sample", temperature=T, seed=11,
                     seq_id=ids, resample="residual_draft", top_k=tk, top_p=tp)
    D1, _ = filter_top_k_top_p(zA[0, layout.mask_group_rows(k, 0)[0]], T, tk, tp)
    qf, _ = filter_top_k_top_p(zB[0, layout.target_rows(k)], T, tk, tp)
    assert 0.2 < np.minimum(D1, qf[0]).sum() < 0.9            # a real mix of acceptances and rejections
    kw = dict(temperature=T, seed=12, seq_id=ids, kv_len=np.full(N, 3), top_k=tk, top_p=tp)
    r = verify_step(zB, rA["next_cand"], rA["next_cand_prob"], k, "sample", resample="residual_draft",
                    draft_tok=rA["next_draft_tok"], draft_prob=rA["next_draft_prob"], **kw)
    acc = (r["n_accept"] >= 1).mean()
    want = np.minimum(D1, qf[0]).sum()
    assert abs(acc - want) < 5 * np.sqrt(want * (1 - want) / N)
    chi, _ = _chi2(np.bincount(r["out_tokens"][:, 0], minlength=V16), qf[0])
    assert chi < 55.0, chi
    # second token, by accepted first candidate c: its law is the filtered Q of row 1 (the row depends on c only
    # through the acceptance, the logits here being fixed)
    sel = r["n_accept"] >= 1
    chi, _ = _chi2(np.bincount(r["out_tokens"][sel, 1], minlength=V16), qf[1])
    assert chi < 55.0, chi
    # Algorithm 1 as printed on the same candidates
    rl = verify_step(zB, rA["next_cand"], rA["next_cand_prob"], k, "sample", resample="paper_literal", **kw)
    mix = np.minimum(D1, qf[0]) + (1 - want) * qf[0]
    chi_l, _ = _chi2(np.bincount(rl["out_tokens"][:, 0], minlength=V16), mix)
    assert chi_l < 55.0, chi_l
    chi_wrong, _ = _chi2(np.bincount(rl["out_tokens"][:, 0], minlength=V16), qf[0])
    assert chi_wrong > 1000.0, chi_wrong
