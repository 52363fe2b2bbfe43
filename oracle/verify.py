"""Verification and emission of one auto-correct step (Algorithm 1, body of
the loop after the model call), vectorised over the batch.

Test infrastructure.  Names follow Algorithm 1: L_c candidates, P_c their
probabilities from the previous step, Q the current target distribution,
a the extra token.  `logits` holds one row per block row; the paper's
"normalized output logits" P are softmax(logits / T) taken in float64.

Row use (1-based Algorithm 1 indices translated to block rows):
  Q = P[l]              -> target row 0 (the root);
  Q = P[l + i(k+1)]     -> target row i (candidate c_i);
  P[idx : idx+k]        -> the k mask rows of group i* (i* = accepted count).

Random numbers are Philox4x32-10 words keyed by the 64-bit seed, with counter
(c0, purpose, sequence id, position):
  ACCEPT  c0 = 0, position L+i,           lane 0: the r of Algorithm 1 for c_i
  TOKEN   c0 = x>>2, position L+i*+1,     lane x&3: Gumbel noise of token x for a ~ Q
  DRAFT   c0 = x>>2, position L+i*+1+o,   lane x&3: Gumbel noise for L_c[o] ~ P[..]
A categorical draw "x ~ w" is argmax_x (log w(x) - log(-log u_x)), lowest index
on ties, which has exactly the law w.

resample:
  "residual_pointmass"  lossless variant: candidates are the arg-max of their
        mask row and carry P_c = 1 (a point-mass draft).  c_i is accepted with
        probability Q(c_i); after a rejection the extra token is drawn from Q
        with the rejected token removed (the residual of a point mass).
        The removal applies only to a candidate that really is a point mass
        (P_c = 1).  Algorithm 1 starts from L_c = [0]*k, P_c = [+inf]*k: such a
        candidate is rejected with certainty, its rejection says nothing about
        the token, and the extra token is drawn from Q unchanged (so token 0
        can be emitted at the first step).  Any other P_c is not a point-mass
        draft either and is treated the same way (a ~ Q, Algorithm 1 as printed).
An acceptance needs an in-range candidate and P_c > 0 (a drafted token cannot
have had probability zero; this also keeps NaN and negative values from passing
the test r*P_c <= Q by accident).
  "paper_literal"       Algorithm 1 as printed: a ~ Q also after a rejection,
        new candidates are sampled from their mask rows and P_c is the sampled
        token's probability.
  "residual_draft"      sampled candidates made lossless (needs top_k > 0): candidate o of the
        next step is drawn from the filtered distribution D_o of its mask row, and the step hands
        D_o on as a compact list (at most top_k tokens with their probabilities, descending) beside
        L_c and P_c = D_o(L_c[o]).  The next step accepts c_i with probability min(1, Q(c_i)/P_c[i])
        as Algorithm 1 does, and after rejecting c_i draws the extra token from the residual
        norm(max(0, Q - D_i)), the rule of speculative sampling that Sec. 3.2's claim of an
        unchanged output distribution rests on; after k acceptances, and in Algorithm 1's initial
        state (empty lists), a ~ Q.  Should the residual have no mass (Q <= D_i everywhere, where a
        rejection has probability zero) Q itself is used.
Greedy mode is the zero-temperature limit: accept iff c_i is the arg-max of Q,
a = argmax Q, new candidates are the mask rows' arg-maxes.

Filtered sampling (App. A.4 runs random sampling with top-k = 10 and top-p = 0.95): with
top_k > 0 every distribution that is sampled from or tested against -- Q of the target rows,
and the mask rows' distributions when candidates are sampled -- is softmax(z / T) restricted
to its top_k largest logits (lowest index first on ties), then to the shortest prefix of
those, in descending order, whose probability reaches top_p, and renormalised.  The
auto-correct step is then lossless with respect to that filtered distribution.
"""
import numpy as np

from .bf16 import as_f64
from .layout import target_rows, mask_group_rows, n_block_rows
from .philox import philox4x32_10, uniform_open

PURPOSE_ACCEPT, PURPOSE_TOKEN, PURPOSE_DRAFT = 0, 1, 2


def softmax_rows(z, T=1.0):
    z = np.asarray(z, dtype=np.float64) / T
    z = z - z.max(axis=-1, keepdims=True)
    e = np.exp(z)
    return e / e.sum(axis=-1, keepdims=True)


def filter_top_k_top_p(z, T, top_k, top_p, as_list=False):
    """z [..., V] logits -> (filtered, renormalised probabilities [..., V], nucleus_margin [...]);
    with as_list the distribution comes as (tokens [..., K], probabilities [..., K], margin) in
    descending order, K = min(top_k, V), dropped entries as token -1 with probability 0.

    Temperature, then top-k, then top-p, in that order: keep the top_k largest z (ties: lower
    index first); p = softmax(z / T) over them; in descending order keep token j while the
    probability of the tokens before it is below top_p (the first one is always kept; top_p >= 1
    keeps all of them).
    nucleus_margin: smallest |that cumulative probability - top_p| over the top-k tokens after the
    first -- how close the floating-point decision "before it is below top_p" came to a tie."""
    z = np.asarray(z, dtype=np.float64)
    shape, V = z.shape[:-1], z.shape[-1]
    z2 = z.reshape(-1, V)
    K = min(int(top_k), V) if top_k > 0 else V
    order = np.argsort(-z2, axis=1, kind="stable")[:, :K]    # descending, lowest index first on ties
    s = np.take_along_axis(z2, order, axis=1) / T
    p = np.exp(s - s[:, :1])
    p /= p.sum(axis=1, keepdims=True)
    cum = np.cumsum(p, axis=1)
    before = np.concatenate((np.zeros((z2.shape[0], 1)), cum[:, :-1]), axis=1)   # probability of the tokens before j
    if top_p >= 1.0:                                         # no nucleus cut at all
        keep = np.ones_like(before, dtype=bool)
        margin = np.full(z2.shape[0], np.inf)
    else:
        keep = before < top_p
        keep[:, 0] = True
        margin = np.abs(before[:, 1:] - top_p).min(axis=1) if K > 1 else np.full(z2.shape[0], np.inf)
    pk = np.where(keep, p, 0.0)
    pk /= pk.sum(axis=1, keepdims=True)
    out = np.zeros_like(z2)
    np.put_along_axis(out, order, pk, axis=1)
    if as_list:
        tok = np.where(keep, order, -1)
        return tok.reshape(shape + (K,)), pk.reshape(shape + (K,)), margin.reshape(shape)
    return out.reshape(shape + (V,)), margin.reshape(shape)


def compact_to_dense(tok, prob, V):
    """Compact distribution lists tok, prob [B, K] -> dense [B, V]; entries with a token outside
    [0, V) or a probability that is not a positive finite number do not count."""
    tok = np.asarray(tok, dtype=np.int64)
    prob = np.asarray(prob, dtype=np.float64)
    ok = (tok >= 0) & (tok < V) & np.isfinite(prob) & (prob > 0)
    out = np.zeros((tok.shape[0], V))
    b = np.broadcast_to(np.arange(tok.shape[0])[:, None], tok.shape)
    np.add.at(out, (b[ok], tok[ok]), prob[ok])
    return out


def gumbel_noise(seed, purpose, seq_id, position, V):
    """-log(-log u_x) for x = 0..V-1; seq_id, position: [B] -> [B, V]."""
    x = np.arange(V, dtype=np.uint64)[None, :]
    w = philox4x32_10(x >> np.uint64(2), purpose,
                      np.asarray(seq_id, dtype=np.uint64)[:, None],
                      np.asarray(position, dtype=np.uint64)[:, None],
                      seed & 0xFFFFFFFF, seed >> 32)
    lane = (x & np.uint64(3)).astype(np.int64)
    lane = np.broadcast_to(lane, w[0].shape)
    word = np.choose(lane, w)
    return -np.log(-np.log(uniform_open(word)))


def accept_uniform(seed, seq_id, position):
    w = philox4x32_10(0, PURPOSE_ACCEPT, np.asarray(seq_id, dtype=np.uint64),
                      np.asarray(position, dtype=np.uint64), seed & 0xFFFFFFFF, seed >> 32)
    return uniform_open(w[0])


def _top2_gap(score):
    """arg-max (lowest index on ties) and the gap to the runner-up, per row."""
    best = np.argmax(score, axis=-1)
    top = np.take_along_axis(score, best[:, None], axis=-1)[:, 0]
    s2 = score.copy()
    np.put_along_axis(s2, best[:, None], -np.inf, axis=-1)
    return best, top - s2.max(axis=-1)


def verify_step(logits, cand, cand_prob, k, mode="greedy", temperature=1.0, seed=0,
                seq_id=None, kv_len=None, resample="residual_pointmass", eos_id=-1, top_k=0, top_p=1.0,
                draft_tok=None, draft_prob=None):
    """logits [B, n_q, V]; cand (L_c) [B, k] ints; cand_prob (P_c) [B, k];
    draft_tok, draft_prob [B, k, K_d] ("residual_draft" only): the compact distributions the
    candidates were drawn from (None = empty lists, Algorithm 1's initial state).  That reading
    also returns next_draft_tok, next_draft_prob [B, k, min(top_k, V)] and bonus_cond [B], the
    condition number max(Q, D) / (Q - D) of the residual weight of the winning token or of its
    runner-up, whichever is larger (1 when no subtraction took place).

    Returns a dict: n_accept (i*), out_tokens [B, k+1] (-1 padded), n_out,
    next_cand, next_cand_prob, finished, and tie diagnostics
    (accept_margin [B, k] relative distance of the acceptance test from
    equality, bonus_gap [B], draft_gap [B, k] Gumbel top-two gaps; inf when
    no floating-point decision was taken; nucleus_margin [B] likewise for the top-p cuts of
    the rows that were read).
    """
    logits = np.asarray(logits)
    B, n_q, V = logits.shape
    assert n_q == n_block_rows(k)
    L_c = np.asarray(cand, dtype=np.int64)
    P_c = np.asarray(cand_prob, dtype=np.float64)
    seq_id = np.arange(B) if seq_id is None else np.asarray(seq_id)
    L = np.zeros(B, dtype=np.int64) if kv_len is None else np.asarray(kv_len, dtype=np.int64)
    bi = np.arange(B)
    T = float(temperature)
    greedy = mode == "greedy"
    trow = target_rows(k)
    z_t = as_f64(logits[:, trow, :])                         # [B, k+1, V]
    in_range = (L_c >= 0) & (L_c < V)
    c_safe = np.where(in_range, L_c, 0)

    if greedy:
        top = np.argmax(z_t, axis=-1)                        # lowest index on ties
    elif top_k > 0:
        Qrows, q_margin = filter_top_k_top_p(z_t, T, top_k, top_p)   # [B, k+1, V], [B, k+1]
    else:
        Qrows = softmax_rows(z_t, T)                         # [B, k+1, V]

    # ---- verification loop (Algorithm 1, for i = 1..k) -------------------
    alive = np.ones(B, dtype=bool)
    i_star = np.zeros(B, dtype=np.int64)
    accept_margin = np.full((B, k), np.inf)
    for i in range(1, k + 1):
        c_i = c_safe[:, i - 1]
        if greedy:
            ok = in_range[:, i - 1] & (top[:, i - 1] == L_c[:, i - 1])
        else:
            Q_ci = np.where(in_range[:, i - 1], Qrows[bi, i - 1, c_i], 0.0)
            r = accept_uniform(seed, seq_id, L + i)
            with np.errstate(invalid="ignore"):
                lhs = r * P_c[:, i - 1]                      # r <= Q/P_c  <=>  r*P_c <= Q
                ok = in_range[:, i - 1] & (P_c[:, i - 1] > 0) & (lhs <= Q_ci)
                marg = np.abs(lhs - Q_ci) / np.maximum(Q_ci, 1e-300)
            accept_margin[:, i - 1] = np.where(alive & np.isfinite(lhs), marg, np.inf)
        alive = alive & ok
        i_star += alive

    # ---- extra token a from the last accepted row ------------------------
    bonus_gap = np.full(B, np.inf)
    bonus_cond = np.ones(B)
    if greedy:
        a = top[bi, i_star]
    else:
        w = Qrows[bi, i_star, :].copy()                      # [B, V]
        if resample == "residual_pointmass":
            rej = i_star < k
            c_rej = c_safe[bi, np.minimum(i_star, k - 1)]
            rej = rej & in_range[bi, np.minimum(i_star, k - 1)]
            rej = rej & (P_c[bi, np.minimum(i_star, k - 1)] == 1.0)   # a point-mass draft only
            w[bi[rej], c_rej[rej]] = 0.0
        if resample == "residual_draft":
            assert top_k > 0, "compact draft distributions need top_k > 0"
            Qw = w.copy()
            D = np.zeros((B, V))
            if draft_tok is not None:
                dt = np.asarray(draft_tok)[bi, np.minimum(i_star, k - 1)]     # list of the rejected candidate
                dp = np.asarray(draft_prob)[bi, np.minimum(i_star, k - 1)]
                D = compact_to_dense(dt, dp, V)
            D[i_star >= k] = 0.0                             # nothing was rejected
            res = np.maximum(Qw - D, 0.0)
            empty = res.sum(axis=1) <= 0.0
            w = np.where(empty[:, None], Qw, res)
            D[empty] = 0.0
        with np.errstate(divide="ignore"):
            score = np.log(w) + gumbel_noise(seed, PURPOSE_TOKEN, seq_id, L + i_star + 1, V)
        a, bonus_gap = _top2_gap(score)
        if resample == "residual_draft":
            s2 = score.copy()
            s2[bi, a] = -np.inf
            for t in (a, np.argmax(s2, axis=-1)):
                ok_t = w[bi, t] > 0
                cond = np.where(ok_t, np.maximum(Qw[bi, t], D[bi, t]) / np.where(ok_t, w[bi, t], 1.0), 1.0)
                bonus_cond = np.maximum(bonus_cond, cond)

    out_tokens = np.full((B, k + 1), -1, dtype=np.int64)
    for j in range(k + 1):
        tok = L_c[:, j] if j < k else a
        out_tokens[:, j] = np.where(j < i_star, tok, np.where(j == i_star, a, -1))
    n_out = i_star + 1

    # ---- end of sequence: keep the tokens before the first <EOS> ---------
    finished = np.zeros(B, dtype=np.uint8)
    if eos_id >= 0:
        is_eos = (out_tokens == eos_id)
        has = is_eos.any(axis=1)
        first = np.argmax(is_eos, axis=1)
        n_out = np.where(has, first, n_out)
        finished = has.astype(np.uint8)
        out_tokens = np.where(np.arange(k + 1)[None, :] < n_out[:, None], out_tokens, -1)

    # ---- new candidates from mask group i* --------------------------------
    next_cand = np.zeros((B, k), dtype=np.int64)
    next_cand_prob = np.zeros((B, k), dtype=np.float64)
    draft_gap = np.full((B, k), np.inf)
    nucleus_margin = np.full(B, np.inf)
    if not greedy and top_k > 0:
        # target rows 0 .. i* are the ones whose filtered distribution was used
        used = np.arange(k + 1)[None, :] <= i_star[:, None]
        nucleus_margin = np.where(used, q_margin, np.inf).min(axis=1)
    K_d = min(int(top_k), V) if top_k > 0 else 0
    next_draft_tok = np.full((B, k, K_d), -1, dtype=np.int64)
    next_draft_prob = np.zeros((B, k, K_d))
    rows = np.array([mask_group_rows(k, g) for g in range(k + 1)])   # [k+1, k]
    for o in range(1, k + 1):
        z = as_f64(logits[bi, rows[i_star, o - 1], :])       # [B, V]
        if greedy:
            next_cand[:, o - 1] = np.argmax(z, axis=-1)
            next_cand_prob[:, o - 1] = softmax_rows(z, 1.0)[bi, next_cand[:, o - 1]]
        elif resample == "residual_pointmass":
            next_cand[:, o - 1] = np.argmax(z, axis=-1)
            next_cand_prob[:, o - 1] = 1.0
        else:
            if top_k > 0:
                p, m_o = filter_top_k_top_p(z, T, top_k, top_p)
                nucleus_margin = np.minimum(nucleus_margin, m_o)
                if resample == "residual_draft":
                    next_draft_tok[:, o - 1], next_draft_prob[:, o - 1], _ = filter_top_k_top_p(z, T, top_k, top_p, as_list=True)
            else:
                p = softmax_rows(z, T)
            with np.errstate(divide="ignore"):
                score = np.log(p) + gumbel_noise(seed, PURPOSE_DRAFT, seq_id, L + i_star + 1 + o, V)
            best, gap = _top2_gap(score)
            next_cand[:, o - 1] = best
            next_cand_prob[:, o - 1] = p[bi, best]
            draft_gap[:, o - 1] = gap

    return dict(n_accept=i_star, out_tokens=out_tokens, n_out=n_out, next_cand=next_cand,
                next_cand_prob=next_cand_prob, finished=finished,
                accept_margin=accept_margin, bonus_gap=bonus_gap, draft_gap=draft_gap,
                nucleus_margin=nucleus_margin, bonus_cond=bonus_cond,
                next_draft_tok=next_draft_tok, next_draft_prob=next_draft_prob)
