"""Output projection followed by verification (greedy or sampling), in float64.

Test infrastructure.  In Algorithm 1 the model call P = M(I) ends with the
language-model head: every block row's final hidden state h is multiplied with
the output embedding W (one row per vocabulary token), logits[r, x] = <h_r, W_x>,
and the rows of P are the softmax of those logits.  The verification loop, the
extra token and the new candidates of Algorithm 1 then read those rows.  The
projection is the plain definition of a matrix product; it is written out here
with numpy's float64 product on exactly converted bf16 inputs, and its result
is handed to `verify.verify_step` unchanged.
"""
import numpy as np

from .bf16 import as_f64
from .verify import verify_step


def lm_head_logits(hidden, weight):
    """hidden [B, n_q, D], weight [V, D] (bf16 bit patterns or floats)
    -> logits [B, n_q, V] float64 with logits[b, r, x] = sum_d hidden[b, r, d] * weight[x, d]."""
    h = as_f64(hidden)
    W = as_f64(weight)
    assert h.shape[-1] == W.shape[-1]
    return h @ W.T


def top_two_gap(logits):
    """[B, n_q, V] -> [B, n_q]: largest value minus the largest value at any other
    index (0 on an exact tie).  The arg-max of a row is a floating-point decision;
    a row whose gap is inside the comparison band is excluded from parity and logged."""
    z = np.asarray(logits, dtype=np.float64)
    best = np.argmax(z, axis=-1)
    top = np.take_along_axis(z, best[..., None], axis=-1)[..., 0]
    rest = z.copy()
    np.put_along_axis(rest, best[..., None], -np.inf, axis=-1)
    return top - rest.max(axis=-1)


def lmhead_verify_step(hidden, weight, cand, cand_prob, k, eos_id=-1, mode="greedy", temperature=1.0,
                       seed=0, seq_id=None, kv_len=None, resample="residual_pointmass"):
    """One step of Algorithm 1 from hidden states: projection, then verification (greedy, or
    rejection sampling with the same Philox keying as verify.verify_step).

    Returns verify_step's dict plus `logits` (float64) and `row_gap` [B, n_q]."""
    logits = lm_head_logits(hidden, weight)
    r = verify_step(logits, cand, cand_prob, k, mode, temperature=temperature, seed=seed, seq_id=seq_id,
                    kv_len=kv_len, resample=resample, eos_id=eos_id)
    r["logits"] = logits
    r["row_gap"] = top_two_gap(logits)
    return r
