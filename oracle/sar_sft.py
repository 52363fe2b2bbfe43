"""Sample transform of semi-autoregressive fine-tuning (Sec. 3.1, App. A.1) -- test infrastructure.

SAR-SFT changes only the data loader: a sample (prompt X, answer Y = y_1..y_N) stays as it is
with probability p_ar; otherwise a position m is drawn from {0, 1, .., N-k}, the k answer
tokens from there on are replaced by the mask token in the input, the label sequence is left
as it is, and input and labels are cut after the first m+k answer tokens.  The model then
sees y_1..y_m, [M]*k and is trained to predict y_1..y_{m+k}.

Readings: m counts kept answer tokens (0-based: m = 0 masks the first k answer tokens), which
is the reading under which "keep the first m+k tokens" and the draw from {0..N-k} agree; an
answer shorter than k cannot be masked and stays autoregressive.  Randomness comes in as two
32-bit words per sample: the sample stays autoregressive when the first word is below
ar_threshold = round(p_ar * 2^32), and m = (second word * (N-k+1)) >> 32 -- integer
arithmetic, so that every implementation takes the same decision.
"""
import numpy as np


def sar_sft_transform(input_ids, labels, prompt_len, answer_len, rand_words, k, mask_token_id,
                      ar_threshold, pad_token_id=0, ignore_index=-100):
    """input_ids, labels [B, S] (a sample occupies its first prompt_len + answer_len slots);
    rand_words [B, 2] uint32.  Returns (input_ids, labels, new_len [B], mask_start [B]) as new
    arrays; mask_start is m, or -1 for a sample left autoregressive."""
    ids = np.array(input_ids, dtype=np.int64, copy=True)
    lab = np.array(labels, dtype=np.int64, copy=True)
    B, S = ids.shape
    new_len = np.zeros(B, dtype=np.int64)
    mask_start = np.full(B, -1, dtype=np.int64)
    for b in range(B):
        P, N = int(prompt_len[b]), int(answer_len[b])
        w0, w1 = int(rand_words[b][0]), int(rand_words[b][1])
        new_len[b] = P + N
        if w0 < int(ar_threshold) or N < k:
            continue                                        # the sample stays autoregressive
        m = (w1 * (N - k + 1)) >> 32                        # uniform on {0, .., N-k}
        mask_start[b] = m
        for j in range(k):
            ids[b, P + m + j] = mask_token_id               # k consecutive answer tokens become [M]
        keep = P + m + k                                    # input and labels are cut after m+k answer tokens
        ids[b, keep:] = pad_token_id
        lab[b, keep:] = ignore_index
        new_len[b] = keep
    return ids, lab, new_len, mask_start
