"""Pins for oracle.sar_sft (Sec. 3.1, App. A.1): a hand-written example, the statistics the text
fixes (share of unchanged samples p_ar, m uniform on {0..N-k}), and the structure of a masked
sample (y_1..y_m, k masks, cut after m+k answer tokens, labels intact up to the cut)."""
import numpy as np

from oracle.sar_sft import sar_sft_transform

M, PAD, IGN = 99, 0, -100


def test_hand_written_example():
    # prompt (7, 8), answer y = 11..16 (N = 6), k = 2.  second word 0x80000000: m = (N-k+1)/2 = 2
    ids = np.array([[7, 8, 11, 12, 13, 14, 15, 16, PAD, PAD]] * 3)
    lab = np.array([[IGN, IGN, 11, 12, 13, 14, 15, 16, IGN, IGN]] * 3)
    words = np.array([[0xFFFFFFFF, 0x80000000],          # masked sample, m = 2
                      [0x00000005, 0x80000000],          # first word below the threshold: unchanged
                      [0xFFFFFFFF, 0xFFFFFFFF]], dtype=np.uint64)   # m = N - k = 4: the last k tokens
    out, olab, n, m = sar_sft_transform(ids, lab, [2, 2, 2], [6, 6, 6], words, 2, M, ar_threshold=10,
                                        pad_token_id=PAD, ignore_index=IGN)
    assert m.tolist() == [2, -1, 4]
    assert out[0].tolist() == [7, 8, 11, 12, M, M, PAD, PAD, PAD, PAD]      # y_1 y_2 [M][M], cut
    assert olab[0].tolist() == [IGN, IGN, 11, 12, 13, 14, IGN, IGN, IGN, IGN]  # labels y_1..y_{m+k}
    assert out[1].tolist() == ids[1].tolist() and olab[1].tolist() == lab[1].tolist()
    assert out[2].tolist() == [7, 8, 11, 12, 13, 14, M, M, PAD, PAD]
    assert olab[2].tolist() == lab[2].tolist()
    assert n.tolist() == [6, 8, 8]
    # the inputs are left as they were
    assert ids[0, 4] == 13


def test_short_answers_stay_autoregressive_and_m_zero_masks_the_first_tokens():
    ids = np.array([[5, 21, 22, PAD, PAD], [5, 21, 22, 23, PAD]])
    lab = np.array([[IGN, 21, 22, IGN, IGN], [IGN, 21, 22, 23, IGN]])
    words = np.array([[0xFFFFFFFF, 0], [0xFFFFFFFF, 0]], dtype=np.uint64)
    out, olab, n, m = sar_sft_transform(ids, lab, [1, 1], [2, 3], words, 3, M, ar_threshold=0)
    assert m.tolist() == [-1, 0]                         # N = 2 < k: unchanged; N = k: only m = 0
    assert out[0].tolist() == ids[0].tolist()
    assert out[1].tolist() == [5, M, M, M, PAD] and olab[1].tolist() == [IGN, 21, 22, 23, IGN]


def test_statistics_follow_the_text():
    rng = np.random.default_rng(0)
    B, P, N, k, p_ar = 200_000, 3, 12, 5, 0.5
    ids = np.tile(np.arange(1, P + N + 1), (B, 1))
    lab = ids.copy()
    words = rng.integers(0, 2 ** 32, size=(B, 2), dtype=np.uint64)
    out, olab, n, m = sar_sft_transform(ids, lab, [P] * B, [N] * B, words, k, M,
                                        ar_threshold=int(round(p_ar * 2 ** 32)))
    unchanged = (m < 0)
    assert abs(unchanged.mean() - p_ar) < 5 * np.sqrt(0.25 / B)          # p_ar of the samples stay
    counts = np.bincount(m[~unchanged], minlength=N - k + 1)
    assert len(counts) == N - k + 1 and counts.min() > 0                 # m in {0..N-k}, all values occur
    expect = (~unchanged).sum() / (N - k + 1)
    assert float(((counts - expect) ** 2 / expect).sum()) < 40.0         # uniform (7 dof)
    # structure of every masked sample
    sel = np.nonzero(~unchanged)[0][:2000]
    for b in sel:
        mm = int(m[b])
        assert (out[b, P + mm: P + mm + k] == M).all() and (out[b, : P + mm] == ids[b, : P + mm]).all()
        assert (out[b, P + mm + k:] == 0).all() and n[b] == P + mm + k
        assert (olab[b, : P + mm + k] == lab[b, : P + mm + k]).all() and (olab[b, P + mm + k:] == -100).all()
    assert (out[unchanged] == ids[unchanged]).all() and (n[unchanged] == P + N).all()
