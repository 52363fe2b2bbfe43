"""SAR-SFT sample transform (Sec. 3.1, App. A.1): the CUDA kernel against oracle.sar_sft on the same
seeded batch and random words, every output exactly."""
import numpy as np
import pytest
import torch

from oracle.sar_sft import sar_sft_transform

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,S,k,p_ar", [(1, 16, 2, 0.0), (257, 300, 5, 0.5), (64, 2048, 5, 0.3), (33, 40, 7, 1.0)])
def test_sar_sft_transform_matches_oracle(B, S, k, p_ar):
    from paper_2402_11809_b200 import build
    build.build()
    from paper_2402_11809_b200 import binding as Bd
    rng = np.random.default_rng(B * 7 + k)
    prompt_len = rng.integers(0, S // 3 + 1, size=B).astype(np.int32)
    answer_len = np.array([rng.integers(0, S - p + 1) for p in prompt_len], dtype=np.int32)
    answer_len[: min(B, 3)] = np.minimum([0, k - 1, k][: min(B, 3)], S - prompt_len[: min(B, 3)])   # too short / just long enough
    ids = rng.integers(1, 30000, size=(B, S)).astype(np.int32)
    lab = ids.copy()
    for b in range(B):
        ids[b, prompt_len[b] + answer_len[b]:] = 0
        lab[b, : prompt_len[b]] = -100
        lab[b, prompt_len[b] + answer_len[b]:] = -100
    words = rng.integers(0, 2 ** 32, size=(B, 2), dtype=np.uint64).astype(np.uint32)
    thr = min(int(round(p_ar * 2 ** 32)), 2 ** 32 - 1)
    want = sar_sft_transform(ids, lab, prompt_len, answer_len, words.astype(np.uint64), k, 32000, thr)
    d = lambda a: torch.from_numpy(a).cuda()
    d_ids, d_lab = d(ids.copy()), d(lab.copy())
    new_len = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    mstart = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    Bd.space_sar_sft_transform(d_ids, d_lab, d(prompt_len), d(answer_len), d(words.view(np.int32)), k, 32000, thr,
                               new_len=new_len, mask_start=mstart)
    torch.cuda.synchronize()
    assert np.array_equal(d_ids.cpu().numpy(), want[0])
    assert np.array_equal(d_lab.cpu().numpy(), want[1])
    assert np.array_equal(new_len.cpu().numpy(), want[2])
    assert np.array_equal(mstart.cpu().numpy(), want[3])
    if 0.0 < p_ar < 1.0:
        assert (want[3] >= 0).any() and (want[3] < 0).any()
