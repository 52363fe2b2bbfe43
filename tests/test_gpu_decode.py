"""The decoding loop of Algorithm 1 with its state on the GPU: space_decode_begin, then per step the
user's model (here the toy language model of oracle/decode.py, its projections taken in torch),
space_attn_step, space_verify_commit and space_decode_advance, enqueued without any host round trip.
The tokens must equal the oracle's autoregressive greedy tokens and the cache the autoregressive
cache (Sec. 3.2: the method is lossless), exactly."""
import numpy as np
import pytest
import torch

from oracle.decode import ToyLM, autoregressive_greedy, space_decode
from oracle.bf16 import bf16_bits_to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2402_11809_b200 import build
    build.build()
    from paper_2402_11809_b200 import binding
    return binding


class TorchToy:
    """The toy model's own layers (embedding, projections, vocabulary head) in torch float64 on the
    GPU: the "user model" around the library's attention."""

    def __init__(self, lm):
        t = lambda a: torch.from_numpy(a).cuda()
        self.emb, self.pos, self.wq, self.wk, self.wv, self.wo = (t(a) for a in (lm.emb, lm.pos, lm.wq, lm.wk, lm.wv, lm.wo))
        self.H, self.d = lm.H, lm.d

    def qkv(self, tokens, positions):                        # [B, n] int -> three [B, n, H, d] bf16
        x = self.emb[tokens.long()] + self.pos[positions.long()]
        sh = tokens.shape + (self.H, self.d)
        return tuple((x @ w).float().to(torch.bfloat16).reshape(sh) for w in (self.wq, self.wk, self.wv))

    def head(self, attn, tokens, positions):                 # attn [B, n, H, d] f32 -> logits [B, n, V] f32
        x = self.emb[tokens.long()] + self.pos[positions.long()]
        return ((x + attn.double().reshape(x.shape)) @ self.wo).float()


@pytest.mark.parametrize("k,seed", [(1, 0), (2, 1), (3, 2), (5, 3)])
def test_decode_driver_equals_autoregressive_greedy(B, k, seed):
    V, H, d, n_new, S = 9, 2, 64, 40, 256
    prompts = [[1, 2, 3, 4], [5, 6, 7, 8, 0, 1]]
    Bn, n_q = len(prompts), (k + 1) ** 2
    lm = ToyLM(V, H, d, seed, bf16=True)
    tm = TorchToy(lm)
    want = []
    for p in prompts:
        w, gap = autoregressive_greedy(lm, p, n_new + 2 * (k + 1))
        assert gap > 1e-2, "the toy model has a near-tie for this seed: pick another"
        want.append(w)
    ctx = B.Context(device=0, max_batch=Bn, n_q_heads=H, n_kv_heads=H, head_dim=d, k_max=k, vocab=V, s_cap=S)
    dev = "cuda"
    kc = torch.zeros((Bn, H, S, d), dtype=torch.bfloat16, device=dev)
    vc = torch.zeros_like(kc)
    kv_len = torch.tensor([len(p) - 1 for p in prompts], dtype=torch.int32, device=dev)
    for b, p in enumerate(prompts):                          # prefill: the cache holds x_1 .. x_{l-1}
        t = torch.tensor(p[:-1], device=dev)[None]
        _, K0, V0 = tm.qkv(t, torch.arange(len(p) - 1, device=dev)[None])
        kc[b, :, : len(p) - 1] = K0[0].permute(1, 0, 2)
        vc[b, :, : len(p) - 1] = V0[0].permute(1, 0, 2)
    i32 = lambda *s: torch.full(s, -7, dtype=torch.int32, device=dev)
    max_tokens = n_new + 2 * (k + 1)
    st = dict(tokens=i32(Bn, max_tokens), n_tokens=i32(Bn), last_token=i32(Bn), cand=i32(Bn, k),
              cand_prob=torch.zeros((Bn, k), device=dev), finished=torch.full((Bn,), 9, dtype=torch.uint8, device=dev),
              block_tokens=i32(Bn, n_q), block_pos=i32(Bn, n_q))
    state = ctx.decode_state(st["tokens"], st["n_tokens"], st["last_token"], st["cand"], st["cand_prob"], kv_len,
                             st["finished"], st["block_tokens"], st["block_pos"], k, mask_token_id=V)
    out = torch.zeros((Bn, n_q, H, d), device=dev)
    status = torch.zeros(Bn, dtype=torch.int32, device=dev)
    vo = dict(n_accept=i32(Bn), out_tokens=i32(Bn, k + 1), n_out=i32(Bn), next_cand=i32(Bn, k),
              next_cand_prob=torch.zeros((Bn, k), device=dev), finished=torch.zeros(Bn, dtype=torch.uint8, device=dev))
    kv_next = i32(Bn)
    ctx.space_decode_begin(state, torch.tensor([p[-1] for p in prompts], dtype=torch.int32, device=dev))
    rows = torch.arange(n_q, device=dev)[None, :]
    bidx = torch.arange(Bn, device=dev)[:, None]
    n_steps = n_new                                          # at least one token per step
    for _ in range(n_steps):                                 # no host synchronisation inside the loop
        q, Kb, Vb = tm.qkv(st["block_tokens"], st["block_pos"])
        pos = kv_len.long()[:, None] + rows                  # the block's rows go behind the verified prefix
        kc[bidx, :, pos] = Kb
        vc[bidx, :, pos] = Vb
        a = ctx.attn_args(q.contiguous(), kc, vc, kv_len, out, k, 1.0 / np.sqrt(d), status=status)
        ctx.space_attn_step(a)
        logits = tm.head(out, st["block_tokens"], st["block_pos"]).contiguous()
        v = ctx.verify_args(logits, st["cand"], st["cand_prob"], kv_len, vo["n_accept"], vo["out_tokens"], vo["n_out"],
                            vo["next_cand"], vo["next_cand_prob"], vo["finished"], k, status=status)
        c = ctx.commit_args(kc, vc, vo["n_accept"], kv_len, k, kv_len_out=kv_next, status=status)
        ctx.space_verify_commit(v, c)
        ctx.space_decode_advance(state, vo["out_tokens"], vo["n_out"], vo["next_cand"], vo["next_cand_prob"],
                                 vo["finished"], kv_next)
    torch.cuda.synchronize()
    assert int(status.abs().sum()) == 0
    n_tok = st["n_tokens"].cpu().numpy()
    toks = st["tokens"].cpu().numpy()
    Kc = bf16_bits_to_f64(kc.view(torch.int16).cpu().numpy().view(np.uint16))
    Vc = bf16_bits_to_f64(vc.view(torch.int16).cpu().numpy().view(np.uint16))
    for b, p in enumerate(prompts):
        assert n_tok[b] >= n_new                              # the token buffer filled up (that ended the sequence)
        got = p + toks[b, : n_tok[b]].tolist()
        assert got == want[b][: len(got)], f"sequence {b}"
        # the cache holds the autoregressive rows of the verified prefix, bit for bit
        L = int(kv_len[b])
        _, Kar, Var = lm.qkv(np.array(got[:L]), np.arange(L))
        assert np.array_equal(Kc[b, :, :L], Kar.transpose(1, 0, 2))
        assert np.array_equal(Vc[b, :, :L], Var.transpose(1, 0, 2))
    # the same decode by the oracle's own loop takes as many steps per token
    r = space_decode(lm, prompts[0], k, n_new)
    assert r["tokens"][: len(prompts[0]) + n_new] == want[0][: len(prompts[0]) + n_new]


def test_decode_driver_latches_eos_and_full_buffers(B):
    # <EOS> ends a sequence (the token itself is not stored); a finished sequence no longer changes
    V, H, d, k, S = 9, 2, 64, 3, 256
    lm = ToyLM(V, H, d, 1, bf16=True)
    prompt = [1, 2, 3, 4]
    free, _ = autoregressive_greedy(lm, prompt, 30)
    eos = free[len(prompt) + 6]
    want, _ = autoregressive_greedy(lm, prompt, 30, eos_id=eos)
    tm = TorchToy(lm)
    n_q, dev = (k + 1) ** 2, "cuda"
    ctx = B.Context(device=0, max_batch=1, n_q_heads=H, n_kv_heads=H, head_dim=d, k_max=k, vocab=V, s_cap=S)
    kc = torch.zeros((1, H, S, d), dtype=torch.bfloat16, device=dev)
    vc = torch.zeros_like(kc)
    kv_len = torch.tensor([len(prompt) - 1], dtype=torch.int32, device=dev)
    _, K0, V0 = tm.qkv(torch.tensor(prompt[:-1], device=dev)[None], torch.arange(len(prompt) - 1, device=dev)[None])
    kc[0, :, : len(prompt) - 1] = K0[0].permute(1, 0, 2)
    vc[0, :, : len(prompt) - 1] = V0[0].permute(1, 0, 2)
    i32 = lambda *s: torch.full(s, -7, dtype=torch.int32, device=dev)
    st = dict(tokens=i32(1, 64), n_tokens=i32(1), last_token=i32(1), cand=i32(1, k), cand_prob=torch.zeros((1, k), device=dev),
              finished=torch.full((1,), 9, dtype=torch.uint8, device=dev), block_tokens=i32(1, n_q), block_pos=i32(1, n_q))
    state = ctx.decode_state(st["tokens"], st["n_tokens"], st["last_token"], st["cand"], st["cand_prob"], kv_len,
                             st["finished"], st["block_tokens"], st["block_pos"], k, mask_token_id=V)
    out = torch.zeros((1, n_q, H, d), device=dev)
    vo = dict(n_accept=i32(1), out_tokens=i32(1, k + 1), n_out=i32(1), next_cand=i32(1, k),
              next_cand_prob=torch.zeros((1, k), device=dev), finished=torch.zeros(1, dtype=torch.uint8, device=dev))
    kv_next = i32(1)
    ctx.space_decode_begin(state, torch.tensor([prompt[-1]], dtype=torch.int32, device=dev))
    assert st["cand"].cpu().tolist() == [[0] * k] and torch.isinf(st["cand_prob"]).all() and int(st["finished"][0]) == 0
    rows = torch.arange(n_q, device=dev)[None, :]
    len_when_done = None
    for step in range(20):
        q, Kb, Vb = tm.qkv(st["block_tokens"], st["block_pos"])
        pos = kv_len.long()[:, None] + rows
        kc[torch.zeros(1, 1, dtype=torch.long, device=dev), :, pos] = Kb
        vc[torch.zeros(1, 1, dtype=torch.long, device=dev), :, pos] = Vb
        ctx.space_attn_step(ctx.attn_args(q.contiguous(), kc, vc, kv_len, out, k, 1.0 / np.sqrt(d)))
        logits = tm.head(out, st["block_tokens"], st["block_pos"]).contiguous()
        v = ctx.verify_args(logits, st["cand"], st["cand_prob"], kv_len, vo["n_accept"], vo["out_tokens"], vo["n_out"],
                            vo["next_cand"], vo["next_cand_prob"], vo["finished"], k, eos_id=eos)
        ctx.space_verify_commit(v, ctx.commit_args(kc, vc, vo["n_accept"], kv_len, k, kv_len_out=kv_next))
        ctx.space_decode_advance(state, vo["out_tokens"], vo["n_out"], vo["next_cand"], vo["next_cand_prob"],
                                 vo["finished"], kv_next)
        if int(st["finished"][0]) and len_when_done is None:
            len_when_done = (int(kv_len[0]), int(st["n_tokens"][0]))
    assert len_when_done is not None
    assert (int(kv_len[0]), int(st["n_tokens"][0])) == len_when_done     # latched: later steps change nothing
    got = prompt + st["tokens"][0, : int(st["n_tokens"][0])].cpu().tolist()
    assert got == want
