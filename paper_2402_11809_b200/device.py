"""Device-side copies of one step's synthetic inputs and outputs (torch is used for memory only)."""
import numpy as np
import torch

from paper_2402_11809_b200 import binding as B


def to_dev(a):
    """numpy -> cuda tensor; uint16 arrays are bf16 bit patterns."""
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    if a.dtype == np.uint32:
        return torch.from_numpy(a.view(np.int32)).cuda()
    return torch.from_numpy(a).cuda()


def bf16_to_bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def make_context(cfg, x, max_batch=None, host_staging=0):
    return B.Context(device=0, max_batch=max_batch or cfg["B"], n_q_heads=cfg["H_q"],
                     n_kv_heads=cfg["H_kv"], head_dim=cfg["d"], k_max=cfg["k"], vocab=cfg["V"],
                     host_staging=host_staging, s_cap=x["s_cap"])


class DeviceStep:
    """Device copies of one input set plus output buffers."""

    def __init__(self, cfg, x):
        self.cfg, self.k = cfg, cfg["k"]
        Bn, k, n_q = cfg["B"], cfg["k"], x["n_q"]
        self.q = to_dev(x["q"])
        self.k_cache = to_dev(x["k_cache"])
        self.v_cache = to_dev(x["v_cache"])
        self.kv_len = to_dev(x["kv_len"])
        # paged cache (workloads.to_pages): k_cache / v_cache are page pools, found through the table
        self.page_table = to_dev(x["page_table"]) if "page_table" in x else None
        self.logits = to_dev(x["logits"])
        self.cand = to_dev(x["cand"])
        self.cand_prob = to_dev(x["cand_prob"])
        self.seq_id = to_dev(x["seq_id"])
        self.scale = x["scale"]
        dev = "cuda"
        self.out = torch.full((Bn, n_q, cfg["H_q"], cfg["d"]), float("nan"), device=dev)
        self.lse = torch.full((Bn, cfg["H_q"], n_q), float("nan"), device=dev)
        self.status = torch.zeros(Bn, dtype=torch.int32, device=dev)
        self.n_accept = torch.full((Bn,), -7, dtype=torch.int32, device=dev)
        self.out_tokens = torch.full((Bn, k + 1), -7, dtype=torch.int32, device=dev)
        self.n_out = torch.full((Bn,), -7, dtype=torch.int32, device=dev)
        self.next_cand = torch.full((Bn, k), -7, dtype=torch.int32, device=dev)
        self.next_cand_prob = torch.full((Bn, k), float("nan"), device=dev)
        self.finished = torch.full((Bn,), 9, dtype=torch.uint8, device=dev)
        self.kv_len_out = torch.full((Bn,), -7, dtype=torch.int32, device=dev)
        self.commit_src = torch.full((Bn, k + 1), -7, dtype=torch.int32, device=dev)
        self.commit_dst = torch.full((Bn, k + 1), -7, dtype=torch.int32, device=dev)

    def attn(self, ctx, impl=B.ATTN_TENSOR, mask_variant=B.MASK_SAME_GROUP, out=None):
        a = ctx.attn_args(self.q, self.k_cache, self.v_cache, self.kv_len,
                          self.out if out is None else out, self.k, self.scale, lse=self.lse,
                          status=self.status, mask_variant=mask_variant, impl=impl, page_table=self.page_table)
        ctx.space_attn_step(a)
        return a

    def verify(self, ctx, mode=B.MODE_GREEDY, temperature=1.0, seed=0,
               resample=B.RESAMPLE_RESIDUAL_POINTMASS, eos_id=-1):
        a = ctx.verify_args(self.logits, self.cand, self.cand_prob, self.kv_len, self.n_accept,
                            self.out_tokens, self.n_out, self.next_cand, self.next_cand_prob,
                            self.finished, self.k, mode=mode, temperature=temperature, seed=seed,
                            resample=resample, eos_id=eos_id, seq_id=self.seq_id, status=self.status)
        ctx.space_verify(a)
        return a

    def verify_commit(self, ctx, mode=B.MODE_GREEDY, temperature=1.0, seed=0,
                      resample=B.RESAMPLE_RESIDUAL_POINTMASS, eos_id=-1, in_place=False):
        v = ctx.verify_args(self.logits, self.cand, self.cand_prob, self.kv_len, self.n_accept,
                            self.out_tokens, self.n_out, self.next_cand, self.next_cand_prob,
                            self.finished, self.k, mode=mode, temperature=temperature, seed=seed,
                            resample=resample, eos_id=eos_id, seq_id=self.seq_id, status=self.status)
        c = ctx.commit_args(self.k_cache, self.v_cache, self.n_accept, self.kv_len, self.k,
                            kv_len_out=self.kv_len if in_place else self.kv_len_out,
                            commit_src=self.commit_src, commit_dst=self.commit_dst, status=self.status, page_table=self.page_table)
        ctx.space_verify_commit(v, c)
        return v, c

    def commit(self, ctx):
        a = ctx.commit_args(self.k_cache, self.v_cache, self.n_accept, self.kv_len, self.k,
                            kv_len_out=self.kv_len_out, commit_src=self.commit_src,
                            commit_dst=self.commit_dst, status=self.status, page_table=self.page_table)
        ctx.space_kv_commit(a)
        return a
