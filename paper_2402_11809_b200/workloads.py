"""Seeded synthetic inputs for one auto-correct decoding step.

Only data generation lives here: shapes, value distributions, ragged lengths
and planted candidates.  None of the step's arithmetic (no attention, softmax,
arg-max or acceptance test) is computed in this module, so the same bytes can
be fed to any implementation of the step.

Every tensor is a numpy array; bf16 tensors are uint16 bit patterns.
"""
import numpy as np

# name -> shape parameters.  L is an inclusive range of verified cache lengths,
# p_accept an inclusive range of the per-sequence probability that a candidate
# is planted as its target row's strict maximum.
CONFIGS = {
    "tiny": dict(B=1, H_q=8, H_kv=8, d=64, L=(128, 128), k=4, V=1000,
                 logits_dtype="f32", sigma=2.0, p_accept=(0.7, 0.7),
                 mode="greedy", temperature=1.0, seed=0),
    "llama7b": dict(B=1, H_q=32, H_kv=32, d=128, L=(2048, 2048), k=5, V=32000,
                    logits_dtype="bf16", sigma=3.0, p_accept=(0.8, 0.8),
                    mode="greedy", temperature=1.0, seed=1),
    "ragged16": dict(B=16, H_q=32, H_kv=32, d=128, L=(512, 4096), k=5, V=32000,
                     logits_dtype="bf16", sigma=3.0, p_accept=(0.3, 0.9),
                     mode="greedy", temperature=1.0, seed=2),
    "gqa70b": dict(B=8, H_q=64, H_kv=8, d=128, L=(8192, 8192), k=6, V=32000,
                   logits_dtype="bf16", sigma=3.0, p_accept=(0.8, 0.8),
                   mode="greedy", temperature=1.0, seed=3),
    "sampling64": dict(B=64, H_q=32, H_kv=8, d=128, L=(1024, 16384), k=4, V=128256,
                       logits_dtype="bf16", sigma=3.0, p_accept=(0.8, 0.8),
                       mode="sample", temperature=0.8, seed=4),
}

# Logit written at a planted candidate.  Greedy: far above any N(0, sigma)
# draw, so the candidate is the row's unique maximum.  Sampling (T = 0.8,
# sigma = 3, V = 128256): exp(16/0.8) is about three times the sum of the
# other terms, so a planted candidate carries roughly 0.75 of the mass.
PLANT_GREEDY = 30.0
PLANT_SAMPLE = 16.0


def f32_to_bf16_bits(x):
    """float32 array -> round-to-nearest-even bf16 bit patterns (uint16)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def n_block_rows(k):
    return (k + 1) * (k + 1)


def resolve(name, **overrides):
    cfg = dict(CONFIGS[name])
    cfg.update(overrides)
    cfg["name"] = name
    return cfg


def _normal_bf16(rng, shape, sigma=1.0):
    x = rng.standard_normal(shape, dtype=np.float32)
    if sigma != 1.0:
        x *= np.float32(sigma)
    return f32_to_bf16_bits(x)


def make_step_inputs(cfg, set_index=0, s_cap=None, poison_tail=False):
    """One step's inputs for `cfg` (a dict from `resolve`).

    set_index picks an independent input set under the same configuration
    (used to rotate distinct sets through the L2 cache in timing runs).
    s_cap is the cache capacity per sequence (default: max length + block rows,
    rounded up to 64).  Cache rows at and beyond L_b + n_q are zero, or NaN
    patterns when poison_tail is set.
    """
    B, H_q, H_kv, d, k, V = (cfg[x] for x in ("B", "H_q", "H_kv", "d", "k", "V"))
    n_q = n_block_rows(k)
    rng = np.random.Generator(np.random.Philox(key=[cfg["seed"], set_index]))
    lo, hi = cfg["L"]
    kv_len = rng.integers(lo, hi + 1, size=B).astype(np.int32)
    if s_cap is None:
        s_cap = ((hi + n_q + 63) // 64) * 64
    fill = np.uint16(0x7FC0) if poison_tail else np.uint16(0)
    k_cache = np.full((B, H_kv, s_cap, d), fill, dtype=np.uint16)
    v_cache = np.full((B, H_kv, s_cap, d), fill, dtype=np.uint16)
    for b in range(B):
        n = int(kv_len[b]) + n_q
        k_cache[b, :, :n, :] = _normal_bf16(rng, (H_kv, n, d))
        v_cache[b, :, :n, :] = _normal_bf16(rng, (H_kv, n, d))
    q = _normal_bf16(rng, (B, n_q, H_q, d))

    if cfg["logits_dtype"] == "f32":
        logits = rng.standard_normal((B, n_q, V), dtype=np.float32) * np.float32(cfg["sigma"])
    else:
        logits = np.empty((B, n_q, V), dtype=np.uint16)
        for b in range(B):
            logits[b] = _normal_bf16(rng, (n_q, V), cfg["sigma"])
    cand = rng.integers(0, V, size=(B, k)).astype(np.int32)
    p_lo, p_hi = cfg["p_accept"]
    p_seq = rng.uniform(p_lo, p_hi, size=B)
    planted = rng.uniform(size=(B, k)) < p_seq[:, None]
    plant = PLANT_GREEDY if cfg["mode"] == "greedy" else PLANT_SAMPLE
    plant_val = np.float32(plant) if logits.dtype == np.float32 \
        else f32_to_bf16_bits(np.array([plant], dtype=np.float32))[0]
    for b in range(B):
        for i in range(k):
            if planted[b, i]:
                logits[b, i * (k + 1), int(cand[b, i])] = plant_val   # target row of c_{i+1}
    cand_prob = np.ones((B, k), dtype=np.float32)
    seq_id = np.arange(B, dtype=np.uint32)
    return dict(q=q, k_cache=k_cache, v_cache=v_cache, kv_len=kv_len, logits=logits,
                cand=cand, cand_prob=cand_prob, seq_id=seq_id, planted=planted,
                s_cap=s_cap, n_q=n_q, scale=float(1.0 / np.sqrt(d)))


PAGE_SIZE = 128


def to_pages(x, seed=0, extra_pages=3, poison=True):
    """The caches of a step's inputs as page pools (the cache of a serving engine with continuous
    batching): returns a copy of x whose k_cache / v_cache are pools [n_pages, H_kv, PAGE_SIZE, d]
    and which carries page_table [B, pages_per_seq] (int32).  Every sequence gets the pages its
    L_b + n_q rows need plus whatever its capacity (s_cap rounded up to whole pages) allows, pages
    of all sequences shuffled among `extra_pages` unused ones.  Rows that hold no key -- the tail
    of a sequence's last page, its spare pages, the unused pages -- are NaN patterns when `poison`
    is set (zero otherwise): nothing may depend on them."""
    kc, vc = x["k_cache"], x["v_cache"]
    B, H, S, d = kc.shape
    n_q = x["n_q"]
    pps = (S + PAGE_SIZE - 1) // PAGE_SIZE
    n_pages = B * pps + extra_pages
    rng = np.random.Generator(np.random.Philox(key=[seed, 12345]))
    table = rng.permutation(n_pages)[: B * pps].reshape(B, pps).astype(np.int32)
    fill = np.uint16(0x7FC0) if poison else np.uint16(0)
    kp = np.full((n_pages, H, PAGE_SIZE, d), fill, dtype=np.uint16)
    vp = np.full((n_pages, H, PAGE_SIZE, d), fill, dtype=np.uint16)
    for b in range(B):
        n = int(x["kv_len"][b]) + n_q
        for j in range((n + PAGE_SIZE - 1) // PAGE_SIZE):
            r = min(PAGE_SIZE, n - j * PAGE_SIZE)
            kp[table[b, j], :, :r, :] = kc[b, :, j * PAGE_SIZE: j * PAGE_SIZE + r, :]
            vp[table[b, j], :, :r, :] = vc[b, :, j * PAGE_SIZE: j * PAGE_SIZE + r, :]
    y = dict(x)
    y.update(k_cache=kp, v_cache=vp, page_table=table, s_cap=pps * PAGE_SIZE)
    return y


def algorithmic_bytes(cfg, kv_len, n_accept=None):
    """Bytes one step has to move at least once: K and V of the cache and block,
    Q, the attention output (as bf16), 2k+1 logits rows per sequence and the
    committed rows (read + write).  Used for roofline reporting only."""
    B, H_q, H_kv, d, k, V = (cfg[x] for x in ("B", "H_q", "H_kv", "d", "k", "V"))
    n_q = n_block_rows(k)
    esz = 4 if cfg["logits_dtype"] == "f32" else 2
    keys = int(np.sum(np.asarray(kv_len, dtype=np.int64) + n_q))
    kv = keys * H_kv * d * 2 * 2
    qo = B * n_q * H_q * d * 2 * 2
    lg = B * (2 * k + 1) * V * esz
    acc = int(np.sum(n_accept)) if n_accept is not None else 0
    cm = acc * H_kv * d * 2 * 2 * 2
    return dict(kv=kv, q_out=qo, logits=lg, commit=cm, total=kv + qo + lg + cm)


# Output-projection workloads: the step starts from the block rows' final hidden
# states and the output embedding instead of ready logits.  D is the hidden size.
LMHEAD_CONFIGS = {
    "lmhead_tiny": dict(B=1, k=4, V=1000, D=256, sigma=2.0, p_accept=(0.7, 0.7), seed=10),
    "lmhead_llama7b": dict(B=1, k=5, V=32000, D=4096, sigma=3.0, p_accept=(0.8, 0.8), seed=11),
    "lmhead_batch4": dict(B=4, k=5, V=32000, D=4096, sigma=3.0, p_accept=(0.3, 0.9), seed=12),
    "lmhead_vocab128k": dict(B=1, k=4, V=128256, D=4096, sigma=3.0, p_accept=(0.8, 0.8), seed=13),
}


def resolve_lmhead(name, **overrides):
    cfg = dict(LMHEAD_CONFIGS[name])
    cfg.update(overrides)
    cfg["name"] = name
    return cfg


def make_lmhead_inputs(cfg, set_index=0):
    """hidden [B, n_q, D] and weight [V, D] as bf16 bit patterns, candidates [B, k].

    weight ~ N(0, sigma^2 / D) and hidden ~ N(0, 1), so a logit is ~ N(0, sigma).
    With probability p per position the candidate is planted: the hidden row that
    scores it is replaced by a multiple of the candidate's own embedding row (plus
    a little noise), which makes that token the row's maximum by a wide margin
    (its logit is near PLANT_GREEDY, every other one near N(0, PLANT_GREEDY / sqrt(D)))."""
    B, k, V, D = (cfg[x] for x in ("B", "k", "V", "D"))
    n_q = n_block_rows(k)
    rng = np.random.Generator(np.random.Philox(key=[cfg["seed"], set_index]))
    w_sigma = cfg["sigma"] / np.sqrt(D)
    weight = np.empty((V, D), dtype=np.uint16)
    step = max(1, (1 << 24) // D)
    for r0 in range(0, V, step):                              # in slabs: bounded temporaries
        r1 = min(V, r0 + step)
        weight[r0:r1] = _normal_bf16(rng, (r1 - r0, D), w_sigma)
    hidden_f = rng.standard_normal((B, n_q, D), dtype=np.float32)
    cand = rng.integers(0, V, size=(B, k)).astype(np.int32)
    p_lo, p_hi = cfg["p_accept"]
    p_seq = rng.uniform(p_lo, p_hi, size=B)
    planted = rng.uniform(size=(B, k)) < p_seq[:, None]
    gain = np.float32(PLANT_GREEDY / cfg["sigma"] ** 2)
    for b in range(B):
        for i in range(k):
            if planted[b, i]:
                w_row = (weight[int(cand[b, i])].astype(np.uint32) << np.uint32(16)).view(np.float32)
                hidden_f[b, i * (k + 1)] = gain * w_row + np.float32(0.05) * hidden_f[b, i * (k + 1)]
    hidden = f32_to_bf16_bits(hidden_f)
    cand_prob = np.ones((B, k), dtype=np.float32)
    return dict(hidden=hidden, weight=weight, cand=cand, cand_prob=cand_prob, planted=planted, n_q=n_q)


def lmhead_algorithmic_bytes(cfg):
    """Bytes the projection step has to move at least once: the output embedding
    read once and the block rows' hidden states."""
    B, k, V, D = (cfg[x] for x in ("B", "k", "V", "D"))
    return dict(weight=V * D * 2, hidden=B * n_block_rows(k) * D * 2,
                total=V * D * 2 + B * n_block_rows(k) * D * 2)
