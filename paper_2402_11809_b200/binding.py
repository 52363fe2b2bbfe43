"""ctypes binding of libspace.so: the same names as include/space.h, argument
marshalling only.  Tensors are torch CUDA tensors (device memory and streams
are torch's); every step of the path runs inside the library's kernels.

Importing this module fails loudly when the compiled library is missing.
"""
import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libspace.so")

SPACE_MAX_K = 7
SPACE_MAX_ROWS = 64
OK = 0
E_INVALID_ARG, E_UNSUPPORTED, E_ALIGNMENT, E_WORKSPACE, E_CUDA, E_NO_DEVICE = -1, -2, -3, -4, -5, -6
E_STATIC_LIMIT = -7
NOALLOC_MAX_BATCH = 8
LMHEAD_MAX_ROWS = 256
MASK_SAME_GROUP, MASK_EQ5_LITERAL = 0, 1
MODE_GREEDY, MODE_SAMPLE = 0, 1
RESAMPLE_RESIDUAL_POINTMASS, RESAMPLE_PAPER_LITERAL, RESAMPLE_RESIDUAL_DRAFT = 0, 1, 2
DTYPE_BF16, DTYPE_F32 = 0, 1
ATTN_TENSOR, ATTN_SIMT, ATTN_TENSOR_ROWS = 0, 1, 2
ST_CAPACITY, ST_BAD_CANDIDATE, ST_TIMEOUT, ST_BAD_PAGE = 1, 2, 4, 8
PAGE_SIZE = 128

EXPORTS = ["space_create", "space_destroy", "space_workspace_bytes", "space_layout",
           "space_attn_step", "space_verify", "space_verify_commit", "space_verify_greedy_noalloc",
           "space_kv_commit",
           "space_lmhead_verify", "space_sar_sft_transform", "space_decode_begin", "space_decode_advance",
           "space_step_host",
           "space_launch_count", "space_profile_enable", "space_profile_read",
           "space_debug_philox", "space_debug_wait_timeout", "space_strerror",
           "space_pager_create", "space_pager_destroy", "space_pager_admit", "space_pager_reserve",
           "space_pager_release", "space_pager_free_pages", "space_pager_rows", "space_pager_batch_table"]

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2402_11809_b200.build` "
        "(there is no CPU fallback)")
lib = C.CDLL(LIB_PATH)


class Config(C.Structure):
    _fields_ = [("device", C.c_int32), ("max_batch", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("k_max", C.c_int32),
                ("vocab", C.c_int32), ("host_staging", C.c_int32), ("s_cap", C.c_int64)]


class Layout(C.Structure):
    _fields_ = [("k", C.c_int32), ("n_q", C.c_int32),
                ("kind", C.c_uint8 * SPACE_MAX_ROWS), ("group", C.c_uint8 * SPACE_MAX_ROWS),
                ("offset", C.c_uint8 * SPACE_MAX_ROWS), ("relpos", C.c_int32 * SPACE_MAX_ROWS),
                ("mask", C.c_uint64 * SPACE_MAX_ROWS), ("target_rows", C.c_int32 * (SPACE_MAX_K + 1))]


class AttnArgs(C.Structure):
    _fields_ = [("batch", C.c_int32), ("k", C.c_int32), ("mask_variant", C.c_int32),
                ("out_dtype", C.c_int32), ("impl", C.c_int32), ("scale", C.c_float),
                ("q", C.c_void_p), ("k_cache", C.c_void_p), ("v_cache", C.c_void_p),
                ("kv_stride_b", C.c_int64), ("kv_stride_h", C.c_int64), ("kv_stride_s", C.c_int64),
                ("kv_len", C.c_void_p), ("out", C.c_void_p), ("lse", C.c_void_p),
                ("status", C.c_void_p), ("page_table", C.c_void_p), ("pages_per_seq", C.c_int32),
                ("n_pages", C.c_int32)]


class VerifyArgs(C.Structure):
    _fields_ = [("batch", C.c_int32), ("k", C.c_int32), ("vocab", C.c_int32),
                ("logits_dtype", C.c_int32), ("mode", C.c_int32), ("resample", C.c_int32),
                ("eos_id", C.c_int32), ("temperature", C.c_float), ("seed", C.c_uint64),
                ("logits", C.c_void_p), ("logits_row_stride", C.c_int64),
                ("cand", C.c_void_p), ("cand_prob", C.c_void_p), ("seq_id", C.c_void_p),
                ("kv_len", C.c_void_p), ("n_accept", C.c_void_p), ("out_tokens", C.c_void_p),
                ("n_out", C.c_void_p), ("next_cand", C.c_void_p), ("next_cand_prob", C.c_void_p),
                ("finished", C.c_void_p), ("status", C.c_void_p),
                ("top_k", C.c_int32), ("top_p", C.c_float),
                ("draft_tok", C.c_void_p), ("draft_prob", C.c_void_p),
                ("next_draft_tok", C.c_void_p), ("next_draft_prob", C.c_void_p)]


class CommitArgs(C.Structure):
    _fields_ = [("batch", C.c_int32), ("k", C.c_int32), ("k_cache", C.c_void_p),
                ("v_cache", C.c_void_p), ("kv_stride_b", C.c_int64), ("kv_stride_h", C.c_int64),
                ("kv_stride_s", C.c_int64), ("n_accept", C.c_void_p), ("kv_len", C.c_void_p),
                ("kv_len_out", C.c_void_p), ("commit_src", C.c_void_p), ("commit_dst", C.c_void_p),
                ("status", C.c_void_p), ("page_table", C.c_void_p), ("pages_per_seq", C.c_int32),
                ("n_pages", C.c_int32)]


class LmHeadArgs(C.Structure):
    _fields_ = [("batch", C.c_int32), ("k", C.c_int32), ("vocab", C.c_int32),
                ("hidden_dim", C.c_int32), ("eos_id", C.c_int32), ("mode", C.c_int32),
                ("resample", C.c_int32), ("temperature", C.c_float), ("seed", C.c_uint64),
                ("hidden", C.c_void_p), ("hidden_row_stride", C.c_int64),
                ("weight", C.c_void_p), ("weight_row_stride", C.c_int64),
                ("cand", C.c_void_p), ("cand_prob", C.c_void_p), ("seq_id", C.c_void_p),
                ("kv_len", C.c_void_p), ("n_accept", C.c_void_p), ("out_tokens", C.c_void_p),
                ("n_out", C.c_void_p), ("next_cand", C.c_void_p), ("next_cand_prob", C.c_void_p),
                ("finished", C.c_void_p), ("status", C.c_void_p), ("row_max", C.c_void_p),
                ("row_argmax", C.c_void_p)]


class DecodeState(C.Structure):
    _fields_ = [("batch", C.c_int32), ("k", C.c_int32), ("max_tokens", C.c_int32),
                ("mask_token_id", C.c_int32), ("mask_variant", C.c_int32), ("reserved", C.c_int32),
                ("tokens", C.c_void_p), ("n_tokens", C.c_void_p), ("last_token", C.c_void_p),
                ("cand", C.c_void_p), ("cand_prob", C.c_void_p), ("kv_len", C.c_void_p),
                ("finished", C.c_void_p), ("block_tokens", C.c_void_p), ("block_pos", C.c_void_p)]


class SarArgs(C.Structure):
    _fields_ = [("batch", C.c_int32), ("seq_cap", C.c_int32), ("k", C.c_int32),
                ("mask_token_id", C.c_int32), ("pad_token_id", C.c_int32), ("ignore_index", C.c_int32),
                ("ar_threshold", C.c_uint32), ("reserved", C.c_int32),
                ("input_ids", C.c_void_p), ("labels", C.c_void_p), ("prompt_len", C.c_void_p),
                ("answer_len", C.c_void_p), ("rand_words", C.c_void_p), ("new_len", C.c_void_p),
                ("mask_start", C.c_void_p)]


class HostStepArgs(C.Structure):
    _fields_ = [("batch", C.c_int32), ("k", C.c_int32), ("vocab", C.c_int32),
                ("logits_dtype", C.c_int32), ("mode", C.c_int32), ("resample", C.c_int32),
                ("eos_id", C.c_int32), ("mask_variant", C.c_int32), ("scale", C.c_float),
                ("temperature", C.c_float), ("seed", C.c_uint64),
                ("q", C.c_void_p), ("k_cache", C.c_void_p), ("v_cache", C.c_void_p),
                ("logits", C.c_void_p), ("cand", C.c_void_p), ("cand_prob", C.c_void_p),
                ("kv_len", C.c_void_p), ("out", C.c_void_p), ("n_accept", C.c_void_p),
                ("out_tokens", C.c_void_p), ("n_out", C.c_void_p), ("next_cand", C.c_void_p),
                ("next_cand_prob", C.c_void_p), ("finished", C.c_void_p), ("status", C.c_void_p),
                ("h2d_bytes", C.c_void_p), ("d2h_bytes", C.c_void_p),
                ("cache_resident", C.c_int32), ("reserved", C.c_int32)]


lib.space_create.argtypes = [C.POINTER(C.c_void_p), C.POINTER(Config)]
lib.space_create.restype = C.c_int
lib.space_destroy.argtypes = [C.c_void_p]
lib.space_destroy.restype = None
lib.space_workspace_bytes.argtypes = [C.POINTER(Config)]
lib.space_workspace_bytes.restype = C.c_size_t
lib.space_layout.argtypes = [C.c_int, C.c_int, C.POINTER(Layout)]
lib.space_layout.restype = C.c_int
for _name, _arg in (("space_attn_step", AttnArgs), ("space_verify", VerifyArgs),
                    ("space_kv_commit", CommitArgs), ("space_step_host", HostStepArgs),
                    ("space_lmhead_verify", LmHeadArgs)):
    getattr(lib, _name).argtypes = [C.c_void_p, C.POINTER(_arg), C.c_void_p]
    getattr(lib, _name).restype = C.c_int
lib.space_sar_sft_transform.argtypes = [C.POINTER(SarArgs), C.c_void_p]
lib.space_sar_sft_transform.restype = C.c_int
lib.space_decode_begin.argtypes = [C.c_void_p, C.POINTER(DecodeState), C.c_void_p, C.c_void_p]
lib.space_decode_begin.restype = C.c_int
lib.space_decode_advance.argtypes = [C.c_void_p, C.POINTER(DecodeState)] + [C.c_void_p] * 7
lib.space_decode_advance.restype = C.c_int
lib.space_verify_commit.argtypes = [C.c_void_p, C.POINTER(VerifyArgs), C.POINTER(CommitArgs), C.c_void_p]
lib.space_verify_commit.restype = C.c_int
lib.space_verify_greedy_noalloc.argtypes = [C.POINTER(VerifyArgs), C.c_void_p]
lib.space_verify_greedy_noalloc.restype = C.c_int
lib.space_launch_count.argtypes = [C.c_void_p]
lib.space_launch_count.restype = C.c_int64
lib.space_profile_enable.argtypes = [C.c_void_p, C.c_int]
lib.space_profile_enable.restype = C.c_int
lib.space_profile_read.argtypes = [C.c_void_p, C.POINTER(C.c_float), C.POINTER(C.c_int64)]
lib.space_profile_read.restype = C.c_int
lib.space_debug_philox.argtypes = [C.c_void_p, C.c_uint64, C.c_int64] + [C.c_void_p] * 6
lib.space_debug_philox.restype = C.c_int
lib.space_debug_wait_timeout.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p, C.c_void_p]
lib.space_debug_wait_timeout.restype = C.c_int
lib.space_strerror.argtypes = [C.c_int]
lib.space_strerror.restype = C.c_char_p
lib.space_pager_create.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_void_p)]
lib.space_pager_create.restype = C.c_int
lib.space_pager_destroy.argtypes = [C.c_void_p]
lib.space_pager_destroy.restype = None
lib.space_pager_admit.argtypes = [C.c_void_p, C.POINTER(C.c_int32)]
lib.space_pager_admit.restype = C.c_int
lib.space_pager_reserve.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
lib.space_pager_reserve.restype = C.c_int
lib.space_pager_release.argtypes = [C.c_void_p, C.c_int32]
lib.space_pager_release.restype = C.c_int
lib.space_pager_free_pages.argtypes = [C.c_void_p]
lib.space_pager_free_pages.restype = C.c_int32
lib.space_pager_rows.argtypes = [C.c_void_p, C.c_int32]
lib.space_pager_rows.restype = C.c_int32
lib.space_pager_batch_table.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
lib.space_pager_batch_table.restype = C.c_int


class SpaceError(RuntimeError):
    def __init__(self, code):
        self.code = code
        super().__init__(f"libspace error {code}: {lib.space_strerror(code).decode()}")


def _check(code):
    if code != OK:
        raise SpaceError(code)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def space_layout(k, mask_variant=MASK_SAME_GROUP):
    lay = Layout()
    _check(lib.space_layout(k, mask_variant, C.byref(lay)))
    return lay


def space_verify_greedy_noalloc(args):
    """Greedy verification with no context and no allocation (see include/space.h)."""
    _check(lib.space_verify_greedy_noalloc(C.byref(args), _stream()))


def space_sar_sft_transform(input_ids, labels, prompt_len, answer_len, rand_words, k, mask_token_id,
                            ar_threshold, pad_token_id=0, ignore_index=-100, new_len=None, mask_start=None):
    """SAR-SFT sample transform on int32 CUDA tensors, in place (see include/space.h)."""
    a = SarArgs(batch=input_ids.shape[0], seq_cap=input_ids.shape[1], k=k, mask_token_id=mask_token_id,
                pad_token_id=pad_token_id, ignore_index=ignore_index, ar_threshold=ar_threshold, reserved=0,
                input_ids=_ptr(input_ids), labels=_ptr(labels), prompt_len=_ptr(prompt_len),
                answer_len=_ptr(answer_len), rand_words=_ptr(rand_words), new_len=_ptr(new_len),
                mask_start=_ptr(mask_start))
    _check(lib.space_sar_sft_transform(C.byref(a), _stream()))


def space_strerror(code):
    return lib.space_strerror(code).decode()


def space_workspace_bytes(**cfg):
    return lib.space_workspace_bytes(C.byref(Config(**cfg)))


class Context:
    """space_create / space_destroy plus the per-step entry points."""

    def __init__(self, device=0, max_batch=1, n_q_heads=32, n_kv_heads=32, head_dim=128, k_max=5,
                 vocab=32000, host_staging=0, s_cap=4096):
        self.cfg = Config(device=device, max_batch=max_batch, n_q_heads=n_q_heads,
                          n_kv_heads=n_kv_heads, head_dim=head_dim, k_max=k_max, vocab=vocab,
                          host_staging=host_staging, s_cap=s_cap)
        self._h = C.c_void_p()
        _check(lib.space_create(C.byref(self._h), C.byref(self.cfg)))

    def close(self):
        if self._h:
            lib.space_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def launch_count(self):
        return lib.space_launch_count(self._h)

    KERNELS = ("attn", "merge", "verify_target", "verify_emit", "commit", "lmhead")

    def space_profile_enable(self, on):
        _check(lib.space_profile_enable(self._h, int(on)))

    def space_profile_read(self):
        """{kernel: (summed ms, launches)} since profiling was enabled; clears the recording."""
        ms = (C.c_float * len(self.KERNELS))()
        n = (C.c_int64 * len(self.KERNELS))()
        _check(lib.space_profile_read(self._h, ms, n))
        return {name: (ms[i], n[i]) for i, name in enumerate(self.KERNELS)}

    # -- space_attn_step --------------------------------------------------
    def attn_args(self, q, k_cache, v_cache, kv_len, out, k, scale, lse=None, status=None,
                  mask_variant=MASK_SAME_GROUP, impl=ATTN_TENSOR, page_table=None):
        """page_table [B, pages_per_seq] int32: k_cache / v_cache are then pools [n_pages, H_kv, PAGE_SIZE, d]."""
        import torch
        assert q.is_contiguous() and out.is_contiguous()
        assert k_cache.stride() == v_cache.stride() and k_cache.stride(3) == 1
        return AttnArgs(batch=q.shape[0], k=k, mask_variant=mask_variant,
                        out_dtype=DTYPE_F32 if out.dtype == torch.float32 else DTYPE_BF16,
                        impl=impl, scale=scale, q=_ptr(q), k_cache=_ptr(k_cache), v_cache=_ptr(v_cache),
                        kv_stride_b=k_cache.stride(0), kv_stride_h=k_cache.stride(1),
                        kv_stride_s=k_cache.stride(2), kv_len=_ptr(kv_len), out=_ptr(out),
                        lse=_ptr(lse), status=_ptr(status), page_table=_ptr(page_table),
                        pages_per_seq=0 if page_table is None else page_table.shape[1],
                        n_pages=0 if page_table is None else k_cache.shape[0])

    def space_attn_step(self, args):
        _check(lib.space_attn_step(self._h, C.byref(args), _stream()))

    # -- space_verify -----------------------------------------------------
    def verify_args(self, logits, cand, cand_prob, kv_len, n_accept, out_tokens, n_out, next_cand,
                    next_cand_prob, finished, k, mode=MODE_GREEDY, temperature=1.0, seed=0,
                    resample=RESAMPLE_RESIDUAL_POINTMASS, eos_id=-1, seq_id=None, status=None,
                    top_k=0, top_p=1.0, draft_tok=None, draft_prob=None, next_draft_tok=None, next_draft_prob=None):
        import torch
        assert logits.stride(2) == 1 and logits.stride(0) == logits.shape[1] * logits.stride(1)
        return VerifyArgs(batch=logits.shape[0], k=k, vocab=logits.shape[2],
                          logits_dtype=DTYPE_F32 if logits.dtype == torch.float32 else DTYPE_BF16,
                          mode=mode, resample=resample, eos_id=eos_id, temperature=temperature,
                          seed=seed, logits=_ptr(logits), logits_row_stride=logits.stride(1),
                          cand=_ptr(cand), cand_prob=_ptr(cand_prob), seq_id=_ptr(seq_id),
                          kv_len=_ptr(kv_len), n_accept=_ptr(n_accept), out_tokens=_ptr(out_tokens),
                          n_out=_ptr(n_out), next_cand=_ptr(next_cand),
                          next_cand_prob=_ptr(next_cand_prob), finished=_ptr(finished),
                          status=_ptr(status), top_k=top_k, top_p=top_p,
                          draft_tok=_ptr(draft_tok), draft_prob=_ptr(draft_prob),
                          next_draft_tok=_ptr(next_draft_tok), next_draft_prob=_ptr(next_draft_prob))

    def space_verify(self, args):
        _check(lib.space_verify(self._h, C.byref(args), _stream()))

    def space_verify_commit(self, vargs, cargs):
        """space_verify + space_kv_commit in one launch less (see include/space.h)."""
        _check(lib.space_verify_commit(self._h, C.byref(vargs), C.byref(cargs), _stream()))

    # -- space_lmhead_verify ----------------------------------------------
    def lmhead_args(self, hidden, weight, cand, n_accept, out_tokens, n_out, next_cand, next_cand_prob,
                    finished, k, eos_id=-1, status=None, row_max=None, row_argmax=None, mode=MODE_GREEDY,
                    temperature=1.0, seed=0, resample=RESAMPLE_RESIDUAL_POINTMASS, cand_prob=None,
                    seq_id=None, kv_len=None):
        """hidden [B, n_q, D] and weight [V, D] bf16 CUDA tensors with contiguous last dimension."""
        assert hidden.stride(2) == 1 and weight.stride(1) == 1
        assert hidden.stride(0) == hidden.shape[1] * hidden.stride(1)
        return LmHeadArgs(batch=hidden.shape[0], k=k, vocab=weight.shape[0], hidden_dim=weight.shape[1],
                          eos_id=eos_id, mode=mode, resample=resample, temperature=temperature, seed=seed,
                          hidden=_ptr(hidden), hidden_row_stride=hidden.stride(1),
                          weight=_ptr(weight), weight_row_stride=weight.stride(0), cand=_ptr(cand),
                          cand_prob=_ptr(cand_prob), seq_id=_ptr(seq_id), kv_len=_ptr(kv_len),
                          n_accept=_ptr(n_accept), out_tokens=_ptr(out_tokens), n_out=_ptr(n_out),
                          next_cand=_ptr(next_cand), next_cand_prob=_ptr(next_cand_prob),
                          finished=_ptr(finished), status=_ptr(status), row_max=_ptr(row_max),
                          row_argmax=_ptr(row_argmax))

    def space_lmhead_verify(self, args):
        _check(lib.space_lmhead_verify(self._h, C.byref(args), _stream()))

    # -- space_kv_commit --------------------------------------------------
    def commit_args(self, k_cache, v_cache, n_accept, kv_len, k, kv_len_out=None, commit_src=None,
                    commit_dst=None, status=None, page_table=None):
        return CommitArgs(batch=n_accept.shape[0], k=k, k_cache=_ptr(k_cache), v_cache=_ptr(v_cache),
                          kv_stride_b=k_cache.stride(0), kv_stride_h=k_cache.stride(1),
                          kv_stride_s=k_cache.stride(2), n_accept=_ptr(n_accept), kv_len=_ptr(kv_len),
                          kv_len_out=_ptr(kv_len_out), commit_src=_ptr(commit_src),
                          commit_dst=_ptr(commit_dst), status=_ptr(status), page_table=_ptr(page_table),
                          pages_per_seq=0 if page_table is None else page_table.shape[1],
                          n_pages=0 if page_table is None else k_cache.shape[0])

    def space_kv_commit(self, args):
        _check(lib.space_kv_commit(self._h, C.byref(args), _stream()))

    # -- decoding loop state (Algorithm 1) ---------------------------------
    def decode_state(self, tokens, n_tokens, last_token, cand, cand_prob, kv_len, finished, block_tokens,
                     block_pos, k, mask_token_id, mask_variant=MASK_SAME_GROUP):
        return DecodeState(batch=tokens.shape[0], k=k, max_tokens=tokens.shape[1], mask_token_id=mask_token_id,
                           mask_variant=mask_variant, reserved=0, tokens=_ptr(tokens), n_tokens=_ptr(n_tokens),
                           last_token=_ptr(last_token), cand=_ptr(cand), cand_prob=_ptr(cand_prob),
                           kv_len=_ptr(kv_len), finished=_ptr(finished), block_tokens=_ptr(block_tokens),
                           block_pos=_ptr(block_pos))

    def space_decode_begin(self, state, last_prompt_token):
        _check(lib.space_decode_begin(self._h, C.byref(state), _ptr(last_prompt_token), _stream()))

    def space_decode_advance(self, state, out_tokens, n_out, next_cand, next_cand_prob, step_finished, kv_len_next):
        _check(lib.space_decode_advance(self._h, C.byref(state), _ptr(out_tokens), _ptr(n_out), _ptr(next_cand),
                                        _ptr(next_cand_prob), _ptr(step_finished), _ptr(kv_len_next), _stream()))

    # -- space_step_host --------------------------------------------------
    def space_step_host(self, args):
        _check(lib.space_step_host(self._h, C.byref(args), _stream()))

    def space_debug_wait_timeout(self, limit_ns, out4):
        """Let a bounded on-chip wait run out (see include/space.h); out4: int32 CUDA tensor of 4."""
        _check(lib.space_debug_wait_timeout(self._h, int(limit_ns), _ptr(out4), _stream()))

    def space_debug_philox(self, seed, c0, c1, c2, c3, out):
        _check(lib.space_debug_philox(self._h, seed, c0.numel(), _ptr(c0), _ptr(c1), _ptr(c2),
                                      _ptr(c3), _ptr(out), _stream()))


class Pager:
    """Page bookkeeping of a paged cache (space_pager_*): slots, pages, batch tables.  Host only."""

    def __init__(self, n_pages, pages_per_seq, max_slots):
        h = C.c_void_p()
        _check(lib.space_pager_create(n_pages, pages_per_seq, max_slots, C.byref(h)))
        self._h, self.pages_per_seq = h, pages_per_seq

    def close(self):
        if self._h:
            lib.space_pager_destroy(self._h)
            self._h = None

    __del__ = close

    def admit(self):
        s = C.c_int32(-1)
        _check(lib.space_pager_admit(self._h, C.byref(s)))
        return s.value

    def reserve(self, slot, n_rows):
        _check(lib.space_pager_reserve(self._h, slot, n_rows))

    def release(self, slot):
        _check(lib.space_pager_release(self._h, slot))

    @property
    def free_pages(self):
        return lib.space_pager_free_pages(self._h)

    def rows(self, slot):
        return lib.space_pager_rows(self._h, slot)

    def batch_table(self, slots):
        import numpy as np
        sl = np.ascontiguousarray(slots, dtype=np.int32)
        out = np.empty((len(sl), self.pages_per_seq), dtype=np.int32)
        _check(lib.space_pager_batch_table(self._h, sl.ctypes.data_as(C.c_void_p), len(sl),
                                           out.ctypes.data_as(C.c_void_p)))
        return out
