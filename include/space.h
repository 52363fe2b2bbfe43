/* libspace - one auto-correct decoding step of SPACE (arXiv 2402.11809) on
 * NVIDIA B200 (sm_100a).
 *
 * One step is the single model invocation of Algorithm 1: the block of
 * (k+1)^2 query rows (last verified token, k candidates, k+1 groups of k mask
 * tokens, Eq. 4) attends over the verified KV cache under the mask of Eq. 5,
 * the resulting logits verify the candidates and propose the next ones
 * (Algorithm 1, Sec. 3.2), and the accepted rows are compacted into the cache.
 *
 * Conventions
 *  - Every pointer named "device" must be device memory of the context's GPU;
 *    "host" pointers are ordinary host memory.  The library never takes
 *    ownership of a caller buffer; it borrows it until the work enqueued on
 *    the given stream has finished.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *    stream).  All entry points except space_step_host are asynchronous and
 *    perform no allocation and no synchronisation after space_create.
 *  - Every entry point that takes a context makes the context's device the
 *    calling thread's current device (cudaSetDevice) and leaves it current.
 *  - Return value: SPACE_OK or a negative SPACE_E_* code; nothing aborts.
 *    Conditions only the GPU can see are reported per sequence in the
 *    `status` array (bit set of SPACE_ST_*).
 *  - Block row order: row g*(k+1)+o, g = 0..k sub-block, o = 0 the real token
 *    (root for g = 0, candidate c_g otherwise), o = 1..k the o-th mask token.
 */
#ifndef SPACE_H
#define SPACE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPACE_MAX_K     7      /* (k+1)^2 <= 64 block rows                    */
#define SPACE_MAX_ROWS  64
#define SPACE_PAGE_SIZE 128    /* key rows per page of a paged cache (the kernels' key tile) */

enum {
  SPACE_OK            =  0,
  SPACE_E_INVALID_ARG = -1,    /* NULL pointer, size out of range             */
  SPACE_E_UNSUPPORTED = -2,    /* shape outside what the kernels implement    */
  SPACE_E_ALIGNMENT   = -3,    /* base pointer / stride not 16-byte aligned   */
  SPACE_E_WORKSPACE   = -4,    /* request exceeds what space_create reserved  */
  SPACE_E_CUDA        = -5,    /* a CUDA runtime or driver call failed        */
  SPACE_E_NO_DEVICE   = -6,    /* no usable sm_100 device                     */
  SPACE_E_STATIC_LIMIT = -7    /* size beyond the fixed scratch of space_verify_greedy_noalloc */
};

enum { SPACE_MASK_SAME_GROUP = 0, SPACE_MASK_EQ5_LITERAL = 1 };
enum { SPACE_MODE_GREEDY = 0, SPACE_MODE_SAMPLE = 1 };
enum { SPACE_RESAMPLE_RESIDUAL_POINTMASS = 0, SPACE_RESAMPLE_PAPER_LITERAL = 1, SPACE_RESAMPLE_RESIDUAL_DRAFT = 2 };
enum { SPACE_DTYPE_BF16 = 0, SPACE_DTYPE_F32 = 1 };
enum { SPACE_ATTN_TENSOR = 0, SPACE_ATTN_SIMT = 1, SPACE_ATTN_TENSOR_ROWS = 2 };

/* per-sequence device status bits */
enum {
  SPACE_ST_CAPACITY      = 1,  /* kv_len + (k+1)^2 exceeds the cache capacity */
  SPACE_ST_BAD_CANDIDATE = 2,  /* a candidate id outside [0, vocab): rejected */
  SPACE_ST_TIMEOUT       = 4,  /* a bounded on-chip wait expired              */
  SPACE_ST_BAD_PAGE      = 8   /* a page-table entry outside [0, n_pages): that page is not
                                  touched (attention reads zeros in its place, the commit skips
                                  the row)                                     */
};

typedef struct space_ctx space_ctx;   /* opaque; owns only its own workspace */

typedef struct {
  int32_t device;        /* CUDA device ordinal                                */
  int32_t max_batch;     /* largest batch any call will pass                   */
  int32_t n_q_heads;     /* H_q                                                */
  int32_t n_kv_heads;    /* H_kv, divides H_q; H_q/H_kv in {1,2,4,8,16}        */
  int32_t head_dim;      /* d in {64, 128}                                     */
  int32_t k_max;         /* largest k any call will pass, 1..SPACE_MAX_K       */
  int32_t vocab;         /* largest vocabulary any verify call will pass       */
  int32_t host_staging;  /* != 0: also reserve device staging for space_step_host */
  int64_t s_cap;         /* cache capacity (rows) per sequence and KV head     */
} space_config;

/* Block layout of Eq. 4 with the visibility rule of Eq. 5 and the position
 * rule of Sec. 3.2 (position = number of visible keys - 1). */
typedef struct {
  int32_t  k;
  int32_t  n_q;                          /* (k+1)^2                            */
  uint8_t  kind[SPACE_MAX_ROWS];         /* 0 real token, 1 mask token         */
  uint8_t  group[SPACE_MAX_ROWS];        /* sub-block g                        */
  uint8_t  offset[SPACE_MAX_ROWS];       /* o                                  */
  int32_t  relpos[SPACE_MAX_ROWS];       /* position id minus kv_len           */
  uint64_t mask[SPACE_MAX_ROWS];         /* bit j: row attends to block row j  */
  int32_t  target_rows[SPACE_MAX_K + 1]; /* row of the real token of sub-block t */
} space_layout_t;

/* Attention of the block over cache + block (Algorithm 1 model call restricted
 * to the attention operator; Eq. 5).  The caller has already written the
 * block's K/V rows at cache positions kv_len[b] .. kv_len[b]+n_q-1. */
typedef struct {
  int32_t batch;            /* B <= max_batch                                  */
  int32_t k;                /* candidates per sequence                         */
  int32_t mask_variant;     /* SPACE_MASK_*                                    */
  int32_t out_dtype;        /* SPACE_DTYPE_F32 or SPACE_DTYPE_BF16             */
  int32_t impl;             /* SPACE_ATTN_TENSOR (default: keys on the MMA M extent),
                               SPACE_ATTN_TENSOR_ROWS (query rows on M) or SPACE_ATTN_SIMT */
  float   scale;            /* softmax scale, normally 1/sqrt(d)               */
  const void*    q;         /* device bf16 [B, n_q, H_q, d], contiguous        */
  const void*    k_cache;   /* device bf16, element (b,h,s,:) at               */
  const void*    v_cache;   /*   b*stride_b + h*stride_h + s*stride_s (elements), d contiguous */
  int64_t kv_stride_b, kv_stride_h, kv_stride_s;  /* multiples of 8 elements   */
  const int32_t* kv_len;    /* device [B] verified lengths L_b                 */
  void*          out;       /* device [B, n_q, H_q, d] of out_dtype            */
  float*         lse;       /* device [B, H_q, n_q] natural-log sum-exp, or NULL */
  int32_t*       status;    /* device [B], OR-ed with SPACE_ST_*, or NULL      */
  /* Paged cache (the serving setting of Sec. 4.3: continuous batching over a pool of pages).
     page_table == NULL: the contiguous cache described above.  Otherwise k_cache / v_cache are
     pools of pages of SPACE_PAGE_SIZE key rows, element (page, h, r, :) at
     page*kv_stride_b + h*kv_stride_h + r*kv_stride_s, and key position s of sequence b (cache
     rows and the block's own rows L_b .. L_b+n_q-1 alike) is row s % SPACE_PAGE_SIZE of page
     page_table[b*pages_per_seq + s / SPACE_PAGE_SIZE].  A sequence's capacity is
     pages_per_seq * SPACE_PAGE_SIZE rows (it replaces s_cap in the SPACE_ST_CAPACITY check, and
     must not exceed the context's s_cap).  Entries past the pages a sequence needs are
     ignored.  Rows of its last page beyond L_b+n_q may hold anything, NaN included.            */
  const int32_t* page_table;   /* device [B, pages_per_seq] or NULL                            */
  int32_t pages_per_seq;
  int32_t n_pages;             /* pages in the pool                                            */
} space_attn_args;

/* Verification and emission (Algorithm 1 after the model call; Sec. 3.2). */
typedef struct {
  int32_t batch, k, vocab;
  int32_t logits_dtype;        /* SPACE_DTYPE_BF16 or SPACE_DTYPE_F32          */
  int32_t mode;                /* SPACE_MODE_*                                 */
  int32_t resample;            /* SPACE_RESAMPLE_* (sampling mode only)        */
  int32_t eos_id;              /* -1: no end-of-sequence handling              */
  float   temperature;         /* > 0 (sampling mode)                          */
  uint64_t seed;               /* Philox key                                   */
  const void*     logits;      /* device [B, n_q, V]; row stride below         */
  int64_t         logits_row_stride;   /* elements between rows; batch stride = n_q * row stride */
  const int32_t*  cand;        /* device [B, k]  L_c                           */
  const float*    cand_prob;   /* device [B, k]  P_c: probability the candidate was drafted with
                                  (sampling mode; ignored in greedy mode).  +inf is Algorithm 1's
                                  initial state and is always rejected; a candidate is accepted only
                                  if its id is in range, P_c > 0 and r * P_c <= Q(c) (NaN, zero and
                                  negative values are rejected).  With SPACE_RESAMPLE_RESIDUAL_POINTMASS
                                  a rejected candidate is removed from the extra token's distribution
                                  only when its P_c is exactly 1 (a point-mass draft); after the
                                  rejection of any other P_c the extra token is drawn from Q itself */
  const uint32_t* seq_id;      /* device [B] or NULL (= batch index)           */
  const int32_t*  kv_len;      /* device [B]: positions for the random counters */
  int32_t* n_accept;           /* device [B]       i*                          */
  int32_t* out_tokens;         /* device [B, k+1]  emitted tokens, -1 padded   */
  int32_t* n_out;              /* device [B]       emitted count               */
  int32_t* next_cand;          /* device [B, k]                                */
  float*   next_cand_prob;     /* device [B, k]                                */
  uint8_t* finished;           /* device [B]       1 once <EOS> was emitted    */
  int32_t* status;             /* device [B] or NULL                           */
  int32_t top_k;               /* sampling mode: 0 = unfiltered; 1..32 = every distribution that is tested
                                  against or sampled from is softmax(z/T) over its top_k largest logits
                                  (lowest token first on ties), cut to the shortest prefix, in descending
                                  order, whose probability reaches top_p, and renormalised (App. A.4 runs
                                  sampling with top-k = 10, top-p = 0.95); ignored in greedy mode        */
  float   top_p;               /* in (0, 1] when top_k > 0 (1 = no nucleus cut)                         */
  /* SPACE_RESAMPLE_RESIDUAL_DRAFT (sampling mode with top_k > 0 through space_verify / space_verify_commit;
     ignored otherwise): sampled candidates whose rejection keeps the output distribution unchanged
     (Sec. 3.2).  Candidate o of the next step is drawn from the filtered distribution D_o of its mask row,
     P_c = D_o(candidate), and D_o is handed on as a list of top_k (token, probability) pairs in descending
     order, dropped entries as (-1, 0).  After rejecting candidate i the extra token is drawn from
     norm(max(0, Q - D_i)) (from Q if that has no mass), after k acceptances from Q.                      */
  const int32_t* draft_tok;    /* device [B, k, top_k] lists the candidates were drawn from, or NULL together
                                  with draft_prob (no lists: Algorithm 1's initial state, a ~ Q)          */
  const float*   draft_prob;   /* device [B, k, top_k]; entries with a token outside [0, vocab) or a
                                  probability that is not positive and finite do not count              */
  int32_t* next_draft_tok;     /* device [B, k, top_k]: lists of the next candidates (required)          */
  float*   next_draft_prob;    /* device [B, k, top_k]                                                   */
} space_verify_args;

/* Output projection fused with verification: the end of the model call P = M(I) of
 * Algorithm 1 (logits[r, x] = <h_r, W_x> for every block row r and vocabulary token
 * x; the rows of P are softmax(logits / T)) and the loop after it (acceptance of the
 * candidates -- against the arg-max chain in greedy mode, by r <= Q/P_c with Philox
 * draws in sampling mode --, extra token, <EOS>, next candidates from the mask rows of
 * group i*; Sec. 3.2).  The logits are never written: only per-row statistics
 * (maximum, lowest arg-max, sum of exponentials, best noisy score) leave the chip. */
#define SPACE_LMHEAD_MAX_ROWS 256   /* block rows one kernel launch covers; a larger batch is
                                       split into groups of sequences, one launch (and one pass
                                       over the output embedding) per group                   */
typedef struct {
  int32_t batch, k, vocab;
  int32_t hidden_dim;          /* D, a multiple of 8                           */
  int32_t eos_id;              /* -1: no end-of-sequence handling              */
  int32_t mode;                /* SPACE_MODE_GREEDY or SPACE_MODE_SAMPLE       */
  int32_t resample;            /* SPACE_RESAMPLE_* (sampling mode)             */
  float   temperature;         /* > 0 (sampling mode)                          */
  uint64_t seed;               /* Philox key (sampling mode), keyed as in space_verify */
  const void* hidden;          /* device bf16 [B * n_q, D]: final hidden state of every block row,
                                  sequence-major, block row order               */
  int64_t hidden_row_stride;   /* elements between rows, a multiple of 8       */
  const void* weight;          /* device bf16 [V, D]: output embedding, one row per token */
  int64_t weight_row_stride;   /* elements between rows, a multiple of 8       */
  const int32_t* cand;         /* device [B, k]  L_c                           */
  const float*   cand_prob;    /* device [B, k]  P_c (sampling mode; may be NULL in greedy mode);
                                  same rules as space_verify_args.cand_prob    */
  const uint32_t* seq_id;      /* device [B] or NULL (= batch index): sequence ids of the random counters */
  const int32_t*  kv_len;      /* device [B] or NULL (= 0): positions of the random counters */
  int32_t* n_accept;           /* device [B]       i*                          */
  int32_t* out_tokens;         /* device [B, k+1]  emitted tokens, -1 padded   */
  int32_t* n_out;              /* device [B]                                   */
  int32_t* next_cand;          /* device [B, k]                                */
  float*   next_cand_prob;     /* device [B, k]  greedy: softmax (T = 1) of the token's own row;
                                  sampling: as space_verify                    */
  uint8_t* finished;           /* device [B]                                   */
  int32_t* status;             /* device [B] or NULL                           */
  float*   row_max;            /* device [B * n_q] or NULL: largest logit of every block row */
  int32_t* row_argmax;         /* device [B * n_q] or NULL: its token (lowest on ties) */
} space_lmhead_args;

/* Compaction of the accepted rows (no counterpart in Algorithm 1, which
 * re-runs the model on the whole sequence; needed by any cached forward). */
typedef struct {
  int32_t batch, k;
  void*   k_cache;             /* device bf16, same addressing as space_attn_args */
  void*   v_cache;
  int64_t kv_stride_b, kv_stride_h, kv_stride_s;
  const int32_t* n_accept;     /* device [B] from space_verify                 */
  const int32_t* kv_len;       /* device [B] lengths before the step           */
  int32_t* kv_len_out;         /* device [B] lengths after, may alias kv_len, or NULL */
  int32_t* commit_src;         /* device [B, k+1] or NULL, -1 padded           */
  int32_t* commit_dst;         /* device [B, k+1] or NULL                      */
  int32_t* status;             /* device [B] or NULL                           */
  const int32_t* page_table;   /* paged cache as in space_attn_args, or NULL (contiguous)      */
  int32_t pages_per_seq;
  int32_t n_pages;
} space_commit_args;

/* Whole step from host memory (copies in, the three stages, copies out). */
typedef struct {
  int32_t batch, k, vocab, logits_dtype, mode, resample, eos_id, mask_variant;
  float   scale, temperature;
  uint64_t seed;
  const void*    q;            /* host bf16 [B, n_q, H_q, d]                   */
  void*          k_cache;      /* host bf16 [B, H_kv, s_cap, d]; committed rows are written back */
  void*          v_cache;
  const void*    logits;       /* host [B, n_q, V] contiguous                  */
  const int32_t* cand;         /* host [B, k]                                  */
  const float*   cand_prob;    /* host [B, k]                                  */
  int32_t*       kv_len;       /* host [B]; updated in place                   */
  float*    out;               /* host f32 [B, n_q, H_q, d]                    */
  int32_t*  n_accept;          /* host [B]                                     */
  int32_t*  out_tokens;        /* host [B, k+1]                                */
  int32_t*  n_out;             /* host [B]                                     */
  int32_t*  next_cand;         /* host [B, k]                                  */
  float*    next_cand_prob;    /* host [B, k]                                  */
  uint8_t*  finished;          /* host [B]                                     */
  int32_t*  status;            /* host [B]                                     */
  int64_t*  h2d_bytes;         /* host, optional: bytes copied to the device   */
  int64_t*  d2h_bytes;         /* host, optional: bytes copied back            */
  int32_t   cache_resident;    /* 0: upload rows 0 .. kv_len+n_q-1 of every sequence's K and V.
                                  1: the KV cache is the decoder's state and already sits in the context's
                                  staging copy from an earlier call (rows 0 .. kv_len-1 of every sequence,
                                  as that call's commit left them); only the block's own rows
                                  kv_len .. kv_len+n_q-1 are uploaded                               */
  int32_t   reserved;          /* 0                                                              */
} space_host_step_args;

/* Create a context on cfg->device: validates the shape, reserves the
 * workspace (split partials, reduction scratch, counters, optional staging).
 * Errors: INVALID_ARG, UNSUPPORTED, NO_DEVICE, CUDA. */
int space_create(space_ctx** out, const space_config* cfg);
void space_destroy(space_ctx* ctx);

/* Device bytes space_create reserves for cfg (0 on invalid cfg). */
size_t space_workspace_bytes(const space_config* cfg);

/* Host only.  Eq. 4 row kinds, Eq. 5 visibility (mask_variant picks the
 * same-group reading of Sec. 3.2 / App. A.3 or Eq. 5 as printed), Sec. 3.2
 * position ids.  Errors: INVALID_ARG for k outside 1..SPACE_MAX_K. */
int space_layout(int k, int mask_variant, space_layout_t* out);

/* Eq. 5 attention of the (k+1)^2 block rows over cache + block. */
int space_attn_step(space_ctx* ctx, const space_attn_args* args, void* stream);

/* Algorithm 1 verification loop, extra token and next candidates. */
int space_verify(space_ctx* ctx, const space_verify_args* args, void* stream);

/* space_verify followed by space_kv_commit with one kernel launch less: the
 * verification kernels also move the accepted cache rows (Algorithm 1's loop
 * body after the model call, then the compaction any cached forward needs).
 * Results are those of the two separate calls, with one freedom: cache rows
 * L+i*+1 .. L+k, which lie beyond the new length and held mask-token rows of
 * the step's block that nothing reads again, are left with unspecified block
 * rows (the single-launch greedy path moves all k candidate rows while the
 * logits still stream, before i* is known).  Rows below the new length and
 * rows from L+k+1 on are exactly as space_kv_commit leaves them.
 * commit->n_accept must be
 * verify->n_accept, and batch and k must agree (INVALID_ARG otherwise); every
 * other rule of the two calls applies.  The attention that reads the cache rows
 * of this step must have been enqueued on `stream` before this call. */
int space_verify_commit(space_ctx* ctx, const space_verify_args* verify, const space_commit_args* commit,
                        void* stream);

/* Greedy verification without any allocation.  (The paper has no counterpart:
 * this entry point exists for how the library is embedded, not for the method.)
 *
 * Some hosts of this library may not allocate device memory once they are
 * running: a serving process that hands all of the GPU's memory to its own pool
 * at start-up leaves nothing for cudaMalloc, and a latency-critical decode loop
 * cannot afford the implicit device-wide synchronisation an allocation can
 * cause.  Such callers cannot use space_create, which reserves a workspace.
 * This call needs no context: its scratch (chunk results and per-sequence
 * arrival counters, SPACE_NOALLOC_MAX_BATCH * 32 KiB + 256 bytes) is a fixed
 * array inside the library image, resident on every GPU that loads the library
 * until the process exits.  It calls no cudaMalloc / cudaFree and no allocating
 * library routine.
 *
 * Same arguments, outputs and results as space_verify in SPACE_MODE_GREEDY
 * (args->mode must be SPACE_MODE_GREEDY; temperature, seed, resample ignored);
 * all (k+1)^2 logits rows are read in one kernel.  Runs on the current device.
 * Limits: batch <= SPACE_NOALLOC_MAX_BATCH, else SPACE_E_STATIC_LIMIT; k in
 * 1..SPACE_MAX_K.
 * The first call on a device is a set-up call: it looks up the array's device
 * address (cudaGetSymbolAddress) and makes the CUDA runtime load the library's
 * device code, which is when the array and the kernels take their (fixed) share
 * of device memory.  Make that call once at start-up as a warm-up - before the
 * host's own pool takes the rest of the memory, and outside any stream capture.
 * Later calls on that device load nothing and reserve nothing.
 * All calls share the one array, which keeps the last call's contents: the
 * arrival counters are cleared at the start of every call, and two calls whose
 * kernels overlap on the GPU (different streams, or several host threads) race
 * on it - serialise them. */
#define SPACE_NOALLOC_MAX_BATCH 8
int space_verify_greedy_noalloc(const space_verify_args* args, void* stream);

/* One step from hidden states (see space_lmhead_args): the output embedding is read
 * once per group of at most SPACE_LMHEAD_MAX_ROWS block rows, products on the tensor cores
 * in bf16 with fp32 accumulation, every decision taken on the fp32 accumulators (arg-max:
 * lowest token on exact ties; sampling: the same tests and Gumbel arg-maxes as
 * space_verify, with the same Philox counters).  Same outputs as space_verify on the
 * logits the projection defines.  Asynchronous on `stream`, no allocation.  One call at
 * a time per context (the calls share the context's reduction scratch).
 * Errors: INVALID_ARG (NULL pointer, sizes, mode, temperature), WORKSPACE (batch or k
 * beyond the context's), ALIGNMENT (16-byte base, strides and D multiples of 8),
 * UNSUPPORTED (one sequence alone exceeds the rows of a launch: cannot happen for k <= 7), CUDA. */
int space_lmhead_verify(space_ctx* ctx, const space_lmhead_args* args, void* stream);

/* Move accepted rows L+g(k+1) -> L+g, g = 1..i*; lengths grow by i*+1. */
int space_kv_commit(space_ctx* ctx, const space_commit_args* args, void* stream);

/* The three stages from host buffers; synchronises `stream` before returning.
 * (The logits go up and the attention output comes down on a second stream of the
 * context, ordered against `stream` by events, so that both copies overlap the kernels;
 * when the call returns everything it enqueued on either stream has finished.)
 * Needs cfg.host_staging.  Only sequence prefixes in use are copied (with
 * cache_resident: only the block's rows, see the field).  The call stages the
 * small per-sequence arrays in a pinned buffer of the context: one call at a
 * time per context.  Errors: INVALID_ARG (NULL pointer), WORKSPACE (no staging,
 * or sizes beyond cfg), CUDA. */
int space_step_host(space_ctx* ctx, const space_host_step_args* args, void* stream);

/* Device-resident state of the decoding loop (Algorithm 1 in full): the generated
 * tokens O, the candidates L_c with their probabilities P_c, the verified length, the
 * <EOS> latch, and the token and position ids of the block rows the next model call
 * evaluates (Eq. 4: the last verified token, then every candidate followed by k mask
 * tokens; Sec. 3.2: position = visible keys - 1).  All arrays are device memory owned
 * by the caller; the library only reads and writes them in the two calls below. */
typedef struct {
  int32_t batch, k;
  int32_t max_tokens;       /* capacity of `tokens` per sequence; a full buffer ends the sequence */
  int32_t mask_token_id;    /* id of the mask token [M]                                       */
  int32_t mask_variant;     /* SPACE_MASK_*: the reading of Eq. 5 the position ids follow     */
  int32_t reserved;         /* 0                                                              */
  int32_t* tokens;          /* [B, max_tokens] generated tokens (the prompt is not stored)    */
  int32_t* n_tokens;        /* [B]   how many of them                                         */
  int32_t* last_token;      /* [B]   x_l: the last verified token, whose KV is not cached yet */
  int32_t* cand;            /* [B, k] L_c                                                     */
  float*   cand_prob;       /* [B, k] P_c                                                     */
  int32_t* kv_len;          /* [B]   verified cache length L_b (set by the caller's prefill)  */
  uint8_t* finished;        /* [B]   1 once <EOS> was met or the token buffer is full; latched */
  int32_t* block_tokens;    /* [B, (k+1)^2] token ids of the next call's block rows           */
  int32_t* block_pos;       /* [B, (k+1)^2] their position ids                                */
} space_decode_state;

/* Initial state of Algorithm 1: no generated token, L_c = [0]*k, P_c = [+inf]*k (so
 * that the first step accepts nothing in sampling mode), finished = 0, and the block
 * rows of the first step.  last_prompt_token: device [B], the last token of every
 * prompt (the cache already holds the tokens before it and state->kv_len says how many).
 * Asynchronous on `stream`.  Errors: INVALID_ARG, WORKSPACE (batch beyond the context's), CUDA. */
int space_decode_begin(space_ctx* ctx, const space_decode_state* state, const int32_t* last_prompt_token,
                       void* stream);

/* End of one loop iteration of Algorithm 1, after space_verify (+ space_kv_commit) of
 * the step: appends the step's out_tokens[b, 0 .. n_out[b]-1] to O, latches finished
 * when the step met <EOS> (step_finished, from space_verify) or the buffer is full,
 * and otherwise carries next_cand / next_cand_prob into L_c / P_c, takes kv_len_next
 * (the commit's kv_len_out; must not alias state->kv_len) as the new length and writes
 * the next call's block rows.  A sequence that is already finished is left untouched:
 * the step's results for it are dropped and its length no longer grows.  All pointers
 * device memory, shapes as in space_verify_args / space_commit_args.
 * Asynchronous on `stream`, no host synchronisation: model, attention, verification,
 * commit and this call can be enqueued step after step, or captured in one CUDA graph. */
int space_decode_advance(space_ctx* ctx, const space_decode_state* state, const int32_t* out_tokens,
                         const int32_t* n_out, const int32_t* next_cand, const float* next_cand_prob,
                         const uint8_t* step_finished, const int32_t* kv_len_next, void* stream);

/* Data-loader transform of semi-autoregressive fine-tuning (Sec. 3.1, App. A.1) on a
 * padded batch of training samples, in place.  A sample (prompt of prompt_len tokens, then
 * an answer y_1..y_N of answer_len tokens, in the first slots of its row) stays as it is
 * with probability p_ar; otherwise a position m is drawn from {0..N-k}, the k answer tokens
 * from there on become mask_token_id in input_ids (labels keep their tokens), and both rows
 * are cut after the first m+k answer tokens (input_ids padded with pad_token_id, labels set
 * to ignore_index).  An answer shorter than k stays autoregressive.
 * Randomness is the caller's: two 32-bit words per sample; the sample stays autoregressive
 * when the first is below ar_threshold (= p_ar * 2^32), and m = (second * (N-k+1)) >> 32.
 * Needs no context; runs on the current device, asynchronous on `stream`.
 * Errors: INVALID_ARG (NULL pointer, sizes), CUDA. */
typedef struct {
  int32_t batch, seq_cap, k;
  int32_t mask_token_id, pad_token_id, ignore_index;
  uint32_t ar_threshold;
  int32_t reserved;            /* 0                                                   */
  int32_t* input_ids;          /* device [B, seq_cap], in place                       */
  int32_t* labels;             /* device [B, seq_cap], in place                       */
  const int32_t* prompt_len;   /* device [B]                                          */
  const int32_t* answer_len;   /* device [B]  N                                       */
  const uint32_t* rand_words;  /* device [B, 2]                                       */
  int32_t* new_len;            /* device [B] or NULL: tokens kept (prompt + answer part) */
  int32_t* mask_start;         /* device [B] or NULL: m, or -1 for an unchanged sample */
} space_sar_args;
int space_sar_sft_transform(const space_sar_args* args, void* stream);

/* Number of kernels this context has launched so far. */
int64_t space_launch_count(const space_ctx* ctx);

/* Per-kernel timing with CUDA events recorded on the launching stream around
 * every kernel (attention, merge, verify target rows, verify emit, commit,
 * projection + verify).
 * space_profile_enable(ctx, 1) starts a fresh recording (at most
 * SPACE_PROFILE_MAX_STEPS steps are kept; later ones are not recorded);
 * space_profile_enable(ctx, 0) stops it.  Do not enable during stream capture.
 * space_profile_read waits for the recorded events, writes the summed
 * milliseconds per kernel into ms[SPACE_K_COUNT] and the number of recorded launches
 * per kernel into n[SPACE_K_COUNT], and clears the recording. */
#define SPACE_PROFILE_MAX_STEPS 4096
enum { SPACE_K_ATTN = 0, SPACE_K_MERGE = 1, SPACE_K_VERIFY_TARGET = 2, SPACE_K_VERIFY_EMIT = 3,
       SPACE_K_COMMIT = 4, SPACE_K_LMHEAD = 5, SPACE_K_COUNT = 6 };
int space_profile_enable(space_ctx* ctx, int on);
int space_profile_read(space_ctx* ctx, float* ms, int64_t* n);

/* Test hook: n Philox4x32-10 blocks (Salmon et al., SC'11) for counters
 * (c0[i], c1[i], c2[i], c3[i]) and key `seed`; out receives 4 words each.
 * All pointers device memory. */
int space_debug_philox(space_ctx* ctx, uint64_t seed, int64_t n, const uint32_t* c0,
                       const uint32_t* c1, const uint32_t* c2, const uint32_t* c3,
                       uint32_t* out, void* stream);

/* Test hook for the bounded on-chip waits (every mbarrier wait of the tensor-core
 * kernels gives up after one second, sets SPACE_ST_TIMEOUT and lets the block drain;
 * no wait in the library is unbounded).  Launches one small kernel that waits, with that
 * same wait routine and a limit of limit_ns (1 .. 10^8 ns), on a barrier nothing ever
 * arrives on.  The kernel returns normally; the context stays usable.
 * out4: device int32[4], written as {status bits: SPACE_ST_TIMEOUT when the wait expired,
 * 8 if a later wait did not also give up, 16 when the block's abort flag was set;
 * the recorded site (77); microseconds the expired wait took; microseconds a second
 * wait took (about 0: a block that has given up never blocks again)}.
 * Errors: INVALID_ARG (NULL, limit out of range), CUDA. */
int space_debug_wait_timeout(space_ctx* ctx, uint64_t limit_ns, int32_t* out4, void* stream);

/* Page bookkeeping for a paged cache shared by sequences that come and go between steps (the
 * serving setting of Sec. 4.3: continuous batching).  Host-side only: it hands out pages of a pool
 * and keeps every sequence's page list; the pool's memory and the device copy of a table belong to
 * the caller.  A sequence occupies a slot from space_pager_admit to space_pager_release; a step's
 * batch is any list of slots, and space_pager_batch_table writes the table rows of those slots in
 * that order, the page_table that space_attn_args / space_commit_args take for that batch.
 * Not thread-safe.  Errors: INVALID_ARG (NULL, slot not in use, sizes out of range), WORKSPACE (no
 * free slot; not enough free pages, in which case nothing has changed). */
typedef struct space_pager space_pager;
int  space_pager_create(int32_t n_pages, int32_t pages_per_seq, int32_t max_slots, space_pager** out);
void space_pager_destroy(space_pager* p);
int  space_pager_admit(space_pager* p, int32_t* slot);          /* a free slot, holding no page yet     */
int  space_pager_reserve(space_pager* p, int32_t slot, int32_t n_rows);
                             /* pages so that cache rows 0 .. n_rows-1 of the slot exist (a sequence
                                of length L needs L + (k+1)^2 rows before its next step); pages a
                                slot already holds stay where they are                                */
int  space_pager_release(space_pager* p, int32_t slot);         /* its pages return to the pool         */
int32_t space_pager_free_pages(const space_pager* p);
int32_t space_pager_rows(const space_pager* p, int32_t slot);   /* rows reserved for the slot, -1 if unused */
int  space_pager_batch_table(const space_pager* p, const int32_t* slots, int32_t n,
                             int32_t* table_out);               /* host [n, pages_per_seq]; -1 = no page */

const char* space_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* SPACE_H */
